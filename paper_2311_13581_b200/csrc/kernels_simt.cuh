// Plain CUDA-core kernels of the decoder step: row assembly, RMSNorm, a warp-per-feature
// GEMM, rotary + KV append, attention, SwiGLU.  They are the whole path of the float32
// configuration (exact float32 products, where tensor cores would round to tf32) and serve
// every configuration for the small element-wise steps.
#pragma once
#include "pass_common.cuh"

namespace pass {

// ---------------------------------------------------------------------------------------
// Row assembly (section "Look-ahead embeddings": the L look-ahead tokens are appended after
// the real tokens; Algorithm 1: drafts are fed as ordinary tokens in the validation call).
// Step mode: sequence b contributes M = 1 + 2k rows
//   [pending, d_1..d_m, LA_1..LA_k, pad...] at positions len_b, len_b+1, ...
// Pad rows (present when m = 0) repeat look-ahead rows; they sit after every live row, so
// the causal mask keeps them from influencing anything, and their outputs are never read.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int effective_m(const SeqState& st, const StepParams* sp) {
    const int k = sp->k;
    return (sp->drop_drafts || st.m != k) ? 0 : st.m;
}

template <typename WT>
__global__ void k_assemble_step(const WT* __restrict__ tok_emb, const WT* __restrict__ la_emb,
                                const SeqState* __restrict__ states, const StepParams* __restrict__ sp,
                                int M, int d, int vocab, float* __restrict__ h,
                                int* __restrict__ row_seq, int* __restrict__ row_pos) {
    const int r = blockIdx.x, b = r / M, i = r % M;
    const SeqState& st = states[b];
    const int k = sp->k;
    const int m = effective_m(st, sp);
    const WT* src;
    if (i == 0) {
        src = tok_emb + (size_t)min(max(st.pending, 0), vocab - 1) * d;
    } else if (i <= m) {
        src = tok_emb + (size_t)min(max(st.drafts[i - 1], 0), vocab - 1) * d;
    } else {
        const int j = (i - m - 1) % max(k, 1);
        src = la_emb + (size_t)j * d;
    }
    for (int c = threadIdx.x; c < d; c += blockDim.x) h[(size_t)r * d + c] = to_f32<WT>(src[c]);
    if (threadIdx.x == 0) {
        row_seq[r] = b;
        row_pos[r] = st.kv_len + i;
    }
}

// Token mode: n rows of one sequence; id >= vocab selects look-ahead embedding id - vocab.
template <typename WT>
__global__ void k_assemble_tokens(const WT* __restrict__ tok_emb, const WT* __restrict__ la_emb,
                                  const SeqState* __restrict__ states, const int* __restrict__ ids,
                                  int seq, int d, int vocab, float* __restrict__ h,
                                  int* __restrict__ row_seq, int* __restrict__ row_pos) {
    const int r = blockIdx.x;
    const int id = ids[r];
    const WT* src = id < vocab ? tok_emb + (size_t)id * d : la_emb + (size_t)(id - vocab) * d;
    for (int c = threadIdx.x; c < d; c += blockDim.x) h[(size_t)r * d + c] = to_f32<WT>(src[c]);
    if (threadIdx.x == 0) {
        row_seq[r] = seq;
        row_pos[r] = states[seq].kv_len + r;
    }
}

// cos/sin of pos * theta^(-2i/d_head) per row, in float64 then rounded: shared by all layers.
__global__ void k_rope_table(const int* __restrict__ row_pos, const double* __restrict__ inv_freq,
                             int half, float2* __restrict__ cs) {
    const int r = blockIdx.x;
    const double p = (double)row_pos[r];
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        double s, c;
        sincos(p * inv_freq[i], &s, &c);
        cs[(size_t)r * half + i] = make_float2((float)c, (float)s);
    }
}

// ---------------------------------------------------------------------------------------
// RMSNorm: y = x * g / sqrt(mean(x^2) + eps)
// ---------------------------------------------------------------------------------------
template <typename WT>
__global__ void k_rmsnorm(const float* __restrict__ x, const WT* __restrict__ g, int d, float eps,
                          float* __restrict__ y) {
    __shared__ float red[32];
    const int r = blockIdx.x;
    const float* xr = x + (size_t)r * d;
    float ss = 0.f;
    for (int c = threadIdx.x; c < d; c += blockDim.x) ss += xr[c] * xr[c];
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x < 32) {
        float v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
        v = warp_sum(v);
        if (threadIdx.x == 0) red[0] = rsqrtf(v / (float)d + eps);
    }
    __syncthreads();
    const float inv = red[0];
    for (int c = threadIdx.x; c < d; c += blockDim.x)
        y[(size_t)r * d + c] = xr[c] * inv * to_f32<WT>(g[c]);
}

// ---------------------------------------------------------------------------------------
// Y[r][n] (+)= sum_k X[r][k] W[n][k]; one warp per output feature, RT rows per pass.
// ---------------------------------------------------------------------------------------
template <typename WT> struct WVec;
template <> struct WVec<float> {
    static constexpr int N = 4;
    __device__ static void load(const float* p, float (&w)[4]) {
        const float4 v = *reinterpret_cast<const float4*>(p);
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
    }
};
template <> struct WVec<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static void load(const __nv_bfloat16* p, float (&w)[8]) {
        const uint4 v = *reinterpret_cast<const uint4*>(p);
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            w[2 * i] = __uint_as_float(u[i] << 16);
            w[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
        }
    }
};

template <typename WT, int RT>
__global__ void k_gemm_simt(const float* __restrict__ X, int ldx, const WT* __restrict__ W, int N,
                            int K, int R, float* __restrict__ Y, int ldy, int accumulate) {
    constexpr int VN = WVec<WT>::N;
    const int lane = threadIdx.x & 31;
    const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (n >= N) return;
    const WT* wrow = W + (size_t)n * K;
    for (int r0 = 0; r0 < R; r0 += RT) {
        float acc[RT];
#pragma unroll
        for (int i = 0; i < RT; i++) acc[i] = 0.f;
        for (int k = lane * VN; k < K; k += 32 * VN) {
            float w[VN];
            WVec<WT>::load(wrow + k, w);
#pragma unroll
            for (int i = 0; i < RT; i++) {
                if (r0 + i < R) {
                    const float* xp = X + (size_t)(r0 + i) * ldx + k;
#pragma unroll
                    for (int j = 0; j < VN; j += 4) {
                        const float4 xv = *reinterpret_cast<const float4*>(xp + j);
                        acc[i] = fmaf(xv.x, w[j], acc[i]);
                        acc[i] = fmaf(xv.y, w[j + 1], acc[i]);
                        acc[i] = fmaf(xv.z, w[j + 2], acc[i]);
                        acc[i] = fmaf(xv.w, w[j + 3], acc[i]);
                    }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < RT; i++) {
            const float s = warp_sum(acc[i]);
            if (lane == 0 && r0 + i < R) {
                float* yp = Y + (size_t)(r0 + i) * ldy + n;
                *yp = accumulate ? *yp + s : s;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// Rotary positions on adjacent pairs (2i, 2i+1) of q and k, then append k, v to the cache at
// the row's position (the cache rows of rejected drafts and look-ahead rows are simply
// overwritten by the next call - that is the rollback).
// qkv: [R][3d] float32 (q | k | v); q is rotated in place.
// ---------------------------------------------------------------------------------------
template <typename KVT>
__global__ void k_rope_kv(float* __restrict__ qkv, const float2* __restrict__ cs,
                          const int* __restrict__ row_seq, const int* __restrict__ row_pos,
                          ModelDims md, int layer, KVT* __restrict__ kc, KVT* __restrict__ vc) {
    const int r = blockIdx.x, d = md.d, dh = md.dh, half = dh / 2;
    const int seq = row_seq[r], pos = row_pos[r];
    float* q = qkv + (size_t)r * 3 * d;
    float* k = q + d;
    float* v = k + d;
    for (int p = threadIdx.x; p < d / 2; p += blockDim.x) {
        const int head = p / half, i = p % half;
        const float2 t = cs[(size_t)r * half + i];
        const float q0 = q[2 * p], q1 = q[2 * p + 1];
        q[2 * p] = q0 * t.x - q1 * t.y;
        q[2 * p + 1] = q0 * t.y + q1 * t.x;
        const float k0 = k[2 * p], k1 = k[2 * p + 1];
        const size_t o = kv_index(md, layer, seq, head, pos) + 2 * i;
        kc[o] = from_f32<KVT>(k0 * t.x - k1 * t.y);
        kc[o + 1] = from_f32<KVT>(k0 * t.y + k1 * t.x);
        vc[o] = from_f32<KVT>(v[2 * p]);
        vc[o + 1] = from_f32<KVT>(v[2 * p + 1]);
    }
}

// ---------------------------------------------------------------------------------------
// Attention, one CTA per (head, row): row r attends to cached positions 0 .. pos_r.
// Each warp walks keys warp, warp+4, ... with an online softmax; warps are merged at the end.
// ---------------------------------------------------------------------------------------
// q: [R][ldq] float32 (rotated queries).  SPLIT = false: out is float32 [R][d];
// SPLIT = true: out is bf16 [rows][d] holding hi parts in rows r and lo parts in rows lo_row0 + r.
template <typename KVT, int DH, bool SPLIT>
__global__ void __launch_bounds__(128)
k_attn_simple(const float* __restrict__ qbuf, int ldq, const int* __restrict__ row_seq,
              const int* __restrict__ row_pos, ModelDims md, int layer,
              const KVT* __restrict__ kc, const KVT* __restrict__ vc, void* __restrict__ out_,
              int lo_row0) {
    constexpr int E = DH / 32;
    const int head = blockIdx.x, r = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int seq = row_seq[r], n_keys = row_pos[r] + 1;
    const float scale = rsqrtf((float)DH);
    float q[E];
#pragma unroll
    for (int e = 0; e < E; e++)
        q[e] = qbuf[(size_t)r * ldq + head * DH + lane * E + e] * scale;
    const KVT* kb = kc + kv_index(md, layer, seq, head, 0);
    const KVT* vb = vc + kv_index(md, layer, seq, head, 0);
    float mx = -INFINITY, l = 0.f, acc[E];
#pragma unroll
    for (int e = 0; e < E; e++) acc[e] = 0.f;
    for (int j = warp; j < n_keys; j += 4) {
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < E; e++) s += q[e] * to_f32<KVT>(kb[(size_t)j * DH + lane * E + e]);
        s = warp_sum(s);
        const float mn = fmaxf(mx, s);
        const float corr = __expf(mx - mn), p = __expf(s - mn);
        l = l * corr + p;
#pragma unroll
        for (int e = 0; e < E; e++)
            acc[e] = acc[e] * corr + p * to_f32<KVT>(vb[(size_t)j * DH + lane * E + e]);
        mx = mn;
    }
    __shared__ float s_m[4], s_l[4], s_acc[4][DH];
    if (lane == 0) { s_m[warp] = mx; s_l[warp] = l; }
#pragma unroll
    for (int e = 0; e < E; e++) s_acc[warp][lane * E + e] = acc[e];
    __syncthreads();
    const float M = fmaxf(fmaxf(s_m[0], s_m[1]), fmaxf(s_m[2], s_m[3]));
    float L = 0.f;
#pragma unroll
    for (int w = 0; w < 4; w++) L += s_l[w] * __expf(s_m[w] - M);
    for (int c = threadIdx.x; c < DH; c += 128) {
        float o = 0.f;
#pragma unroll
        for (int w = 0; w < 4; w++) o += s_acc[w][c] * __expf(s_m[w] - M);
        o /= L;
        if constexpr (SPLIT) {
            __nv_bfloat16* out = (__nv_bfloat16*)out_;
            const __nv_bfloat16 hi = __float2bfloat16_rn(o);
            out[(size_t)r * md.d + head * DH + c] = hi;
            out[(size_t)(lo_row0 + r) * md.d + head * DH + c] = __float2bfloat16_rn(o - __bfloat162float(hi));
        } else {
            ((float*)out_)[(size_t)r * md.d + head * DH + c] = o;
        }
    }
}

// After row assembly on the tensor-core path: the input of the first GEMM and the partial sums of
// squares that its epilogue turns into the RMSNorm factor.  x = h * g is split into bf16 hi + lo
// rows; sumsq[t][r] = sum of h^2 over features 128t .. 128t+127.
__global__ void __launch_bounds__(128)
k_split_norm_input(const float* __restrict__ h, const __nv_bfloat16* __restrict__ g, int d,
                   __nv_bfloat16* __restrict__ xn, int lo_row0, float* __restrict__ sumsq, int tile_rows) {
    __shared__ float red[4];
    const int r = blockIdx.x;
    // tile_rows > 0: token tiles of tile_rows hi rows followed by their lo rows (prompt chunks with hi + lo parts)
    const int xr = tile_rows ? (r / tile_rows) * 2 * tile_rows + r % tile_rows : r;
    for (int t = 0; t < d / 128; t++) {
        const int n = t * 128 + threadIdx.x;
        const float v = h[(size_t)r * d + n];
        const float x = v * __bfloat162float(g[n]);
        const __nv_bfloat16 hi = __float2bfloat16_rn(x);
        xn[(size_t)xr * d + n] = hi;
        if (lo_row0 >= 0) xn[(size_t)(lo_row0 + xr) * d + n] = __float2bfloat16_rn(x - __bfloat162float(hi));   // < 0: plain bf16 rows
        const float ss = warp_sum(v * v);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        if (threadIdx.x == 0) sumsq[(size_t)t * kRowsCap + r] = red[0] + red[1] + red[2] + red[3];
    }
}

// The three kernels ahead of a decode step's first GEMM in one: row assembly (k_assemble_step), rotary
// table (k_rope_table) and the first layer's norm input (k_split_norm_input), same arithmetic.  Grid
// (rows, d / 1024), 256 threads: thread t of chunk c handles columns 1024 c + 256 j + t, j = 0..3, so warps
// 0-3 (4-7) of pass j cover tile 8 c + 2 j (+ 1) of 128 columns.
__global__ void __launch_bounds__(256)
k_step_input(const __nv_bfloat16* __restrict__ tok_emb, const __nv_bfloat16* __restrict__ la_emb,
             const SeqState* __restrict__ states, const StepParams* __restrict__ sp, int M, int d, int vocab,
             float* __restrict__ h, int* __restrict__ row_seq, int* __restrict__ row_pos,
             const double* __restrict__ inv_freq, int half, float2* __restrict__ cs,
             const __nv_bfloat16* __restrict__ g, __nv_bfloat16* __restrict__ xn, int lo_row0,
             float* __restrict__ sumsq) {
    __shared__ float red[4][8];
    const int r = blockIdx.x, chunk = blockIdx.y, b = r / M, i = r % M;
    const SeqState& st = states[b];
    const int k = sp->k;
    const int m = effective_m(st, sp);
    const __nv_bfloat16* src;
    if (i == 0) {
        src = tok_emb + (size_t)min(max(st.pending, 0), vocab - 1) * d;
    } else if (i <= m) {
        src = tok_emb + (size_t)min(max(st.drafts[i - 1], 0), vocab - 1) * d;
    } else {
        const int j = (i - m - 1) % max(k, 1);
        src = la_emb + (size_t)j * d;
    }
    float v[4];
#pragma unroll
    for (int j = 0; j < 4; j++) {
        const int c = chunk * 1024 + j * 256 + threadIdx.x;
        v[j] = c < d ? __bfloat162float(src[c]) : 0.f;
    }
#pragma unroll
    for (int j = 0; j < 4; j++) {
        const int c = chunk * 1024 + j * 256 + threadIdx.x;
        if (c < d) {
            h[(size_t)r * d + c] = v[j];
            const float x = v[j] * __bfloat162float(g[c]);
            const __nv_bfloat16 hi = __float2bfloat16_rn(x);
            xn[(size_t)r * d + c] = hi;
            xn[(size_t)(lo_row0 + r) * d + c] = __float2bfloat16_rn(x - __bfloat162float(hi));
        }
        const float ss = warp_sum(v[j] * v[j]);
        if ((threadIdx.x & 31) == 0) red[j][threadIdx.x >> 5] = ss;
    }
    __syncthreads();
    if (threadIdx.x < 8) {
        const int j = threadIdx.x >> 1, w0 = (threadIdx.x & 1) * 4, t = chunk * 8 + threadIdx.x;
        if (t * 128 < d) sumsq[(size_t)t * kRowsCap + r] = red[j][w0] + red[j][w0 + 1] + red[j][w0 + 2] + red[j][w0 + 3];
    }
    if (chunk == 0) {
        const int pos = st.kv_len + i;
        if (threadIdx.x == 0) {
            row_seq[r] = b;
            row_pos[r] = pos;
        }
        for (int q = threadIdx.x; q < half; q += blockDim.x) {
            double sn, cn;
            sincos((double)pos * inv_freq[q], &sn, &cn);
            cs[(size_t)r * half + q] = make_float2((float)cn, (float)sn);
        }
    }
}

// Plain split of float32 rows into bf16 hi + lo rows (no gain).
__global__ void k_split_rows(const float* __restrict__ x, int K, __nv_bfloat16* __restrict__ out, int lo_row0) {
    const int r = blockIdx.y;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= K) return;
    const float v = x[(size_t)r * K + c];
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    out[(size_t)r * K + c] = hi;
    out[(size_t)(lo_row0 + r) * K + c] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// Weight matrix W[N][K] (row-major bf16) copied into the order the streaming GEMM reads it:
// [tile][k-block][box_rows][64] - every (tile, k-block) box is one contiguous run of box_rows * 128
// bytes instead of box_rows pieces of 128 bytes that lie a whole matrix row apart.  Rows and columns
// beyond the matrix are zeros.  One thread moves 16 bytes.
__global__ void k_pack_weight(const __nv_bfloat16* __restrict__ W, int N, int K, int box_rows, int n_tiles,
                              int kb_per_tile, __nv_bfloat16* __restrict__ out) {
    const size_t total = (size_t)n_tiles * kb_per_tile * box_rows * 8;      // 16-byte chunks
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c8 = (int)(i & 7);
        const size_t rest = i >> 3;
        const int r = (int)(rest % box_rows);
        const size_t box = rest / box_rows;
        const int kb = (int)(box % kb_per_tile), tile = (int)(box / kb_per_tile);
        const int row = tile * box_rows + r, col = kb * 64 + c8 * 8;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (row < N && col < K) v = *reinterpret_cast<const uint4*>(W + (size_t)row * K + col);   // K is a multiple of 8
        reinterpret_cast<uint4*>(out)[i] = v;
    }
}

// F[r][j] = silu(G[r][j]) * U[r][j], GU: [R][2f] (gate | up)
__global__ void k_swiglu(const float* __restrict__ gu, int f, float* __restrict__ act) {
    const int r = blockIdx.y;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= f) return;
    const float g = gu[(size_t)r * 2 * f + j], u = gu[(size_t)r * 2 * f + f + j];
    act[(size_t)r * f + j] = g / (1.f + __expf(-g)) * u;
}

}  // namespace pass
