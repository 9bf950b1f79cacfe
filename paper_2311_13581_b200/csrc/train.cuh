// Kernels of the look-ahead-embedding training step (Supplementary material, "Training details": the model
// is frozen, only the L look-ahead input embeddings are trained, the loss is taken on their outputs).
//
// Because of the causal mask nothing but the look-ahead rows depends on the look-ahead embeddings, so the
// backward pass runs over those rows alone (L per sequence, at most 64 in a batch): the prompt rows only
// contribute their cached keys and values, which are constants here.  The linear layers of both passes are the
// weight-streaming tensor-core GEMM (the backward ones on transposed copies of the weights); what is left is
// small and lives in this file as plain kernels: loss, the backward of RMSNorm, SwiGLU, rotary positions and
// attention, the sum over the batch, AdamW.
#pragma once
#include "pass_common.cuh"

namespace pass {

// Transposed weights in streaming order.  The transposed matrix Wt [N][K] is made of n_src source matrices
// side by side along K: Wt[row][m * rows_src + i] = src_m[i][row], src_m being [rows_src][N] row-major
// (Q, K, V stacked for the backward of the QKV projection, gate and up for that of the feed-forward input).
// Output: boxes of 128 x 64 elements, [tile][k-block][128][64], zeros beyond the matrix.  One block per box,
// thread r = row r of the box: its loads run along a source row together with the other threads'.
struct PackTSources { const __nv_bfloat16* src[3]; };
__global__ void __launch_bounds__(128)
k_pack_weight_t(PackTSources s, int n_src, int rows_src, int N, int kb_per_tile, __nv_bfloat16* __restrict__ out) {
    const int box = blockIdx.x, tile = box / kb_per_tile, kb = box % kb_per_tile;
    const int row = tile * 128 + threadIdx.x;
    const int K = n_src * rows_src;
    __align__(16) __nv_bfloat16 v[64];
#pragma unroll
    for (int c = 0; c < 64; c++) {
        const int col = kb * 64 + c;
        float x = 0.f;
        if (row < N && col < K) x = __bfloat162float(s.src[col / rows_src][(size_t)(col % rows_src) * N + row]);
        v[c] = __float2bfloat16_rn(x);      // exact: the value was a bf16
    }
    uint4* dst = reinterpret_cast<uint4*>(out + ((size_t)box * 128 + threadIdx.x) * 64);
#pragma unroll
    for (int q = 0; q < 8; q++) dst[q] = reinterpret_cast<const uint4*>(v)[q];
}

// Rows of the training forward: row r = b * L + t is look-ahead token t of sequence b, at position len_b + t.
__global__ void k_train_rows(const SeqState* __restrict__ states, const float* __restrict__ la_master, int L, int d,
                             float* __restrict__ h, int* __restrict__ row_seq, int* __restrict__ row_pos) {
    const int r = blockIdx.x, b = r / L, t = r % L;
    if (threadIdx.x == 0) {
        row_seq[r] = b;
        row_pos[r] = states[b].kv_len + t;
    }
    for (int c = threadIdx.x; c < d; c += blockDim.x) h[(size_t)r * d + c] = la_master[(size_t)t * d + c];
}

__global__ void k_add_rows(float* __restrict__ h, const float* __restrict__ y, size_t n) {
    const size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (i < n) h[i] += y[i];
}

// gate | up as the interleaved GEMM leaves them: block t of 128 columns = gate features 64t.. then up features 64t..
__device__ __forceinline__ size_t il_gate(int j) { return (size_t)(j >> 6) * 128 + (j & 63); }
__global__ void k_swiglu_il(const float* __restrict__ gu, int ld, int f, float* __restrict__ act) {
    const int r = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= f) return;
    const float g = gu[(size_t)r * ld + il_gate(j)], u = gu[(size_t)r * ld + il_gate(j) + 64];
    act[(size_t)r * f + j] = g / (1.f + __expf(-g)) * u;
}
// d act -> [d gate (f) | d up (f)] per row
__global__ void k_swiglu_il_bwd(const float* __restrict__ gu, int ld, int f, const float* __restrict__ dact,
                                float* __restrict__ dgu) {
    const int r = blockIdx.y, j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= f) return;
    const float g = gu[(size_t)r * ld + il_gate(j)], u = gu[(size_t)r * ld + il_gate(j) + 64];
    const float s = 1.f / (1.f + __expf(-g)), da = dact[(size_t)r * f + j];
    dgu[(size_t)r * 2 * f + j] = da * u * s * (1.f + g * (1.f - s));
    dgu[(size_t)r * 2 * f + f + j] = da * g * s;
}

// Cross entropy of row r against target[r], scaled: loss_row[r] = lse - z[target]; dz = (softmax - onehot) * scale.
__global__ void __launch_bounds__(256)
k_ce_grad(const float* __restrict__ logits, const int* __restrict__ target, int V, float scale,
          float* __restrict__ dlogits, float* __restrict__ loss_row) {
    __shared__ float red[8];
    __shared__ float s_m, s_l;
    const int r = blockIdx.x;
    const float* z = logits + (size_t)r * V;
    float m = -INFINITY;
    for (int i = threadIdx.x; i < V; i += 256) m = fmaxf(m, z[i]);
    m = warp_max(m);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) { float x = red[0]; for (int i = 1; i < 8; i++) x = fmaxf(x, red[i]); s_m = x; }
    __syncthreads();
    m = s_m;
    float l = 0.f;
    for (int i = threadIdx.x; i < V; i += 256) l += expf(z[i] - m);
    l = warp_sum(l);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = l;
    __syncthreads();
    if (threadIdx.x == 0) { float x = 0.f; for (int i = 0; i < 8; i++) x += red[i]; s_l = x; }
    __syncthreads();
    const float inv = 1.f / s_l;
    const int tg = target[r];
    for (int i = threadIdx.x; i < V; i += 256)
        dlogits[(size_t)r * V + i] = (expf(z[i] - m) * inv - (i == tg ? 1.f : 0.f)) * scale;
    if (threadIdx.x == 0) loss_row[r] = m + logf(s_l) - z[tg];
}

// y = x r g, r = (mean x^2 + eps)^(-1/2):  dx = r g dy - x r^3 mean(g dy x).  out[r] = add[r] + dx (add may be out).
template <typename WT>
__global__ void __launch_bounds__(256)
k_rmsnorm_bwd(const float* __restrict__ dy, const float* __restrict__ x, const WT* __restrict__ g, int d, float eps,
              const float* __restrict__ add, float* __restrict__ out) {
    __shared__ float red[2][8];
    const int r = blockIdx.x;
    float ss = 0.f, ux = 0.f;
    for (int i = threadIdx.x; i < d; i += 256) {
        const float xv = x[(size_t)r * d + i];
        ss += xv * xv;
        ux += dy[(size_t)r * d + i] * to_f32<WT>(g[i]) * xv;
    }
    ss = warp_sum(ss);
    ux = warp_sum(ux);
    if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = ss; red[1][threadIdx.x >> 5] = ux; }
    __syncthreads();
    float tss = 0.f, tux = 0.f;
    for (int i = 0; i < 8; i++) { tss += red[0][i]; tux += red[1][i]; }
    const float rr = rsqrtf(tss / d + eps), k = rr * rr * rr * (tux / d);
    for (int i = threadIdx.x; i < d; i += 256) {
        const size_t o = (size_t)r * d + i;
        const float dx = rr * to_f32<WT>(g[i]) * dy[o] - x[o] * k;
        out[o] = (add ? add[o] : 0.f) + dx;
    }
}

// Inverse rotation of the query and key parts of dqkv [R][3d] (the rotation is linear and orthogonal, so its
// derivative is its transpose): for the pair (2i, 2i+1), dx0 = dy0 c + dy1 s, dx1 = dy1 c - dy0 s.
__global__ void k_rope_bwd(float* __restrict__ dqkv, const float2* __restrict__ cs, int d, int dh) {
    const int r = blockIdx.x, half = dh / 2;
    for (int p = threadIdx.x; p < d; p += blockDim.x) {          // p: pair index over q (d/2 pairs) then k (d/2 pairs)
        const int which = p / (d / 2), q = p % (d / 2);
        const float2 c = cs[(size_t)r * half + q % half];
        float* v = dqkv + (size_t)r * 3 * d + (size_t)which * d + 2 * q;
        const float y0 = v[0], y1 = v[1];
        v[0] = y0 * c.x + y1 * c.y;
        v[1] = y1 * c.x - y0 * c.y;
    }
}

// Backward of attention for the look-ahead rows of one (sequence, head).  Rows t = 0..L-1 at positions len + t;
// row t attends keys 0 .. len + t.  q (rotated), k, v rows of the look-ahead tokens are in qkv [R][3d]; all keys
// and values (the look-ahead rows' included, as the forward stored them) are in the cache.  With P = softmax(S),
// S = q k^T / sqrt(dh), dP = dO V^T:  dS = P (dP - sum_j P dP),  dq = dS K / sqrt(dh),  dk_j = sum_t dS_tj q_t /
// sqrt(dh),  dv_j = sum_t P_tj dO_t — the last two only for the look-ahead keys (the others are constants).
// scratch: [sequences * heads][2][L][n_max] floats (P, then dS).  Grid (heads, sequences), 128 threads.
template <typename KVT, int DH>
__global__ void __launch_bounds__(128)
k_attn_la_bwd(const float* __restrict__ qkv, const float* __restrict__ dattn, const SeqState* __restrict__ states,
              ModelDims md, int layer, int L, const KVT* __restrict__ kc, const KVT* __restrict__ vc,
              float* __restrict__ scratch, int n_max, float* __restrict__ dqkv) {
    __shared__ float s_q[PASS_MAX_LOOKAHEAD][DH], s_do[PASS_MAX_LOOKAHEAD][DH];
    __shared__ float s_red[4];
    __shared__ float s_stat[PASS_MAX_LOOKAHEAD][3];          // max, 1 / sum, D = sum_j P dP
    const int head = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, d = md.d;
    const int len = states[b].kv_len;                        // cached positions before the look-ahead rows
    const float scale = rsqrtf((float)DH);
    const KVT* K = kc + kv_index(md, layer, b, head, 0);
    const KVT* V = vc + kv_index(md, layer, b, head, 0);
    float* P = scratch + ((size_t)(b * md.H + head) * 2) * L * n_max;
    float* dS = P + (size_t)L * n_max;
    for (int i = tid; i < L * DH; i += 128) {
        const int t = i / DH, c = i % DH;
        s_q[t][c] = qkv[(size_t)(b * L + t) * 3 * d + head * DH + c];
        s_do[t][c] = dattn[(size_t)(b * L + t) * d + head * DH + c];
    }
    __syncthreads();
    auto block_reduce = [&](float v, bool is_max) -> float {
        v = is_max ? warp_max(v) : warp_sum(v);
        __syncthreads();
        if ((tid & 31) == 0) s_red[tid >> 5] = v;
        __syncthreads();
        return is_max ? fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]))
                      : (s_red[0] + s_red[1]) + (s_red[2] + s_red[3]);
    };
    // thread per key: scores and dP
    for (int t = 0; t < L; t++) {
        const int n = len + t + 1;
        float m = -INFINITY;
        for (int j = tid; j < n; j += 128) {
            float s = 0.f, dp = 0.f;
            for (int c = 0; c < DH; c++) {
                s += s_q[t][c] * to_f32<KVT>(K[(size_t)j * DH + c]);
                dp += s_do[t][c] * to_f32<KVT>(V[(size_t)j * DH + c]);
            }
            s *= scale;
            P[(size_t)t * n_max + j] = s;
            dS[(size_t)t * n_max + j] = dp;
            m = fmaxf(m, s);
        }
        m = block_reduce(m, true);
        float l = 0.f;
        for (int j = tid; j < n; j += 128) l += expf(P[(size_t)t * n_max + j] - m);
        l = block_reduce(l, false);
        float dd = 0.f;
        for (int j = tid; j < n; j += 128) {
            const float p = expf(P[(size_t)t * n_max + j] - m) / l;
            P[(size_t)t * n_max + j] = p;
            dd += p * dS[(size_t)t * n_max + j];
        }
        dd = block_reduce(dd, false);
        for (int j = tid; j < n; j += 128)
            dS[(size_t)t * n_max + j] = P[(size_t)t * n_max + j] * (dS[(size_t)t * n_max + j] - dd);
        if (tid == 0) { s_stat[t][0] = m; s_stat[t][1] = 1.f / l; s_stat[t][2] = dd; }
    }
    __syncthreads();
    // thread per feature: dq of every row; dk, dv of the look-ahead keys
    for (int c = tid; c < DH; c += 128) {
        for (int t = 0; t < L; t++) {
            const int n = len + t + 1;
            float acc = 0.f;
            for (int j = 0; j < n; j++) acc += dS[(size_t)t * n_max + j] * to_f32<KVT>(K[(size_t)j * DH + c]);
            dqkv[(size_t)(b * L + t) * 3 * d + head * DH + c] = acc * scale;
        }
        for (int u = 0; u < L; u++) {                     // key of look-ahead row u, seen by rows t >= u
            const int j = len + u;
            float dk = 0.f, dv = 0.f;
            for (int t = u; t < L; t++) {
                dk += dS[(size_t)t * n_max + j] * s_q[t][c];
                dv += P[(size_t)t * n_max + j] * s_do[t][c];
            }
            dqkv[(size_t)(b * L + u) * 3 * d + d + head * DH + c] = dk * scale;
            dqkv[(size_t)(b * L + u) * 3 * d + 2 * d + head * DH + c] = dv;
        }
    }
}

// grad[t] = sum over the sequences of d loss / d (input row of look-ahead token t); then one AdamW update
// (decoupled weight decay) of the float32 master rows with the learning rate of this update.
__global__ void k_la_grad_adamw(const float* __restrict__ dh, int B, int L, int d, float* __restrict__ grad,
                                float* __restrict__ master, float* __restrict__ m, float* __restrict__ v,
                                float lr, float beta1, float beta2, float eps, float weight_decay,
                                float bias1, float bias2, int apply) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= L * d) return;
    const int t = i / d, c = i % d;
    float g = 0.f;
    for (int b = 0; b < B; b++) g += dh[(size_t)(b * L + t) * d + c];
    grad[i] = g;
    if (!apply) return;
    float p = master[i] * (1.f - lr * weight_decay);
    const float mm = beta1 * m[i] + (1.f - beta1) * g;
    const float vv = beta2 * v[i] + (1.f - beta2) * g * g;
    m[i] = mm;
    v[i] = vv;
    p -= lr * (mm / bias1) / (sqrtf(vv / bias2) + eps);
    master[i] = p;
}

template <typename WT>
__global__ void k_rows_convert(const WT* __restrict__ src, float* __restrict__ dst, size_t n, int to_float) {
    const size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (i >= n) return;
    if (to_float) dst[i] = to_f32<WT>(src[i]);
    else const_cast<WT*>(src)[i] = from_f32<WT>(dst[i]);
}

}  // namespace pass
