// Split-K ("flash-decoding") attention for the few causal query rows of one PaSS step over a long
// contiguous bf16 KV cache.  The paper's premise is that a decoding call re-reads "the past keys
// and values tensors" once whatever the number of rows: here one CTA streams one slice of one
// head's keys/values exactly once and serves all M <= 32 rows of the sequence from it.
//
//   grid  = (heads, sequences, n_split); 128 threads = 4 warps
//   K/V   : cp.async, 64-key blocks, a ring of two or three stages in shared memory, 16-byte chunks XOR-swizzled
//   math  : mma.sync m16n8k16 bf16 (S = Q K^T, O += P V), fp32 online softmax per warp
//   split : each slice leaves (O, max, sum) partials; the last slice to finish (counter per
//           sequence and head) merges them in slice order and writes the bf16 hi/lo rows that
//           feed the output projection.
// Row i of a sequence sits at position len + i and may attend to keys 0 .. len + i.
#pragma once
#include "pass_common.cuh"

namespace pass {

constexpr int kAttnBK = 64;        // keys per block
constexpr int kAttnStages = 3;
constexpr int kAttnMaxSplit = 16;

struct AttnParams {
    const float* q;                // [rows][ldq] rotated queries, float32
    int ldq;
    const int* row_seq;            // [rows]
    const int* row_pos;            // [rows]
    ModelDims md;
    int layer;
    const __nv_bfloat16* kc;
    const __nv_bfloat16* vc;
    int M;                         // rows per sequence (1 + 2k)
    int n_split;
    float* part_o;                 // [B][H][n_split][32][DH]
    float* part_ml;                // [B][H][n_split][32][2]
    int* counters;                 // [B*H], zero between launches
    __nv_bfloat16* out;            // [rows][d] hi parts, lo parts lo_row0 rows further down
    int lo_row0;                   // < 0: plain bf16 output rows, no lo parts
    int debug_stale;               // test hook: the early part pretends the tables said len - debug_stale
    int out_tile_rows;             // > 0: output rows are laid out in token tiles of this many rows, hi rows of a tile
                                   // followed by its lo rows (the layout the next GEMM of a prompt chunk reads)
    int* status;                   // kStatusTimeout is raised here (k_attn_tc, the only attention kernel that waits)
    unsigned long long* trace;     // k_attn_tc, PASS_TRACE: [head / 4][16 slices][8] %globaltimer stamps of every fourth head's CTAs
    int debug_stuck;               // test hook (k_attn_tc): the scores are never announced, so the bounded waits run out
    int rows_per_block;            // 0: blockIdx.y = sequence, M rows each (a decode step).  > 0: ONE sequence of M rows
                                   // (a prompt chunk), blockIdx.y = block of rows_per_block rows - causal flash attention
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// Merge of the slices of one (sequence, head) by the CTA that delivered last.  NS = most slices this
// instance handles, EB = output elements per thread and batch, NT = threads of the CTA.  The first batch of partial outputs and
// the (max, sum) pairs are requested together, before anything waits: for the usual case (up to 4 slices,
// up to 12 rows of 128) the whole merge is one trip to L2.
template <int DH, int NS, int EB, int NT = 128>
__device__ __forceinline__ void attn_merge(const AttnParams& p, size_t hb, int row0, int head, float* sm_f) {
    const int tid = threadIdx.x, M = p.M;
    auto load_batch = [&](int base, float (&vals)[EB][NS]) {
#pragma unroll
        for (int e = 0; e < EB; e++) {
            const int idx = min(base + e * NT + tid, M * DH - 1);
            const int i = idx / DH, dcol = idx % DH;
#pragma unroll
            for (int sidx = 0; sidx < NS; sidx++)
                vals[e][sidx] = sidx < p.n_split ? __ldcg(p.part_o + (hb + sidx * 32 + i) * DH + dcol) : 0.f;
        }
    };
    float vals[EB][NS];
    load_batch(0, vals);
    for (int i = tid; i < M; i += NT) {
        float2 ml[NS];
#pragma unroll
        for (int sidx = 0; sidx < NS; sidx++)
            ml[sidx] = sidx < p.n_split ? __ldcg(reinterpret_cast<const float2*>(p.part_ml) + hb + sidx * 32 + i)
                                        : make_float2(-INFINITY, 0.f);
        float mm = -INFINITY;
#pragma unroll
        for (int sidx = 0; sidx < NS; sidx++) mm = fmaxf(mm, ml[sidx].x);
        float ll = 0.f, f[NS];
#pragma unroll
        for (int sidx = 0; sidx < NS; sidx++) {
            f[sidx] = ml[sidx].x == -INFINITY ? 0.f : exp2f(ml[sidx].x - mm);
            ll += ml[sidx].y * f[sidx];
        }
        const float inv = 1.f / ll;
#pragma unroll
        for (int sidx = 0; sidx < NS; sidx++)
            if (sidx < p.n_split) sm_f[sidx * 32 + i] = f[sidx] * inv;
    }
    __syncthreads();
    for (int base = 0; base < M * DH; base += NT * EB) {
        if (base > 0) load_batch(base, vals);
#pragma unroll
        for (int e = 0; e < EB; e++) {
            const int idx = base + e * NT + tid;
            if (idx < M * DH) {
                const int i = idx / DH, dcol = idx % DH;
                float v = 0.f;
#pragma unroll
                for (int sidx = 0; sidx < NS; sidx++)
                    if (sidx < p.n_split) v += vals[e][sidx] * sm_f[sidx * 32 + i];
                const __nv_bfloat16 hi = __float2bfloat16_rn(v);
                p.out[(size_t)(row0 + i) * p.md.d + head * DH + dcol] = hi;
                p.out[(size_t)(p.lo_row0 + row0 + i) * p.md.d + head * DH + dcol] = __float2bfloat16_rn(v - __bfloat162float(hi));
            }
        }
    }
}

// CL: the slices of one (sequence, head) form a thread-block cluster (n_split CTAs along z) and are
// merged through distributed shared memory: every CTA leaves its slice's unnormalised output and its
// (max, sum) pairs in its own shared memory, the cluster synchronises once, and each CTA then merges a
// share of the output rows reading all slices with ld.shared::cluster.  Compared with the merge through
// global memory this saves the partial stores, the fence, the arrival counter and a trip to L2.
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_dsmem_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t ra;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
    return v;
}

// Registers (NREG): the CTA of a step of up to nine rows shares its SM with the step's GEMM CTA, which takes 136
// registers x 256 threads, so 232 x 128 are left for it - and it is measurably faster with them than with 168
// (2.796 -> 2.778 ms per step at 512 cached positions, 3.077 -> 3.005 ms at 2048).  Where three of these CTAs
// share an SM (steps of ten rows or more): 168.
// MT = m-tiles of 16 rows per CTA (4 warps: MT = 4 gives every warp its own 16 rows and all keys of a block,
// the usual flash-attention split for many rows).  HL = queries and probabilities as bf16 hi + lo pairs;
// without it they are single bf16 values (prompt chunks in plain bf16, half the MMAs).
// CHUNK = the rows are one sequence's prompt chunk (rows_per_block, out_tile_rows, optional lo parts); the
// decode step's instances have it off and carry none of that code.  ST = depth of the key / value ring: 2 (64 KB at
// d_head 128) in the decode step - beside the GEMM CTA a third stage buys nothing, a seventh stage of the GEMM's
// ring does (2.778 -> 2.748 ms), and three CTAs of two stages fit an SM where they have it to themselves -, 3
// for prompt chunks and the doubled slices of long caches.
template <int DH, int MT, bool CL, bool HL = true, bool CHUNK = false, int ST = kAttnStages, int NREG = 232>
__global__ void __maxnreg__(NREG)
k_attn_fd(const AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem_attn[];
    constexpr int CH = DH / 8;                       // 16-byte chunks per key
    constexpr int TILE_BYTES = kAttnBK * DH * 2;     // one K (or V) block
    constexpr int KPW = 16 * MT;                     // keys per warp and block
    __shared__ int s_last;

    // Programmatic dependent launch: let the next kernel (the output projection) become resident and
    // start streaming its weights now.  This kernel itself is resident long before its queries exist, and
    // uses the time: blocks that hold nothing but cache rows of earlier steps (positions < len, which no
    // kernel of this step writes) are fetched before the wait.  The row tables they are addressed through
    // are read again after the wait; should they differ (this part ran before the tables of this step were
    // written), everything is fetched again.  Rows of this step are written by the kernel being waited
    // for and are touched only after the wait.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int head = blockIdx.x, b = blockIdx.y, split = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int mt = warp % MT, part = warp / MT;
    // a decode step: rows b*M .. of sequence b; a prompt chunk: rows b*rows_per_block .. of the one sequence
    const int row0 = CHUNK ? b * p.rows_per_block : b * p.M;
    const int M = CHUNK ? min(p.rows_per_block, p.M - row0) : p.M;
    // one thread reads the tables for all, so that the whole CTA works from the same pair even if it
    // reads while they are being written
    __shared__ int s_tab[2];
    if (tid == 0) {
        s_tab[0] = *(volatile const int*)(p.row_seq + row0);
        s_tab[1] = *(volatile const int*)(p.row_pos + row0);
    }
    __syncthreads();
    int seq, len, k_begin, k_end, nb;
    const __nv_bfloat16 *kbase, *vbase;
    auto slice = [&](int seq_, int len_) {
        seq = seq_;
        len = len_;
        const int n_tot = len + M;
        // keys are dealt out in granules of 16 (one warp's share of a block), so that no slice is left
        // empty while another holds a whole block more
        int chunk = (n_tot + p.n_split - 1) / p.n_split;
        chunk = ((chunk + 15) / 16) * 16;
        k_begin = split * chunk;
        k_end = min(n_tot, k_begin + chunk);
        nb = k_end > k_begin ? (k_end - k_begin + kAttnBK - 1) / kAttnBK : 0;
        kbase = p.kc + kv_index(p.md, p.layer, seq, head, 0);
        vbase = p.vc + kv_index(p.md, p.layer, seq, head, 0);
    };
    slice(s_tab[0], max(0, s_tab[1] - p.debug_stale));
    // rows of this launch's own chunk ahead of this block are cache rows the awaited kernel writes: in chunk
    // mode only positions before the chunk's first row may be fetched early
    const int early_len = CHUNK ? min(len, *(volatile const int*)(p.row_pos)) : len;
    const uint32_t sK = smem_u32(smem_attn), sV = sK + ST * TILE_BYTES;

    auto load_block = [&](int blk) {
        const int st = blk % ST;
        const int kb = k_begin + blk * kAttnBK;
        for (int idx = tid; idx < kAttnBK * CH; idx += 128) {
            const int key = idx / CH, c = idx % CH;
            const int gk = kb + key;
            const bool ok = gk < k_end;
            const size_t off = (size_t)(ok ? gk : 0) * DH + c * 8;
            const uint32_t d = (uint32_t)((key * CH + (c ^ (key & 7))) * 16);
            cp_async16(sK + st * TILE_BYTES + d, kbase + off, ok ? 16 : 0);
            cp_async16(sV + st * TILE_BYTES + d, vbase + off, ok ? 16 : 0);
        }
    };

    // first ring fill: blocks of old rows now, the rest (and the queries) after the wait
    uint32_t early = 0;
#pragma unroll
    for (int st = 0; st < ST; st++) {
        if (st < nb && min(k_end, k_begin + (st + 1) * kAttnBK) <= early_len) { load_block(st); early |= 1u << st; }
    }
    cp_async_commit();
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // Three trips to L2 start here and overlap: the row tables (final now), the queries, and - once the tables are
    // in - the blocks that were not fetched early.  The queries are asked for before anything waits for the tables.
    const int seq_f = __ldcg(p.row_seq + row0), len_f = __ldcg(p.row_pos + row0);    // the same for every thread
    float2 qraw[DH / 16][4];
    {
        const int i0 = mt * 16 + g, i1 = i0 + 8;
        const float* q0 = p.q + (size_t)(row0 + i0) * p.ldq + head * DH;
        const float* q1 = p.q + (size_t)(row0 + i1) * p.ldq + head * DH;
#pragma unroll
        for (int ks = 0; ks < DH / 16; ks++) {
            const int c = ks * 16 + 2 * t;
            const float2 z = make_float2(0.f, 0.f);
            qraw[ks][0] = i0 < M ? *reinterpret_cast<const float2*>(q0 + c) : z;
            qraw[ks][1] = i1 < M ? *reinterpret_cast<const float2*>(q1 + c) : z;
            qraw[ks][2] = i0 < M ? *reinterpret_cast<const float2*>(q0 + c + 8) : z;
            qraw[ks][3] = i1 < M ? *reinterpret_cast<const float2*>(q1 + c + 8) : z;
        }
    }
    {
        if (seq_f != seq || len_f != len) {
            // the early part worked from tables of an earlier step: let its copies land, then start over
            cp_async_wait<0>();
            __syncthreads();
            slice(seq_f, len_f);
            early = 0;
        }
    }
#pragma unroll
    for (int st = 0; st < ST; st++) {
        if (st < nb && !((early >> st) & 1u)) load_block(st);
        cp_async_commit();
    }

    // query fragments (A operand), scaled by log2(e)/sqrt(d_head) so that exp2 can be used.  Queries and
    // probabilities are carried as bf16 hi + bf16 lo (two MMAs each): a single bf16 rounding of q or p
    // (2^-9 relative) would go straight into the output, since the output is a sum of the same terms.
    uint32_t qf[DH / 16][4], qfl[DH / 16][4];
    {
        const float sc = 1.4426950408889634f * rsqrtf((float)DH);
#pragma unroll
        for (int ks = 0; ks < DH / 16; ks++) {
#pragma unroll
            for (int e = 0; e < 4; e++) {
                const float x = qraw[ks][e].x * sc, y = qraw[ks][e].y * sc;
                const __nv_bfloat162 hi = __floats2bfloat162_rn(x, y);
                qf[ks][e] = *reinterpret_cast<const uint32_t*>(&hi);
                qfl[ks][e] = pack_bf16(x - __low2float(hi), y - __high2float(hi));
            }
        }
    }

    float o[DH / 8][4];
#pragma unroll
    for (int n = 0; n < DH / 8; n++) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

    for (int blk = 0; blk < nb; blk++) {
        if (blk > 0) {
            // everybody is done with block blk-1: its stage takes block blk-1+stages
            __syncthreads();
            if (blk - 1 + ST < nb) load_block(blk - 1 + ST);
            cp_async_commit();
        }
        cp_async_wait<ST - 1>();
        __syncthreads();
        const int st = blk % ST;
        const uint32_t kS = sK + st * TILE_BYTES, vS = sV + st * TILE_BYTES;
#pragma unroll
        for (int sub = 0; sub < MT; sub++) {
            const int key0 = part * KPW + sub * 16;          // within the block
            const int gkey0 = k_begin + blk * kAttnBK + key0;
            if (gkey0 >= k_end) continue;
            float s[2][4], sl[2][4];      // hi and lo query parts accumulate apart: four chains of 8 MMAs, not two of 16
#pragma unroll
            for (int n = 0; n < 2; n++) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f; sl[n][0] = sl[n][1] = sl[n][2] = sl[n][3] = 0.f; }
            {
                const int mi = lane >> 3, rr = lane & 7;
                const int key = key0 + (mi >> 1) * 8 + rr;
#pragma unroll
                for (int ks = 0; ks < DH / 16; ks++) {
                    const int c = 2 * ks + (mi & 1);
                    uint32_t r[4];
                    ldsm_x4(kS + (uint32_t)((key * CH + (c ^ (key & 7))) * 16), r);
                    mma_bf16_16816(s[0], qf[ks], r[0], r[1]);
                    mma_bf16_16816(s[1], qf[ks], r[2], r[3]);
                    if (HL) {
                        mma_bf16_16816(sl[0], qfl[ks], r[0], r[1]);
                        mma_bf16_16816(sl[1], qfl[ks], r[2], r[3]);
                    }
                }
#pragma unroll
                for (int n = 0; n < 2; n++)
#pragma unroll
                    for (int e = 0; e < 4; e++) s[n][e] += sl[n][e];
            }
            // causal mask: row i sees key j iff j <= len + i
            const int i0 = mt * 16 + g, i1 = i0 + 8;
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int n = 0; n < 2; n++)
#pragma unroll
                for (int e = 0; e < 2; e++) {
                    const int j = gkey0 + n * 8 + 2 * t + e;
                    if (j > len + i0 || j >= k_end) s[n][e] = -INFINITY;
                    if (j > len + i1 || j >= k_end) s[n][2 + e] = -INFINITY;
                    mx0 = fmaxf(mx0, s[n][e]);
                    mx1 = fmaxf(mx1, s[n][2 + e]);
                }
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
            const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
            const float c0 = mn0 == -INFINITY ? 1.f : exp2f(m_run[0] - mn0);
            const float c1 = mn1 == -INFINITY ? 1.f : exp2f(m_run[1] - mn1);
            const float b0 = mn0 == -INFINITY ? 0.f : mn0, b1 = mn1 == -INFINITY ? 0.f : mn1;
            m_run[0] = mn0;
            m_run[1] = mn1;
            float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
            for (int n = 0; n < 2; n++)
#pragma unroll
                for (int e = 0; e < 2; e++) {
                    s[n][e] = exp2f(s[n][e] - b0);
                    s[n][2 + e] = exp2f(s[n][2 + e] - b1);
                    ps0 += s[n][e];
                    ps1 += s[n][2 + e];
                }
            l_run[0] = l_run[0] * c0 + ps0;
            l_run[1] = l_run[1] * c1 + ps1;
#pragma unroll
            for (int n = 0; n < DH / 8; n++) { o[n][0] *= c0; o[n][1] *= c0; o[n][2] *= c1; o[n][3] *= c1; }
            uint32_t pa[4], pl[4];
            {
                const float ps[4][2] = {{s[0][0], s[0][1]}, {s[0][2], s[0][3]}, {s[1][0], s[1][1]}, {s[1][2], s[1][3]}};
#pragma unroll
                for (int e = 0; e < 4; e++) {
                    const __nv_bfloat162 hi = __floats2bfloat162_rn(ps[e][0], ps[e][1]);
                    pa[e] = *reinterpret_cast<const uint32_t*>(&hi);
                    pl[e] = pack_bf16(ps[e][0] - __low2float(hi), ps[e][1] - __high2float(hi));
                }
            }
            {
                const int mi = lane >> 3, rr = lane & 7;
                const int key = key0 + (mi & 1) * 8 + rr;
#pragma unroll
                for (int np = 0; np < DH / 16; np++) {
                    const int c = 2 * np + (mi >> 1);
                    uint32_t r[4];
                    ldsm_x4_trans(vS + (uint32_t)((key * CH + (c ^ (key & 7))) * 16), r);
                    mma_bf16_16816(o[2 * np], pa, r[0], r[1]);
                    mma_bf16_16816(o[2 * np + 1], pa, r[2], r[3]);
                    if (HL) {
                        mma_bf16_16816(o[2 * np], pl, r[0], r[1]);
                        mma_bf16_16816(o[2 * np + 1], pl, r[2], r[3]);
                    }
                }
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();

    // merge the warps that share an m-tile; shared memory is reused as [4][16][DH] + stats
    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1);
    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
    float* sm_o = reinterpret_cast<float*>(smem_attn);
    float* sm_m = sm_o + 4 * 16 * DH;
    float* sm_l = sm_m + 64;
    // staging rows are swizzled in blocks of 8 floats by (row & 3) so that the eight rows a warp writes
    // at once fall into different banks; rows beyond M are not written (nobody reads them)
    {
        const bool live0 = mt * 16 + g < M, live1 = mt * 16 + g + 8 < M;
        const int sw = (g & 3) * 8;
#pragma unroll
        for (int n = 0; n < DH / 8; n++) {
            const int col = (n * 8 + 2 * t) ^ sw;
            if (live0) *reinterpret_cast<float2*>(sm_o + ((warp * 16 + g) * DH + col)) = make_float2(o[n][0], o[n][1]);
            if (live1) *reinterpret_cast<float2*>(sm_o + ((warp * 16 + g + 8) * DH + col)) = make_float2(o[n][2], o[n][3]);
        }
    }
    if (t == 0) {
        sm_m[warp * 16 + g] = m_run[0]; sm_m[warp * 16 + g + 8] = m_run[1];
        sm_l[warp * 16 + g] = l_run[0]; sm_l[warp * 16 + g + 8] = l_run[1];
    }
    __syncthreads();
    constexpr int NP = 4 / MT;                       // warps per m-tile
    const size_t pbase = ((size_t)(b * p.md.H + head) * p.n_split + split) * 32;
    for (int idx = tid; idx < M * DH; idx += 128) {  // live rows only
        const int i = idx / DH, dcol = idx % DH;     // i = row within the sequence
        const int tile = i / 16, rr = i % 16;
        float mm = -INFINITY;
#pragma unroll
        for (int q = 0; q < NP; q++) mm = fmaxf(mm, sm_m[(q * MT + tile) * 16 + rr]);
        float acc = 0.f, ll = 0.f;
#pragma unroll
        for (int q = 0; q < NP; q++) {
            const int w = q * MT + tile;
            const float mw = sm_m[w * 16 + rr];
            const float f = mw == -INFINITY ? 0.f : exp2f(mw - mm);
            acc += sm_o[(w * 16 + rr) * DH + (dcol ^ ((rr & 3) * 8))] * f;
            ll += sm_l[w * 16 + rr] * f;
        }
        if (p.n_split == 1) {
            const float v = acc / ll;
            const __nv_bfloat16 hi = __float2bfloat16_rn(v);
            const int g_row = row0 + i;
            const int o_row = (CHUNK && p.out_tile_rows) ? (g_row / p.out_tile_rows) * 2 * p.out_tile_rows + g_row % p.out_tile_rows : g_row;
            p.out[(size_t)o_row * p.md.d + head * DH + dcol] = hi;
            if (!CHUNK || p.lo_row0 >= 0) p.out[(size_t)(p.lo_row0 + o_row) * p.md.d + head * DH + dcol] = __float2bfloat16_rn(v - __bfloat162float(hi));
        } else if (CL) {
            float* cl_o = sm_o + 4 * 16 * DH + 128;          // [32][DH], behind the warp staging area
            float* cl_ml = cl_o + 32 * DH;                   // [32][2]
            cl_o[i * DH + dcol] = acc;
            if (dcol == 0) { cl_ml[i * 2] = mm; cl_ml[i * 2 + 1] = ll; }
        } else {
            p.part_o[(pbase + i) * DH + dcol] = acc;
            if (dcol == 0) { p.part_ml[(pbase + i) * 2] = mm; p.part_ml[(pbase + i) * 2 + 1] = ll; }
        }
    }
    if (p.n_split == 1) return;
    if (CL) {
        constexpr int NSMAX = 8;
        const uint32_t cl_o_addr = smem_u32(sm_o + 4 * 16 * DH + 128), cl_ml_addr = cl_o_addr + 32 * DH * 4;
        const int ns = p.n_split;
        const uint32_t rank = cluster_ctarank();
        cluster_sync_all();                                  // every slice's partials are in place
        for (int idx = (int)rank * 128 + tid; idx < M * DH; idx += ns * 128) {
            const int i = idx / DH;
            float ms[NSMAX], ls[NSMAX], os[NSMAX];
#pragma unroll
            for (int sidx = 0; sidx < NSMAX; sidx++) {
                if (sidx < ns) {
                    ms[sidx] = ld_dsmem_f32(cl_ml_addr + (uint32_t)(i * 2) * 4, sidx);
                    ls[sidx] = ld_dsmem_f32(cl_ml_addr + (uint32_t)(i * 2 + 1) * 4, sidx);
                    os[sidx] = ld_dsmem_f32(cl_o_addr + (uint32_t)idx * 4, sidx);
                } else { ms[sidx] = -INFINITY; ls[sidx] = 0.f; os[sidx] = 0.f; }
            }
            float mm = -INFINITY;
#pragma unroll
            for (int sidx = 0; sidx < NSMAX; sidx++) mm = fmaxf(mm, ms[sidx]);
            float ll = 0.f, v = 0.f;
#pragma unroll
            for (int sidx = 0; sidx < NSMAX; sidx++) {
                const float f = ms[sidx] == -INFINITY ? 0.f : exp2f(ms[sidx] - mm);
                ll += ls[sidx] * f;
                v += os[sidx] * f;
            }
            v /= ll;
            const int dcol = idx % DH;
            const __nv_bfloat16 hi = __float2bfloat16_rn(v);
            p.out[(size_t)(row0 + i) * p.md.d + head * DH + dcol] = hi;
            p.out[(size_t)(p.lo_row0 + row0 + i) * p.md.d + head * DH + dcol] = __float2bfloat16_rn(v - __bfloat162float(hi));
        }
        cluster_sync_all();                                  // nobody leaves while its memory is still being read
        return;
    }

    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int prev = atomicAdd(p.counters + b * p.md.H + head, 1);
        s_last = prev == p.n_split - 1;
        if (s_last) p.counters[b * p.md.H + head] = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // The last slice merges all slices.
    const size_t hb = (size_t)(b * p.md.H + head) * p.n_split * 32;
    float* sm_f = reinterpret_cast<float*>(smem_attn);             // [n_split][32] weight of slice s for row i
    if (p.n_split <= 4) attn_merge<DH, 4, 12>(p, hb, row0, head, sm_f);
    else attn_merge<DH, kAttnMaxSplit, 4>(p, hb, row0, head, sm_f);
}

}  // namespace pass
