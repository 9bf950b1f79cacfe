// Decode-step attention for LONG caches with the score product on the 5th-generation tensor cores.
//
// The split-K kernel of attn_fd.cuh computes S = Q K^T and O += P V with mma.sync.  From a few thousand
// cached positions on, its key loop is bound by the instructions each warp has to get through per key
// (copy requests, two products in hi + lo pairs, a softmax update every 16 keys), not by reading the cache:
// 45 % of the memory bandwidth at 8192 positions.  Here the score product moves to tcgen05.mma:
//
//   S^T [128 keys x 32] = K_block [128 keys x 128] (operand A, K-major, straight from the cache by TMA)
//                         x (Q_hi | Q_lo)^T [32 x 128] (operand B, written once to shared memory)
//
// accumulated in TMEM, two buffers, so the product of block j+1 runs while block j is in the softmax.  A
// softmax thread owns one key of the block (one TMEM lane) and all 16 rows; it adds the hi and lo columns,
// masks, and keeps an online softmax per row together with the 31 other keys of its warp (one redux.sync per
// row for the maximum; the sums stay per thread until the end).  O += P V stays on mma.sync - the cache holds
// V as [key][d_head], the wrong way round for a K-major tcgen05 operand - with each warp multiplying the
// probabilities of its own 32 keys (turned into A fragments through a private strip of shared memory) by its
// 32 value rows.  Copies are TMA requests of one thread.  Two groups of four softmax warps take the blocks
// alternately, each with its own TMEM buffer; warps, then key slices, are merged as in attn_fd.cuh.
//
//   grid = (heads, sequences, n_split), 320 threads: warp 0 TMA, warp 1 TMEM + MMA issue, warps 2-9 softmax + PV
//   K / V blocks of 128 keys (32 KB each), two stages of each; d_head = 128, at most 16 rows per sequence.
// Every wait is bounded (mbar_wait); when one runs out the CTA raises kStatusTimeout, lets its copies land,
// frees its TMEM and returns without output.
#pragma once
#include "attn_fd.cuh"
#include "gemm_tc.cuh"

namespace pass {

constexpr int kTcBK = 128;                 // keys per block
constexpr int kTcDH = 128;
constexpr int kTcThreads = 320;
constexpr int kTcTile = kTcBK * kTcDH * 2;             // one K (or V) block: 32 KB = two boxes of [128 keys][64], 128B swizzle
constexpr int kTcQBytes = 32 * kTcDH * 2;              // (Q_hi | Q_lo): 32 rows = two slabs of [32][64]
constexpr int kTcPStride = 80;                         // bytes per row of a probability strip (32 keys + 16 bytes: no bank conflicts)
constexpr int kTcPStrip = 2 * 16 * kTcPStride;         // one warp: hi rows, then lo rows
constexpr int kTcSmem = 1024 + 4 * kTcTile + kTcQBytes + 8 * kTcPStrip;

struct AttnTcMaps { CUtensorMap k, v; };   // each cache as a matrix [all (layer, sequence, head, position)][128], box 64 x 128

// byte offset of 16-byte chunk c (0..15) of key row `key` in a block
__device__ __forceinline__ uint32_t tc_tile_off(int key, int c) {
    return (uint32_t)((c >> 3) * (kTcBK * 128) + key * 128 + (((c & 7) ^ (key & 7)) << 4));
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 32; i++) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float warp_max_f32(float v) {       // one instruction on sm_100a
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ void st_shared_b16(uint32_t addr, __nv_bfloat16 v) {
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(*reinterpret_cast<const unsigned short*>(&v)) : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Stamps of every fourth head's CTAs only: reads of %globaltimer from all CTAs at once queue up behind one another.
// Slots: 0 entry, 1 dependency wait over, 2 first key block in shared memory, 3 last score product issued,
// 4 last softmax / P V done, 5 slice's partial output in memory, 6 slices of the head merged.
#define PASS_ATTN_TRACE(slot) do { if (p.trace && (blockIdx.x & 3) == 0) p.trace[((blockIdx.x >> 2) * 16 + blockIdx.z) * 8 + (slot)] = global_ns(); } while (0)

__global__ void __launch_bounds__(kTcThreads, 1)
k_attn_tc(const __grid_constant__ AttnTcMaps maps, const AttnParams p) {
    // aligned to 1024 bytes by hand below: asking for it here would pad the static shared memory of EVERY kernel
    // of the translation unit to that alignment, and the step's GEMM and attention CTAs would no longer share an SM
    extern __shared__ __align__(128) uint8_t smem_tc[];
    __shared__ __align__(8) uint64_t s_bar[12];      // full_k[2], full_v[2], empty_k[2], empty_v[2], s_full[2], s_empty[2]
    __shared__ uint32_t s_tmem;
    __shared__ int s_abort, s_last, s_issued;
    __shared__ float sm_m[8 * 16], sm_l[8 * 16];
    const int head = blockIdx.x, b = blockIdx.y, split = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int M = p.M, row0 = b * M;
    if (tid == 0) PASS_ATTN_TRACE(0);
    const uint32_t base = (smem_u32(smem_tc) + 1023u) & ~1023u;
    const uint32_t sK = base, sV = sK + 2 * kTcTile, sQ = sV + 2 * kTcTile, sP = sQ + kTcQBytes;
    const uint32_t bar = smem_u32(&s_bar[0]);
    const uint32_t b_fk = bar, b_fv = bar + 16, b_ek = bar + 32, b_ev = bar + 48, b_sf = bar + 64, b_se = bar + 80;
    if (tid == 0) {
        for (int s = 0; s < 2; s++) {
            mbar_init(b_fk + 8 * s, 1); mbar_init(b_fv + 8 * s, 1);
            mbar_init(b_ek + 8 * s, 1); mbar_init(b_ev + 8 * s, 4);
            mbar_init(b_sf + 8 * s, 1); mbar_init(b_se + 8 * s, 4);
        }
        s_abort = 0;
        s_issued = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&s_tmem), 64);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    griddep_launch_dependents();
    griddep_wait();                                   // the queries and this step's cache rows come from the kernel before
    if (tid == 0) PASS_ATTN_TRACE(1);

    // this CTA's slice of the keys, in whole blocks
    const int seq = __ldcg(p.row_seq + row0), len = __ldcg(p.row_pos + row0);
    const int n_tot = len + M;
    int chunk = (n_tot + p.n_split - 1) / p.n_split;
    chunk = ((chunk + kTcBK - 1) / kTcBK) * kTcBK;
    const int k_begin = split * chunk, k_end = min(n_tot, k_begin + chunk);
    const int nb = k_end > k_begin ? (k_end - k_begin + kTcBK - 1) / kTcBK : 0;
    const int map_row0 = (int)(kv_index(p.md, p.layer, seq, head, 0) / kTcDH) + k_begin;   // first key of the slice in the cache maps

    float o[kTcDH / 8][4];
    float m_run[16], l_part[16];
#pragma unroll
    for (int n = 0; n < kTcDH / 8; n++) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
#pragma unroll
    for (int i = 0; i < 16; i++) { m_run[i] = -INFINITY; l_part[i] = 0.f; }

    if (warp == 0) {
        // ---------------------------------------------------------------- copies
        if (lane == 0) {
            const uint64_t pol = policy_evict_first();
            for (int j = 0; j < nb; j++) {
                const int s = j & 1;
                const uint32_t par = ((j >> 1) & 1) ^ 1;
                if (!mbar_wait(b_ek + 8 * s, par, &s_abort, p.status)) break;
                mbar_expect_tx(b_fk + 8 * s, kTcTile);
                tma_load_2d(sK + s * kTcTile, &maps.k, b_fk + 8 * s, 0, map_row0 + j * kTcBK, pol);
                tma_load_2d(sK + s * kTcTile + kTcTile / 2, &maps.k, b_fk + 8 * s, 64, map_row0 + j * kTcBK, pol);
                if (!mbar_wait(b_ev + 8 * s, par, &s_abort, p.status)) { *(volatile int*)&s_issued = 2 * j + 1; break; }
                mbar_expect_tx(b_fv + 8 * s, kTcTile);
                tma_load_2d(sV + s * kTcTile, &maps.v, b_fv + 8 * s, 0, map_row0 + j * kTcBK, pol);
                tma_load_2d(sV + s * kTcTile + kTcTile / 2, &maps.v, b_fv + 8 * s, 64, map_row0 + j * kTcBK, pol);
                *(volatile int*)&s_issued = 2 * j + 2;
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- S^T = K Q^T
        asm volatile("bar.sync 1, 288;" ::: "memory");                  // the queries are in shared memory
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(32);
            for (int j = 0; j < nb; j++) {
                const int s = j & 1;
                const uint32_t par = (j >> 1) & 1;
                if (!mbar_wait(b_fk + 8 * s, par, &s_abort, p.status)) break;
                if (!mbar_wait(b_se + 8 * s, par ^ 1, &s_abort, p.status)) break;
                if (j == 0) PASS_ATTN_TRACE(2);
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < kTcDH / 16; kk++) {
                    const uint64_t a_desc = smem_desc_sw128(sK + s * kTcTile + (kk >> 2) * (kTcTile / 2)) + 2 * (kk & 3);
                    const uint64_t b_desc = smem_desc_sw128(sQ + (kk >> 2) * (kTcQBytes / 2)) + 2 * (kk & 3);
                    umma_bf16(tmem + s * 32, a_desc, b_desc, idesc, kk > 0 ? 1u : 0u);
                }
                umma_commit(b_ek + 8 * s);       // the key block may be overwritten
                if (!p.debug_stuck) umma_commit(b_sf + 8 * s);       // the scores are complete
            }
            PASS_ATTN_TRACE(3);
        }
    } else {
        // ---------------------------------------------------------------- softmax and O += P V
        const int sw = warp - 2, wg = sw >> 2, quad = warp & 3;      // a warp reaches TMEM lanes 32 * (warp % 4) ..
        const int g = lane >> 2;
        {
            // queries, scaled by log2(e) / sqrt(d_head) so that exp2 can be used, as bf16 hi + lo rows of operand B
            const int st = sw * 32 + lane, r = st >> 4, c = st & 15;
            const float sc = 1.4426950408889634f * rsqrtf((float)kTcDH);
            float x[8];
            if (r < M) {
                const float4 a = *reinterpret_cast<const float4*>(p.q + (size_t)(row0 + r) * p.ldq + head * kTcDH + c * 8);
                const float4 bq = *reinterpret_cast<const float4*>(p.q + (size_t)(row0 + r) * p.ldq + head * kTcDH + c * 8 + 4);
                x[0] = a.x * sc; x[1] = a.y * sc; x[2] = a.z * sc; x[3] = a.w * sc;
                x[4] = bq.x * sc; x[5] = bq.y * sc; x[6] = bq.z * sc; x[7] = bq.w * sc;
            } else {
#pragma unroll
                for (int e = 0; e < 8; e++) x[e] = 0.f;
            }
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int e = 0; e < 4; e++) {
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(x[2 * e], x[2 * e + 1]);
                hi[e] = *reinterpret_cast<const uint32_t*>(&h2);
                lo[e] = pack_bf16(x[2 * e] - __low2float(h2), x[2 * e + 1] - __high2float(h2));
            }
            const uint32_t off = (uint32_t)((c >> 3) * (kTcQBytes / 2) + r * 128 + (((c & 7) ^ (r & 7)) << 4));
            st_shared_v4(sQ + off, hi[0], hi[1], hi[2], hi[3]);
            st_shared_v4(sQ + off + 16 * 128, lo[0], lo[1], lo[2], lo[3]);
            fence_proxy_async();
            asm volatile("bar.sync 1, 288;" ::: "memory");
        }
        const uint32_t strip = sP + sw * kTcPStrip;
        const int mi = lane >> 3, rr = lane & 7;
        for (int j = wg; j < nb; j += 2) {
            const int s = j & 1;
            const uint32_t par = (j >> 1) & 1;
            if (!mbar_wait(b_sf + 8 * s, par, &s_abort, p.status)) break;
            tc_fence_after();
            float v[32];
            tmem_ld32(tmem + ((uint32_t)(quad * 32) << 16) + s * 32, v);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(b_se + 8 * s);               // the next block but one may be multiplied into this buffer
            float sc_[16];
#pragma unroll
            for (int i = 0; i < 16; i++) sc_[i] = v[i] + v[16 + i];
            const int key0 = k_begin + j * kTcBK + quad * 32;          // this warp's first key
            if (key0 + 31 > len || key0 + 32 > k_end) {
                // causal mask: row i sees key jg iff jg <= len + i; keys from k_end on belong to nobody
                const int jg = key0 + lane;
#pragma unroll
                for (int i = 0; i < 16; i++)
                    if (jg > len + i || jg >= k_end) sc_[i] = -INFINITY;
            }
            bool changed = false;
            float mn[16];
#pragma unroll
            for (int i = 0; i < 16; i++) {
                mn[i] = fmaxf(m_run[i], warp_max_f32(sc_[i]));
                changed |= mn[i] != m_run[i];
            }
            if (changed) {                                           // the same for every lane: the maxima are warp-wide
                float c0 = 1.f, c1 = 1.f;
#pragma unroll
                for (int i = 0; i < 16; i++) {
                    const float corr = mn[i] == -INFINITY ? 1.f : exp2f(m_run[i] - mn[i]);
                    l_part[i] *= corr;
                    m_run[i] = mn[i];
                    if (i < 8) { if (g == i) c0 = corr; } else { if (g == i - 8) c1 = corr; }
                }
#pragma unroll
                for (int n = 0; n < kTcDH / 8; n++) { o[n][0] *= c0; o[n][1] *= c0; o[n][2] *= c1; o[n][3] *= c1; }
            }
#pragma unroll
            for (int i = 0; i < 16; i++) {
                const float pr = exp2f(sc_[i] - (mn[i] == -INFINITY ? 0.f : mn[i]));
                l_part[i] += pr;
                const __nv_bfloat16 ph = __float2bfloat16_rn(pr);
                st_shared_b16(strip + i * kTcPStride + lane * 2, ph);
                st_shared_b16(strip + 16 * kTcPStride + i * kTcPStride + lane * 2, __float2bfloat16_rn(pr - __bfloat162float(ph)));
            }
            if (!mbar_wait(b_fv + 8 * s, par, &s_abort, p.status)) break;
            const uint32_t vS = sV + s * kTcTile;
            if (key0 + 32 > k_end && key0 + lane >= k_end) {
                // value rows past the slice hold whatever the cache holds there; 0 x that must stay 0
#pragma unroll
                for (int c = 0; c < 16; c++) st_shared_v4(vS + tc_tile_off(quad * 32 + lane, c), 0u, 0u, 0u, 0u);
            }
            __syncwarp();
#pragma unroll
            for (int ks = 0; ks < 2; ks++) {
                uint32_t pa[4], pl[4];
                const uint32_t a_off = (uint32_t)(((mi & 1) * 8 + rr) * kTcPStride + (ks * 2 + (mi >> 1)) * 16);
                ldsm_x4(strip + a_off, pa);
                ldsm_x4(strip + 16 * kTcPStride + a_off, pl);
                const int key = quad * 32 + ks * 16 + (mi & 1) * 8 + rr;
#pragma unroll
                for (int np = 0; np < kTcDH / 16; np++) {
                    uint32_t r[4];
                    ldsm_x4_trans(vS + tc_tile_off(key, 2 * np + (mi >> 1)), r);
                    mma_bf16_16816(o[2 * np], pa, r[0], r[1]);
                    mma_bf16_16816(o[2 * np + 1], pa, r[2], r[3]);
                    mma_bf16_16816(o[2 * np], pl, r[0], r[1]);
                    mma_bf16_16816(o[2 * np + 1], pl, r[2], r[3]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(b_ev + 8 * s);               // the value block may be overwritten
        }
        if (warp == 2 && lane == 0) PASS_ATTN_TRACE(4);
    }
    __syncthreads();
    if (*(volatile int*)&s_abort) {
        if (tid == 0) {
            // let every copy that was requested land before the shared memory is given back
            const int issued = *(volatile int*)&s_issued;           // 2 per block: keys, values
            for (int f = issued - 4 < 0 ? 0 : issued - 4; f < issued; f++) {
                const int j = f >> 1;
                const uint32_t fb = ((f & 1) ? b_fv : b_fk) + 8 * (j & 1);
                const long long t0 = clock64();
                while (!mbar_try_wait(fb, (j >> 1) & 1))
                    if (clock64() - t0 > kWaitCycles) break;
            }
        }
        __syncthreads();
        if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, 64); }
        return;
    }
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, 64); }

    // merge the eight softmax warps; the key and value stages are free now and stage their outputs
    float* sm_o = reinterpret_cast<float*>(smem_tc + (base - smem_u32(smem_tc)));      // [8][16][128]
    if (warp >= 2) {
        const int sw = warp - 2, g = lane >> 2, t = lane & 3;
#pragma unroll
        for (int i = 0; i < 16; i++) {
            const float lt = warp_sum(l_part[i]);
            if (lane == i) { sm_m[sw * 16 + i] = m_run[i]; sm_l[sw * 16 + i] = lt; }
        }
        const bool live0 = g < M, live1 = g + 8 < M;
        const int swz = (g & 3) * 8;
#pragma unroll
        for (int n = 0; n < kTcDH / 8; n++) {
            const int col = (n * 8 + 2 * t) ^ swz;
            if (live0) *reinterpret_cast<float2*>(sm_o + ((sw * 16 + g) * kTcDH + col)) = make_float2(o[n][0], o[n][1]);
            if (live1) *reinterpret_cast<float2*>(sm_o + ((sw * 16 + g + 8) * kTcDH + col)) = make_float2(o[n][2], o[n][3]);
        }
    }
    __syncthreads();
    const size_t pbase = ((size_t)(b * p.md.H + head) * p.n_split + split) * 32;
    for (int idx = tid; idx < M * kTcDH; idx += kTcThreads) {
        const int i = idx / kTcDH, dcol = idx % kTcDH;
        float mm = -INFINITY;
#pragma unroll
        for (int w = 0; w < 8; w++) mm = fmaxf(mm, sm_m[w * 16 + i]);
        float acc = 0.f, ll = 0.f;
#pragma unroll
        for (int w = 0; w < 8; w++) {
            const float mw = sm_m[w * 16 + i];
            const float f = mw == -INFINITY ? 0.f : exp2f(mw - mm);
            acc += sm_o[(w * 16 + i) * kTcDH + (dcol ^ ((i & 3) * 8))] * f;
            ll += sm_l[w * 16 + i] * f;
        }
        if (p.n_split == 1) {
            const float v = acc / ll;
            const __nv_bfloat16 hi = __float2bfloat16_rn(v);
            p.out[(size_t)(row0 + i) * p.md.d + head * kTcDH + dcol] = hi;
            p.out[(size_t)(p.lo_row0 + row0 + i) * p.md.d + head * kTcDH + dcol] = __float2bfloat16_rn(v - __bfloat162float(hi));
        } else {
            p.part_o[(pbase + i) * kTcDH + dcol] = acc;
            if (dcol == 0) { p.part_ml[(pbase + i) * 2] = mm; p.part_ml[(pbase + i) * 2 + 1] = ll; }
        }
    }
    if (p.n_split == 1) return;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        PASS_ATTN_TRACE(5);
        const int prev = atomicAdd(p.counters + b * p.md.H + head, 1);
        s_last = prev == p.n_split - 1;
        if (s_last) p.counters[b * p.md.H + head] = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const size_t hb = (size_t)(b * p.md.H + head) * p.n_split * 32;
    float* sm_f = sm_o;                                              // [n_split][32] weight of slice s for row i
    if (p.n_split <= 4) attn_merge<kTcDH, 4, 4, kTcThreads>(p, hb, row0, head, sm_f);
    else attn_merge<kTcDH, kAttnMaxSplit, 2, kTcThreads>(p, hb, row0, head, sm_f);
    if (p.trace) {
        __syncthreads();
        if (tid == 0) PASS_ATTN_TRACE(6);
    }
}

}  // namespace pass
