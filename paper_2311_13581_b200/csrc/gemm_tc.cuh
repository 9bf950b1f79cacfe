// Weight-streaming skinny GEMM for the bf16 decoder step on sm_100a.
//
//   Y[r][n] = sum_k X[r][k] * W[n][k],   r < R <= 128 token rows, W bf16 [N][K] row-major
//
// The step is bound by reading W once from HBM (the paper's premise: "reading the full set of
// parameters from memory ... forms the primary bottleneck"), so the kernel is built around the
// weight stream:
//   * W tiles [128 features x 64 k] (128-byte rows, 128B swizzle) arrive by TMA into a shared-memory
//     ring; the matching activation tile [npad rows x 64 k] rides in the same stage.
//   * tcgen05.mma with the WEIGHT tile as operand A (M = 128) and the token rows as operand B
//     (N = npad, a multiple of 16), fp32 accumulators in TMEM: the token dimension is padded to
//     16s, not to 64/128.  Activations are carried as bf16 hi + bf16 lo rows (x = hi + lo), which
//     doubles N at no HBM cost and keeps activation rounding out of the result.
//   * stream-K: the (tile, k-block) units of one GEMM are cut into equal contiguous ranges, one per
//     CTA (one CTA per SM), so every SM pulls the same number of weight bytes whatever N is; with at
//     least as many tiles as CTAs only the n_tiles mod CTAs odd tiles are streamed and the GEMM ends
//     on whole tiles (see get_piece).  A tile cut across CTAs is summed in k order - deterministic -
//     by one CTA, which then runs the fused epilogue: the CTA holding the tile's first k-blocks (that
//     piece is the last of its own range), which finds the other parts in EMPTY-or-value words (no
//     counter, see ll_gather).  Up to nine token rows (k <= 4) go through that in one pass of nine rows; more
//     rows (k >= 5, batches) in passes of eight, in an instantiation of the kernel with three epilogue groups
//     that take the passes in turn (k_gemm_tc_many).  (The prompt-chunk instantiation computes every unit
//     whole and shares nothing.)
//   * warp roles: warp 0 weight loads, warp 6 activation loads, warp 1 TMEM allocation + MMA issue,
//     warps 2-5 epilogue (TMEM -> registers -> fused epilogue; k_gemm_tc_many: also warps 8-11 and 12-15);
//     two accumulator buffers so the epilogue of one piece overlaps the main loop of the next.
//   * one launch runs a chain of dependent GEMMs (see k_gemm_tc) so that the weight ring never drains
//     at a GEMM boundary.
//   * programmatic dependent launch: weight tiles do not depend on the previous kernel, so they are
//     requested before griddepcontrol.wait; only activation loads and the epilogue wait.
//   * every mbarrier wait is bounded; on expiry the CTA raises kStatusTimeout, drains its copies,
//     frees TMEM and returns.
#pragma once
#include <cuda.h>

#include "pass_common.cuh"

namespace pass {

constexpr int kTileN = 128;
constexpr int kTokTile = 256;                           // token rows of one accumulator at most (the MMA's N)
constexpr int kBlockK = 64;
constexpr int kGemmThreads = 256;
constexpr int kATileBytes = kTileN * kBlockK * 2;       // 16 KB
constexpr long long kWaitCycles = 400000000LL;          // ~0.2 s at 2 GHz
// Upper limit (ns) for which one mbarrier.try_wait may park the thread in hardware.  A parked waiter
// takes no issue slots from the epilogue warps on its scheduler and wakes as soon as the phase completes.
constexpr uint32_t kSuspendHintNs = 20000;

enum GemmEpilogue { kEpiLogits = 0, kEpiQKV = 1, kEpiResid = 2, kEpiSwiGLU = 3 };

struct GemmParams {
    int n_tiles, kb_per_tile;
    int seg_tiles0, seg_tiles1;    // plain mode: tiles of weight map 0 and 1 (the rest is map 2)
    int interleave;                // 1: tile t = rows [64t, 64t+64) of map 0 (gate) and of map 1 (up)
    int packed;                    // 1: the weight maps are over the packed copy [tile][k-block][box rows][64]
                                   // (see k_pack_weight): a box is addressed by its number, not by row and column
    int npad, rh, R;               // B rows (hi | lo halves of rh rows each), live rows
    int n_tok_tiles;               // > 0 (prompt chunks): the token rows are cut into tiles of npad rows too; unit u of
                                   // the schedule is (feature tile u / n_tok_tiles, token tile u % n_tok_tiles) and
                                   // n_tiles counts units.  0: one token tile, unit = feature tile
    int whole_only;                // 1: every unit is computed whole by one CTA (unit j * CTAs + c), nothing is split
    int has_lo;                    // 1: token row r is B row r (bf16 hi part) + B row rh + r (lo part), R <= rh;
                                   // 0: npad plain bf16 rows (prompt chunks of up to 256 tokens), R <= npad
    int stages;
    int epi;
    int n_out;                     // output features in total
    float* partial_ws;             // [gridDim][2][rows][128] fp32 + arrival counter per tile: prompt-chunk instantiation only
    float* ll_ws;                  // [gridDim][2][rh][128] fp32 words, EMPTY between launches: every launch of the step's kernel
    int* tile_counters;            // [n_tiles], zero between launches
    int* status;
    // rstd of the input rows (epilogues that follow an RMSNorm): parts [n_parts_in][kRowsCap]
    const float* sumsq_in;
    int n_parts_in;
    float inv_d_in, eps;
    // kEpiLogits
    float* logits;                 // [R][n_out]
    // kEpiQKV
    float* q_out;                  // [R][d]
    const float2* rope_cs;         // [R][dh/2]
    const int* row_seq;
    const int* row_pos;
    ModelDims md;
    int layer;
    __nv_bfloat16* kc;
    __nv_bfloat16* vc;
    // kEpiResid
    float* h;                      // [R][d] residual stream, updated in place
    const __nv_bfloat16* gain_next;
    __nv_bfloat16* xn_out;         // [2*rh_out.. rows][d]: hi rows then lo rows
    int xn_lo_row0;                // first lo row of xn_out / act_out
    float* sumsq_out;              // [n_tiles][kRowsCap]
    // kEpiSwiGLU
    __nv_bfloat16* act_out;        // [rows][f]
};

// ------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kSuspendHintNs) : "memory");
    return ok;
}
// Bounded wait: false when the CTA is giving up (another role timed out, or this wait did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* s_abort, int* g_status) {
    if (mbar_try_wait(bar, parity)) return true;          // the usual case costs no clock read
    const long long t0 = clock64();
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 127u) == 127u) {
            if (*s_abort) return false;
            if (clock64() - t0 > kWaitCycles) {
                *s_abort = 1;
                atomicOr(g_status, kStatusTimeout);
                return false;
            }
        }
    }
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"((uint64_t)map), "r"(bar), "r"(x), "r"(y), "l"(policy) : "memory");
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void griddep_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void griddep_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&v)[8]) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 8; i++) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void epi_bar() {            // the 128 epilogue threads only
    asm volatile("bar.sync 1, 128;" ::: "memory");
}
// MANY: kEpiGroups groups of 128 epilogue threads (barriers 1 .. kEpiGroups), and one more barrier for all of them
constexpr int kEpiGroups = 3;
template <bool MANY>
__device__ __forceinline__ void epi_bar_g(int group) {
    if (!MANY) asm volatile("bar.sync 1, 128;" ::: "memory");
    else asm volatile("bar.sync %0, 128;" ::"r"(1 + group) : "memory");
}
template <bool MANY>
__device__ __forceinline__ void epi_bar_all() {
    if (!MANY) asm volatile("bar.sync 1, 128;" ::: "memory");
    else asm volatile("bar.sync %0, %1;" ::"n"(kEpiGroups + 1), "n"(kEpiGroups * 128) : "memory");
}

// Shared-memory matrix descriptor: K-major tile with 128-byte rows, 128B swizzle; 8-row groups are
// 1024 bytes apart (stride byte offset), descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;                 // leading byte offset (unused with swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset
    d |= (uint64_t)1 << 46;                 // version
    d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
    return d;
}
// kind::f16 instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = npad.
__device__ __forceinline__ uint32_t instr_desc_bf16(int npad) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(npad >> 3) << 17) | ((uint32_t)(kTileN >> 4) << 24);
}

// ------------------------------------------------------------------------------------ schedule
struct Piece {
    int tile, kb0, kb1;      // k-blocks [kb0, kb1) of the tile
    int n_pieces, index;     // how many CTAs share the tile, and which of them this is (k order)
    int slot;                // partial slot of this CTA (0 = its first piece, 1 = a later one)
    int first_slot;          // slot used by the tile's first contributor (the only one that may have begun earlier)
};

__host__ __device__ __forceinline__ long long unit_start(long long c, long long U, long long G) { return c * U / G; }
__host__ __device__ __forceinline__ int unit_owner(long long x, long long U, long long G) {
    return (int)(((x + 1) * G - 1) / U);
}

// The it-th piece of CTA `c`; returns false when the CTA's range is exhausted.
//
// With at least as many tiles as CTAs the schedule has two phases.  First the n_tiles mod G "odd" tiles
// are streamed: their (tile, k-block) units are dealt out evenly, so tiles are shared and the last CTA to
// deliver sums the parts - early in the GEMM, while the MMAs already work on what follows.  Then every
// CTA computes whole tiles of its own.  The GEMM therefore ends on whole tiles, whose epilogue needs no
// other CTA: no arrival counter and no trip for partial sums on the path to the next GEMM.  With fewer
// tiles than CTAs everything is streamed.
__host__ __device__ __forceinline__ bool get_piece(const GemmParams& p, int c, int G, int it, Piece& out) {
    if (p.whole_only) {
        // prompt chunks: many large units, each done whole; CTAs that run side by side take neighbouring units,
        // i.e. the token tiles of the same few feature tiles, so a weight tile leaves HBM once and is then found in L2
        const long long tile = (long long)it * G + c;
        if (tile >= p.n_tiles) return false;
        out.tile = (int)tile;
        out.kb0 = 0;
        out.kb1 = p.kb_per_tile;
        out.n_pieces = 1;
        out.index = out.slot = out.first_slot = 0;
        return true;
    }
    const int rounds = p.n_tiles >= G ? p.n_tiles / G : 0;      // whole tiles per CTA
    const int n_sk = p.n_tiles - rounds * G;                     // tiles that are streamed, [0, n_sk)
    const long long U = (long long)n_sk * p.kb_per_tile;
    int sk_pieces = 0;
    if (U > 0) {
        int Gs = G;
        if (Gs > U) Gs = (int)U;      // fewer units than CTAs: only the first U CTAs stream
        if (c < Gs) {
            const long long s = unit_start(c, U, Gs), e = unit_start(c + 1, U, Gs);
            if (s < e) {
                const int t0 = (int)(s / p.kb_per_tile);
                sk_pieces = (int)((e - 1) / p.kb_per_tile) - t0 + 1;
                if (it < sk_pieces) {
                    const int tile = t0 + it;
                    const long long ts = (long long)tile * p.kb_per_tile;
                    const long long a = ts > s ? ts : s;
                    const long long b = (ts + p.kb_per_tile) < e ? (ts + p.kb_per_tile) : e;
                    out.tile = tile;
                    out.kb0 = (int)(a - ts);
                    out.kb1 = (int)(b - ts);
                    const int c_first = unit_owner(ts, U, Gs), c_last = unit_owner(ts + p.kb_per_tile - 1, U, Gs);
                    out.n_pieces = c_last - c_first + 1;
                    out.index = c - c_first;
                    out.slot = (a == s) ? 0 : 1;
                    out.first_slot = (unit_start(c_first, U, Gs) >= ts) ? 0 : 1;
                    return true;
                }
            }
        }
    }
    const int j = it - sk_pieces;
    if (j >= rounds) return false;
    out.tile = n_sk + j * G + c;
    out.kb0 = 0;
    out.kb1 = p.kb_per_tile;
    out.n_pieces = 1;
    out.index = 0;
    out.slot = 0;
    out.first_slot = 0;
    return true;
}

// ------------------------------------------------------------------------------------ epilogues
// Thread = one feature of the tile (TMEM lane); v[j] = result for token rows c0 .. c0+NR-1 (NR = 8, or 9 so
// that the 1 + 2k rows of k = 4 look-ahead tokens go through in one pass).
struct EpiCtx {
    int lane_in_tile;        // 0..127
    float* s_rstd;           // [kTokTile]
    float* s_x;              // [128][9] exchange buffer
    const unsigned long long* s_kvoff;   // [kTokTile] cache offset of head 0, feature 0 of each token row (kEpiQKV)
    int row_base;            // first token row of the token tile being finished (0 unless the rows are tiled)
    int rows_live;           // live rows of that token tile; s_rstd / s_kvoff are indexed by the row within the tile
    int group;               // epilogue group of this thread (0 unless the kernel has two)
    int out_row_base;        // row of xn_out / act_out that holds the tile's first token (its lo part xn_lo_row0 further
                             // down): token tiles of hi | lo rows are laid out one after another, as the next GEMM reads them
};

__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(x);
    lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// hv_pre: for kEpiResid the caller may hand in the residual values h[c0..c0+7][n] it has already
// loaded (so that this trip to L2 overlaps with another); nullptr = load them here.
// g_pre / cs_pre: likewise the next norm's gain for this feature (kEpiResid) and the eight rotation pairs
// (kEpiQKV), fetched by the caller while it was still waiting for the accumulator.
template <int NR, bool BIG, bool MANY = false>
__device__ __forceinline__ void epi_store(const GemmParams& p, const EpiCtx& ec, int tile, int c0, float (&v)[NR],
                                          const float* hv_pre = nullptr, const float* g_pre = nullptr,
                                          const float2* cs_pre = nullptr) {
    const int L = ec.lane_in_tile;
    // the step's kernel (BIG = false) has one token tile of hi | lo rows: these fold to constants there
    const int row_base = BIG ? ec.row_base : 0, out_row_base = BIG ? ec.out_row_base : 0;
    const int rows_live = BIG ? ec.rows_live : p.R;
    const bool has_lo = BIG ? p.has_lo != 0 : true;
    if (p.epi == kEpiLogits) {
        const int n = tile * kTileN + L;
        if (n < p.n_out) {
#pragma unroll
            for (int j = 0; j < NR; j++)
                if (c0 + j < rows_live) p.logits[(size_t)(row_base + c0 + j) * p.n_out + n] = v[j] * ec.s_rstd[c0 + j];
        }
    } else if (p.epi == kEpiQKV) {
        const int d = p.md.d, dh = p.md.dh;
        const int n = tile * kTileN + L;
        const int which = n / d, c = n % d, head = c / dh, i = c % dh;
        // everything that is read is fetched before the first store, so that the loads overlap
        size_t kvo[NR];
        float2 cs[NR];
        const size_t head_off = ((size_t)head * p.md.cap) * dh + i;
#pragma unroll
        for (int j = 0; j < NR; j++) {
            const int r = min(c0 + j, rows_live - 1);
            kvo[j] = (size_t)ec.s_kvoff[r] + head_off;
            cs[j] = cs_pre ? cs_pre[j] : __ldg(p.rope_cs + (size_t)(row_base + r) * (dh / 2) + (i >> 1));
        }
#pragma unroll
        for (int j = 0; j < NR; j++) {
            const int r = c0 + j;
            const float x = v[j] * (r < rows_live ? ec.s_rstd[r] : 0.f);
            const float other = __shfl_xor_sync(0xffffffffu, x, 1);
            if (r < rows_live) {
                if (which == 2) {
                    p.vc[kvo[j]] = __float2bfloat16_rn(x);
                } else {
                    const float y = (i & 1) ? other * cs[j].y + x * cs[j].x : x * cs[j].x - other * cs[j].y;
                    if (which == 0) p.q_out[(size_t)(row_base + r) * d + c] = y;
                    else p.kc[kvo[j]] = __float2bfloat16_rn(y);
                }
            }
        }
    } else if (p.epi == kEpiResid) {
        const int d = p.n_out;
        const int n = tile * kTileN + L;
        const float g = g_pre ? *g_pre : (n < d ? __bfloat162float(p.gain_next[n]) : 0.f);
        const int warp_q = (threadIdx.x >> 5) & 3, lane = threadIdx.x & 31;
        float ss[NR], hv[NR];
#pragma unroll
        for (int j = 0; j < NR; j++)      // all loads first: they are independent of the stores below
            hv[j] = hv_pre ? hv_pre[j] : ((c0 + j < rows_live && n < d) ? __ldcg(p.h + (size_t)(row_base + c0 + j) * d + n) : 0.f);
#pragma unroll
        for (int j = 0; j < NR; j++) {
            const int r = row_base + c0 + j;
            float hn = 0.f;
            if (c0 + j < rows_live && n < d) {
                hn = hv[j] + v[j];
                p.h[(size_t)r * d + n] = hn;
                __nv_bfloat16 hi, lo;
                split_bf16(hn * g, hi, lo);
                const size_t orow = (size_t)(out_row_base + c0 + j);
                p.xn_out[orow * d + n] = hi;
                if (has_lo) p.xn_out[(orow + p.xn_lo_row0) * d + n] = lo;
            }
            ss[j] = hn * hn;
        }
        // the butterfly reductions of all rows side by side: each level issues NR independent shuffles, so
        // the shuffle latency is paid five times, not 5 NR times
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
            for (int j = 0; j < NR; j++) ss[j] += __shfl_xor_sync(0xffffffffu, ss[j], o);
        }
        epi_bar_g<MANY>(ec.group);                                  // s_x free
        if (lane == 0) {
#pragma unroll
            for (int j = 0; j < NR; j++) ec.s_x[warp_q * NR + j] = ss[j];
        }
        epi_bar_g<MANY>(ec.group);
        if (L < NR && c0 + L < rows_live)
            p.sumsq_out[(size_t)tile * kRowsCap + row_base + c0 + L] =
                ec.s_x[L] + ec.s_x[NR + L] + ec.s_x[2 * NR + L] + ec.s_x[3 * NR + L];
    } else {  // kEpiSwiGLU: lanes 0..63 gate features 64*tile + L, lanes 64..127 the matching up features
        // Both halves of the threads work after the exchange: a gate lane finishes the even rows of its
        // feature (it reads the up values from the exchange buffer), the matching up lane the odd rows
        // (it reads the gate values).
        epi_bar_g<MANY>(ec.group);                                  // s_x free
#pragma unroll
        for (int j = 0; j < NR; j++) ec.s_x[L * 9 + j] = v[j];
        epi_bar_g<MANY>(ec.group);
        const int feat = L & 63, other = L < 64 ? L + 64 : L - 64, n = tile * 64 + feat;
        if (n < p.n_out) {
#pragma unroll
            for (int j = 0; j < NR; j++) {
                if (c0 + j < rows_live && ((j & 1) == (L >> 6))) {
                    const float rs = ec.s_rstd[c0 + j];
                    const float mine = v[j] * rs, theirs = ec.s_x[other * 9 + j] * rs;
                    const float g = L < 64 ? mine : theirs, u = L < 64 ? theirs : mine;
                    __nv_bfloat16 hi, lo;
                    split_bf16(g / (1.f + __expf(-g)) * u, hi, lo);
                    const size_t orow = (size_t)(out_row_base + c0 + j);
                    p.act_out[orow * p.n_out + n] = hi;
                    if (has_lo) p.act_out[(orow + p.xn_lo_row0) * p.n_out + n] = lo;
                }
            }
        }
    }
}

// Partial sums are handed over without a counter: a slot word is either EMPTY (all
// bits set - a NaN pattern that fp32 arithmetic never produces, it makes the canonical 0x7fffffff) or a
// value.  Contributors just store their values; the finisher loads the words it needs and repeats the
// load until none of them is empty; when it is done with a tile it stores EMPTY back, so every launch
// finds the slots as the first one did (the workspace is filled with 0xff bytes when it is created).
// A 4-byte word is written and read in one piece, hence no fence, no arrival counter and no second trip
// to L2.  Slot layout [row][feature].  Should a value ever come out as the EMPTY pattern, the finisher
// runs into its bounded wait and the launch reports a time-out; nothing is consumed silently.
constexpr uint32_t kEmptyWord = 0xFFFFFFFFu;
__device__ __forceinline__ void st_word(float* p, uint32_t w) {
    asm volatile("st.relaxed.gpu.global.b32 [%0], %1;" ::"l"(p), "r"(w) : "memory");
}
__device__ __forceinline__ uint32_t ld_word(const float* p) {
    uint32_t w;
    asm volatile("ld.relaxed.gpu.global.b32 %0, [%1];" : "=r"(w) : "l"(p) : "memory");
    return w;
}
constexpr int kLLRows = 9;          // rows fetched per trip (1 + 2k rows of k = 4 look-ahead tokens)
constexpr int kLLPeers = 5;         // other contributors fetched per trip

// acc[j] += value of row row0 + j from each of `n_others` contributors (slots `first` + q * stride, k order),
// for this thread's feature.  Spins (bounded) until no word is EMPTY, then marks the words EMPTY again if
// `reset`.  Returns false on time-out.
template <int kLLRows>
__device__ __forceinline__ bool ll_gather(float* first, size_t stride, int n_others, int row0, int nrows,
                                          float (&acc)[kLLRows], volatile int* s_abort, int* g_status) {
    bool fine = true;
    for (int q0 = 0; q0 < n_others; q0 += kLLPeers) {
        uint32_t w[kLLPeers][kLLRows];
        const long long t0 = clock64();
        for (;;) {
            bool ok = true;
#pragma unroll
            for (int qq = 0; qq < kLLPeers; qq++) {
                const float* src = first + (size_t)(q0 + qq) * stride + (size_t)row0 * kTileN;
#pragma unroll
                for (int j = 0; j < kLLRows; j++)
                    w[qq][j] = (q0 + qq < n_others && j < nrows) ? ld_word(src + (size_t)j * kTileN) : 0u;
            }
#pragma unroll
            for (int qq = 0; qq < kLLPeers; qq++)
#pragma unroll
                for (int j = 0; j < kLLRows; j++) ok &= w[qq][j] != kEmptyWord;
            if (ok) break;
            if (*s_abort || clock64() - t0 > kWaitCycles) {
                *s_abort = 1;
                atomicOr(g_status, kStatusTimeout);
                fine = false;
                break;
            }
        }
#pragma unroll
        for (int qq = 0; qq < kLLPeers; qq++)
#pragma unroll
            for (int j = 0; j < kLLRows; j++) acc[j] += __uint_as_float(w[qq][j]);
    }
    return fine;
}
// the words ll_gather consumed become EMPTY again (after the tile's results are out: off the critical path)
__device__ __forceinline__ void ll_reset(float* first, size_t stride, int n_others, int nrows) {
    for (int q = 0; q < n_others; q++)
        for (int j = 0; j < nrows; j++) st_word(first + (size_t)q * stride + (size_t)j * kTileN, kEmptyWord);
}

// ------------------------------------------------------------------------------------ kernel
// A launch runs a CHAIN of up to kMaxOps dependent GEMMs (for a decoder layer: output projection ->
// gate|up -> down -> next layer's QKV).  Inside the chain there is no kernel boundary: the weight
// producer walks straight from the last tile of one GEMM into the first tile of the next, so the
// shared-memory ring stays full of weights while the consumers wait for the previous GEMM's epilogues.
// The wait itself is a counter per GEMM ("tiles whose epilogue is complete"), bumped with release
// semantics by the CTA that finishes a tile and read with acquire semantics by every CTA's activation
// producer and epilogue warps before they touch the next GEMM.  The counters only grow from launch to
// launch (the host clears them at the start of a forward and tells each launch which totals to wait for),
// so a launch ends without any bookkeeping.  All CTAs of the grid are resident (one per SM), the counter
// only ever waits for work of an EARLIER GEMM, and every wait is bounded.
constexpr int kMaxOps = 4;
// pieces of a CTA per GEMM that are worked out once and kept in shared memory.  A CTA has at most
// n_tiles / CTAs + 2 pieces (whole tiles plus at most two streamed ones)
constexpr int kPieceCache = 16;
struct ChainMaps { CUtensorMap m[kMaxOps][4]; };      // per GEMM: weight maps 0..2, activation map
struct ChainParams {
    int n_ops;
    int stages;
    int npad;                  // row padding, shared by all GEMMs of the chain
    int test_stuck;            // test hook: the first GEMM's contributors keep their partial sums to themselves (or do
                               // not announce them), so a bounded wait runs out and the launch reports kStatusTimeout
    int hold;                  // 1: no weight request for a GEMM before this CTA's epilogue of the previous one is over
                               // (off by default)
    int* op_done;              // [kMaxOps] tiles completed by the GEMM in chain position i, counted over ALL launches
                               // since the counters were last cleared (the host clears them at the start of a forward)
    int op_target[kMaxOps];    // value of op_done[i] once this launch's GEMM i is complete
    int* status;
    unsigned long long* trace;     // optional %globaltimer stamps [kMaxOps][CTA][8] of this launch (nullptr = off)
    GemmParams op[kMaxOps];
};
// Only every 16th CTA leaves stamps: reads of %globaltimer from all CTAs at once queue up behind one another
// (tens of microseconds for 148 readers) and would stretch the very hand-overs the trace is meant to show.
#define PASS_TRACE(oi, slot) do { if (TRACE && cp.trace && (blockIdx.x & 15) == 0) cp.trace[((size_t)(oi) * gridDim.x + blockIdx.x) * 8 + (slot)] = global_ns(); } while (0)

__device__ __forceinline__ bool wait_count(const int* counter, int target, volatile int* s_abort, int* g_status) {
    const long long t0 = clock64();
    for (;;) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
        if (v >= target) return true;
        if (*s_abort) return false;
        if (clock64() - t0 > kWaitCycles) {
            *s_abort = 1;
            atomicOr(g_status, kStatusTimeout);
            return false;
        }
        __nanosleep(64);
    }
}

// weight tile of (tile, k-block): box index 0/1 -> (map, row); plain mode has a single 128-row box.
// The coordinates of k-block kb are (kb * kBlockK, y) in a row-major matrix and (0, y * kb_per_tile +
// kb * box rows) in the packed copy; weight_xy turns the one into the other.
__device__ __forceinline__ void weight_box(const GemmParams& p, const CUtensorMap* m4, int tile, int box,
                                           const CUtensorMap*& m, int& y) {
    if (p.interleave) {
        m = m4 + (box ? 1 : 0);
        y = tile * 64;
    } else {
        int tl = tile;
        m = m4;
        if (tl >= p.seg_tiles0) {
            tl -= p.seg_tiles0;
            m = m4 + 1;
            if (tl >= p.seg_tiles1) { tl -= p.seg_tiles1; m = m4 + 2; }
        }
        y = tl * kTileN;
    }
}
__device__ __forceinline__ void weight_xy(const GemmParams& p, int y_rowmajor, int kb, int& x, int& y) {
    if (p.packed) {
        x = 0;
        y = y_rowmajor * p.kb_per_tile + kb * (p.interleave ? 64 : kTileN);
    } else {
        x = kb * kBlockK;
        y = y_rowmajor;
    }
}

// BIG = false: the decode step's kernel (hi | lo rows, one token tile).  BIG = true adds what prompt chunks
// need (token tiles, plain bf16 rows, whole-unit schedule, loads one row group ahead in the epilogue); it is a
// second instantiation so that the step's kernel keeps its registers.
template <bool BIG, bool MANY = false, bool TRACE = true>
__device__ __forceinline__ void gemm_chain_body(const ChainMaps& maps, const ChainParams& cp) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t s_bars[2 * 16 + 4];   // full[S], empty[S], acc_full[2], acc_empty[2]
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ int s_issued, s_issued_b;
    __shared__ int s_epi_done;
    __shared__ int s_last;
    __shared__ int s_epi_fail;
    // (the step's kernel shares its SM with an attention CTA of 64 KB and fills the rest with a seventh stage of its
    // ring: static shared memory that grows by more than 12 KB ends that)
    __shared__ float s_rstd[BIG ? kTokTile : kMaxRows];
    __shared__ unsigned long long s_kvoff[BIG ? kTokTile : kMaxRows];
    __shared__ float s_x[(MANY ? kEpiGroups : 1) * 128 * 9];
    // this CTA's pieces of every GEMM of the chain, worked out once (the schedule arithmetic uses
    // 64-bit divisions, which would otherwise sit between two pieces on every role's critical path)
    __shared__ Piece s_piece[kMaxOps][kPieceCache];
    __shared__ int s_piece_ok[kMaxOps][kPieceCache];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = cp.stages;
    const int G = gridDim.x, cta = blockIdx.x;
    if (threadIdx.x >= 128 && threadIdx.x < 128 + kMaxOps * kPieceCache) {
        const int oi = (threadIdx.x - 128) / kPieceCache, it = (threadIdx.x - 128) % kPieceCache;
        Piece pc;
        pc.tile = pc.kb0 = pc.kb1 = pc.n_pieces = pc.index = pc.slot = pc.first_slot = 0;
        const bool v = oi < cp.n_ops && get_piece(cp.op[oi], cta, G, it, pc);
        s_piece[oi][it] = pc;
        s_piece_ok[oi][it] = v ? 1 : 0;
    }
    auto fetch_piece = [&](int oi, int it, Piece& out) -> bool {
        if (it < kPieceCache) {
            if (!s_piece_ok[oi][it]) return false;
            out = s_piece[oi][it];
            return true;
        }
        // (the step's kernels never get here: the host sends a launch whose CTAs have more pieces than the cache
        // holds to the traced instantiation, which like the prompt-chunk one keeps the arithmetic)
        if (BIG || TRACE) return get_piece(cp.op[oi], cta, G, it, out);
        return false;
    };
    const uint32_t stage_bytes = kATileBytes + cp.npad * 128;
    const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar_full = smem_u32(&s_bars[0]), bar_empty = bar_full + 8 * 16;
    const uint32_t bar_accf = bar_full + 8 * 32, bar_acce = bar_accf + 16;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * cp.npad) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; s++) { mbar_init(bar_full + 8 * s, 2); mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < 2; b++) { mbar_init(bar_accf + 8 * b, 1); mbar_init(bar_acce + 8 * b, MANY ? 4 * kEpiGroups : 4); }
        s_abort = 0;
        s_issued = 0;
        s_issued_b = 0;
        s_epi_done = -1;
        s_epi_fail = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&s_tmem_base), tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    griddep_launch_dependents();

    // One TMA request costs its issuing thread a couple of hundred cycles, so the requests of a stage
    // are spread over two single-thread roles in different warps:
    //   warp 0: weight box 0 of every stage (never waits for anything but ring space: weights are constant)
    //   warp 6: activation tile of every stage (+ weight box 1 when the stage has two boxes)
    if (warp == 0) {
        // ---------------------------------------------------------------- weight producer
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first();
            int fill = 0, s = 0;
            uint32_t ph = 0;
            bool ok = true;
            Piece pc;
            for (int oi = 0; ok && oi < cp.n_ops; oi++) {
                const GemmParams& p = cp.op[oi];
                const uint32_t a_box_bytes = p.interleave ? kATileBytes / 2 : kATileBytes;
                if (TRACE && cp.hold && oi > 0) {
                    const long long t0 = clock64();
                    while (*(volatile int*)&s_epi_done < oi - 1) {
                        if (*(volatile int*)&s_abort || clock64() - t0 > kWaitCycles) { ok = false; break; }
                        __nanosleep(100);
                    }
                }
                for (int it = 0; ok && fetch_piece(oi, it, pc); it++) {
                    const CUtensorMap* m;
                    int y;
                    weight_box(p, maps.m[oi], (BIG && p.n_tok_tiles > 0) ? pc.tile / p.n_tok_tiles : pc.tile, 0, m, y);
                    for (int kb = pc.kb0; kb < pc.kb1; kb++) {
                        // (stage and phase are counted along: a division by the ring depth per stage is time this
                        // single thread does not have)
                        if (!mbar_wait(bar_empty + 8 * s, ph ^ 1, &s_abort, cp.status)) { ok = false; break; }
                        mbar_expect_tx(bar_full + 8 * s, a_box_bytes);
                        int wx, wy;
                        weight_xy(p, y, kb, wx, wy);
                        tma_load_2d(tiles_base + s * stage_bytes, m, bar_full + 8 * s, wx, wy, pol_w);
                        fill++;
                        if (++s == S) { s = 0; ph ^= 1; }
                    }
                }
            }
            *(volatile int*)&s_issued = fill;          // for the teardown after a wait that ran out
        }
    } else if (warp == 6) {
        // ---------------------------------------------------------------- activation producer
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
            int fill = 0, s = 0;
            uint32_t ph = 0;
            bool ok = true;
            Piece pc;
            griddep_wait();                    // the first GEMM's activations are the previous kernel's output
            for (int oi = 0; ok && oi < cp.n_ops; oi++) {
                const GemmParams& p = cp.op[oi];
                const uint32_t a_box_bytes = p.interleave ? kATileBytes / 2 : kATileBytes;
                if (oi > 0) {
                    // activations of this GEMM = results of the previous one, written by other SMs
                    if (!wait_count(cp.op_done + oi - 1, cp.op_target[oi - 1], &s_abort, cp.status)) break;
                    asm volatile("fence.proxy.async;" ::: "memory");   // generic-proxy data -> TMA reads
                }
                PASS_TRACE(oi, 0);
                for (int it = 0; ok && fetch_piece(oi, it, pc); it++) {
                    const CUtensorMap* m;
                    int y;
                    weight_box(p, maps.m[oi], (BIG && p.n_tok_tiles > 0) ? pc.tile / p.n_tok_tiles : pc.tile, 1, m, y);
                    const int b_row0 = (BIG && p.n_tok_tiles > 0) ? (pc.tile % p.n_tok_tiles) * p.npad : 0;    // token tile
                    for (int kb = pc.kb0; kb < pc.kb1; kb++) {
                        if (!mbar_wait(bar_empty + 8 * s, ph ^ 1, &s_abort, cp.status)) { ok = false; break; }
                        const uint32_t dst = tiles_base + s * stage_bytes;
                        if (p.interleave) {
                            mbar_expect_tx(bar_full + 8 * s, stage_bytes - a_box_bytes);
                            int wx, wy;
                            weight_xy(p, y, kb, wx, wy);
                            tma_load_2d(dst + kATileBytes / 2, m, bar_full + 8 * s, wx, wy, pol_w);
                        } else {
                            mbar_expect_tx(bar_full + 8 * s, stage_bytes - kATileBytes);
                        }
                        tma_load_2d(dst + kATileBytes, &maps.m[oi][3], bar_full + 8 * s, kb * kBlockK, b_row0, pol_x);
                        fill++;
                        if (++s == S) { s = 0; ph ^= 1; }
                    }
                }
            }
            *(volatile int*)&s_issued_b = fill;        // for the teardown after a wait that ran out
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issue
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(cp.npad);
            int pidx = 0, s = 0;
            uint32_t ph = 0;
            bool ok = true;
            Piece pc;
            for (int oi = 0; ok && oi < cp.n_ops; oi++) {
                const GemmParams& p = cp.op[oi];
                bool first = true;
                for (int it = 0; ok && fetch_piece(oi, it, pc); it++, pidx++) {
                    const int buf = pidx & 1;
                    if (!mbar_wait(bar_acce + 8 * buf, ((pidx >> 1) & 1) ^ 1, &s_abort, cp.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + buf * cp.npad;
                    for (int kb = pc.kb0; kb < pc.kb1; kb++) {
                        if (!mbar_wait(bar_full + 8 * s, ph, &s_abort, cp.status)) { ok = false; break; }
                        if (first) { PASS_TRACE(oi, 1); first = false; }
                        tc_fence_after();
                        const uint32_t a_addr = tiles_base + s * stage_bytes, b_addr = a_addr + kATileBytes;
                        const uint64_t a_desc = smem_desc_sw128(a_addr), b_desc = smem_desc_sw128(b_addr);
#pragma unroll
                        for (int kk = 0; kk < kBlockK / 16; kk++)
                            umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb > pc.kb0 || kk > 0) ? 1u : 0u);
                        umma_commit(bar_empty + 8 * s);      // frees the stage when these MMAs have read it
                        if (++s == S) { s = 0; ph ^= 1; }
                    }
                    if (ok) umma_commit(bar_accf + 8 * buf);  // accumulator of this piece complete
                }
                PASS_TRACE(oi, 2);
            }
        }
    } else if ((warp >= 2 && warp <= 5) || (MANY && warp >= 8)) {
        // ---------------------------------------------------------------- epilogue (128 threads; MANY: kEpiGroups
        // groups of 128, warps 2-5, 8-11, 12-15, which share every tile: the passes of eight token rows go round)
        const int wq = warp & 3;                      // TMEM lanes 32*wq .. 32*wq+31
        const int ge = MANY && warp >= 8 ? (warp - 4) >> 2 : 0;
        EpiCtx ec;
        ec.lane_in_tile = wq * 32 + lane;
        ec.s_rstd = s_rstd;
        ec.s_x = s_x + ge * 128 * 9;
        ec.s_kvoff = s_kvoff;
        ec.group = ge;
        const int et = (warp - (ge ? 4 + 4 * ge : 2)) * 32 + lane;        // 0..127 within the group
        griddep_wait();
        int pidx = 0;
        bool ok = true;
        Piece pc;
        for (int oi = 0; ok && oi < cp.n_ops; oi++) {
            const GemmParams& p = cp.op[oi];
            if (oi > 0) {
                // one thread waits for the previous GEMM; the outcome is made uniform through the barrier
                if (et == 0 && ge == 0 && !wait_count(cp.op_done + oi - 1, cp.op_target[oi - 1], &s_abort, cp.status))
                    *(volatile int*)&s_epi_fail = 1;
                epi_bar_all<MANY>();                 // (both groups leave together, and nobody still reads the row tables)
                if (*(volatile int*)&s_epi_fail) { ok = false; break; }
            }
            // rstd of the input rows: eight lanes per row, each sums every eighth part (its loads are
            // independent, so a row costs one trip to L2 whatever the number of parts), then a fixed-order
            // butterfly.  The first accumulator of a short first piece may already be waiting for us.
            // (rows of the token tile that starts at row `base`; the tables are indexed by the row within the tile)
            auto fill_row_tables = [&](int base, int n_rows) {
                for (int r0 = 0; r0 < n_rows; r0 += 16) {
                    const int lr = r0 + (et >> 3), r = base + lr, l8 = et & 7;
                    float ss = 0.f;
                    if (p.sumsq_in && lr < n_rows) {
                        float part[4] = {0.f, 0.f, 0.f, 0.f};
                        for (int t0 = 0; t0 < p.n_parts_in; t0 += 32) {
#pragma unroll
                            for (int u = 0; u < 4; u++) {
                                const int t = t0 + u * 8 + l8;
                                if (t < p.n_parts_in) part[u] += __ldcg(p.sumsq_in + (size_t)t * kRowsCap + r);
                            }
                        }
                        ss = (part[0] + part[1]) + (part[2] + part[3]);
                    }
                    ss += __shfl_xor_sync(0xffffffffu, ss, 1);
                    ss += __shfl_xor_sync(0xffffffffu, ss, 2);
                    ss += __shfl_xor_sync(0xffffffffu, ss, 4);
                    if (lr < n_rows && l8 == 0) {
                        s_rstd[lr] = p.sumsq_in ? rsqrtf(ss * p.inv_d_in + p.eps) : 1.f;
                        if (p.epi == kEpiQKV)
                            s_kvoff[lr] = kv_index(p.md, p.layer, __ldg(p.row_seq + r), 0, __ldg(p.row_pos + r));
                    }
                }
            };
            int cur_tt = -1;
            ec.row_base = 0;
            ec.out_row_base = 0;
            ec.rows_live = p.R;
            if (!BIG || p.n_tok_tiles == 0) fill_row_tables(0, p.R);
            epi_bar_g<MANY>(ge);
            const bool has_lo = !BIG || p.has_lo;
            const int rows_acc = has_lo ? p.rh : p.npad;            // token rows held by an accumulator
            const size_t slot_floats = (size_t)rows_acc * kTileN;
            const bool signal = oi + 1 < cp.n_ops;   // a later GEMM of the chain waits for this one's tiles
            for (int it = 0; ok && fetch_piece(oi, it, pc); it++, pidx++) {
                const int buf = pidx & 1;
                // what the epilogue of this tile reads besides the accumulator is requested now, so that
                // the trip to L2 is over by the time the accumulator is complete
                float g_pre = 0.f;
                float2 cs_pre[kLLRows] = {};
                const bool pre = !MANY && p.rh == 16 && has_lo && pc.index == 0;
                if (pre && p.epi == kEpiResid) {
                    const int n = pc.tile * kTileN + ec.lane_in_tile;
                    g_pre = n < p.n_out ? __bfloat162float(p.gain_next[n]) : 0.f;
                }
                if (pre && p.epi == kEpiQKV) {
                    const int i2 = ((pc.tile * kTileN + ec.lane_in_tile) % p.md.dh) >> 1;
#pragma unroll
                    for (int j = 0; j < kLLRows; j++)
                        cs_pre[j] = __ldg(p.rope_cs + (size_t)min(j, p.R - 1) * (p.md.dh / 2) + i2);
                }
                int ftile = pc.tile;                           // feature tile of this piece
                if (BIG && p.n_tok_tiles > 0) {
                    ftile = pc.tile / p.n_tok_tiles;
                    const int tt = pc.tile % p.n_tok_tiles;
                    if (tt != cur_tt) {                        // another token tile: its rows' factors and cache offsets
                        epi_bar_g<MANY>(ge);
                        const int tile_tokens = p.has_lo ? p.rh : p.npad;
                        ec.row_base = tt * tile_tokens;
                        ec.out_row_base = tt * p.npad;
                        ec.rows_live = min(tile_tokens, p.R - ec.row_base);
                        fill_row_tables(ec.row_base, ec.rows_live);
                        cur_tt = tt;
                    }
                }
                // each thread waits for itself; the outcome is made uniform before any barrier is used
                if (!mbar_wait(bar_accf + 8 * buf, (pidx >> 1) & 1, &s_abort, cp.status)) *(volatile int*)&s_epi_fail = 1;
                epi_bar_all<MANY>();
                if (*(volatile int*)&s_epi_fail) { ok = false; break; }
                if (et == 0 && ge == 0) PASS_TRACE(oi, 4);
                tc_fence_after();
                const bool whole = pc.n_pieces == 1;
                const bool ll = !MANY && p.rh == 16 && has_lo;          // 9..16 rows (padded to 16): counter-free hand-over, fixed finisher
                float* ll_peer = nullptr;                      // finisher: the slots to mark empty once the tile is out
                int ll_n = 0;
                const uint32_t t_addr = tmem_base + ((uint32_t)(wq * 32) << 16) + buf * cp.npad;
                bool tile_done = whole;
                if (ll) {
                    float av[16];
#pragma unroll
                    for (int c0 = 0; c0 < 16; c0 += 8) {
                        float hi[8], lo[8];
                        tmem_ld8(t_addr + c0, hi);
                        tmem_ld8(t_addr + 16 + c0, lo);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 8; j++) av[c0 + j] = hi[j] + lo[j];
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_acce + 8 * buf);
                    if (!whole && pc.index != 0) {
                        // a later part of the tile: hand it to the CTA that holds the tile's first k-blocks
                        float* dst = p.ll_ws + ((size_t)cta * 2 + pc.slot) * slot_floats + ec.lane_in_tile;
#pragma unroll
                        for (int j = 0; j < 16; j++)
                            if (j < p.R && !(TRACE && cp.test_stuck && oi == 0)) st_word(dst + (size_t)j * kTileN, __float_as_uint(av[j]));
                    } else {
                        // A whole tile, or the tile's first part.  The first part is this CTA's LAST piece of the
                        // GEMM (its range ends inside the tile), so it is the natural finisher: the other parts
                        // were either computed at the very start of their CTAs' ranges or finish together with it.
                        tile_done = true;
                        const int n = pc.tile * kTileN + ec.lane_in_tile;
                        float hv[kLLRows];
#pragma unroll
                        for (int j = 0; j < kLLRows; j++)
                            hv[j] = (p.epi == kEpiResid && j < p.R && n < p.n_out) ? __ldcg(p.h + (size_t)j * p.n_out + n) : 0.f;
                        // every contributor but the first keeps its part in slot 0 (its range begins inside the tile)
                        float* peer = p.ll_ws + ((size_t)(cta + 1) * 2) * slot_floats + ec.lane_in_tile;
                        const size_t peer_stride = 2 * slot_floats;
                        // the (at most nine) rows go through the epilogue in one pass: the 1 + 2k rows of up to four
                        // look-ahead tokens (steps of more rows run in k_gemm_tc_many)
                        {
                            float a9[kLLRows], h9[kLLRows];
                            float2 cs9[kLLRows];
#pragma unroll
                            for (int j = 0; j < kLLRows; j++) { a9[j] = av[j]; h9[j] = hv[j]; cs9[j] = cs_pre[j]; }
                            if (!whole)
                                ll_gather<kLLRows>(peer, peer_stride, pc.n_pieces - 1, 0, min(p.R, kLLRows), a9, &s_abort, cp.status);
                            if (et == 0 && !whole) PASS_TRACE(oi, 5);
                            epi_store<kLLRows, BIG, MANY>(p, ec, pc.tile, 0, a9, p.epi == kEpiResid ? h9 : nullptr,
                                               p.epi == kEpiResid ? &g_pre : nullptr, p.epi == kEpiQKV ? cs9 : nullptr);
                        }
                        if (!whole) { ll_peer = peer; ll_n = pc.n_pieces - 1; }
                    }
                } else if (MANY) {
                    // Ten token rows or more (k >= 5, batches): the same counter-free hand-over, eight rows at a time;
                    // pass q (rows 8q .. 8q+7) belongs to epilogue group q mod kEpiGroups.
                    const bool contributor = !whole && pc.index != 0;
                    float* peer = p.ll_ws + ((size_t)(cta + 1) * 2) * slot_floats + ec.lane_in_tile;
                    const size_t peer_stride = 2 * slot_floats;
                    const int n = pc.tile * kTileN + ec.lane_in_tile;
                    if (p.epi == kEpiResid) g_pre = n < p.n_out ? __bfloat162float(p.gain_next[n]) : 0.f;
                    if (!contributor) tile_done = true;
                    const int n_pass = p.rh / 8;
                    bool released = false;
                    auto release_acc = [&]() {              // this warp has read the accumulator out: the MMA warp may have it back
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_acce + 8 * buf);
                        released = true;
                    };
#pragma unroll 1
                    for (int q = ge; q < n_pass; q += kEpiGroups) {
                        const int row = 8 * q;
                        float a8[8];
                        {
                            float hi[8], lo[8];
                            tmem_ld8(t_addr + row, hi);
                            tmem_ld8(t_addr + p.rh + row, lo);
                            tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 8; j++) a8[j] = hi[j] + lo[j];
                        }
                        if (q + kEpiGroups >= n_pass) release_acc();
                        if (row >= p.R) continue;
                        if (contributor) {
                            float* dst = p.ll_ws + ((size_t)cta * 2 + pc.slot) * slot_floats + ec.lane_in_tile;
#pragma unroll
                            for (int j = 0; j < 8; j++)
                                if (row + j < p.R && !(TRACE && cp.test_stuck && oi == 0)) st_word(dst + (size_t)(row + j) * kTileN, __float_as_uint(a8[j]));
                            continue;
                        }
                        float h8[8];
#pragma unroll
                        for (int j = 0; j < 8; j++)
                            h8[j] = (p.epi == kEpiResid && row + j < p.R && n < p.n_out) ? __ldcg(p.h + (size_t)(row + j) * p.n_out + n) : 0.f;
                        if (!whole)
                            ll_gather<8>(peer, peer_stride, pc.n_pieces - 1, row, min(p.R - row, 8), a8, &s_abort, cp.status);
                        epi_store<8, BIG, MANY>(p, ec, pc.tile, row, a8, p.epi == kEpiResid ? h8 : nullptr,
                                                p.epi == kEpiResid ? &g_pre : nullptr, nullptr);
                    }
                    if (!released) release_acc();
                    if (!contributor && !whole) { ll_peer = peer; ll_n = pc.n_pieces - 1; }
                } else if (BIG) {               // prompt chunks (the step's kernel never gets here: it has hi | lo rows)
                float* my_slot = p.partial_ws + ((size_t)cta * 2 + pc.slot) * slot_floats;
                // Whole tiles of many rows (prompt chunks): what the residual epilogue reads is requested one
                // group of eight rows ahead, so that a group does not begin with a trip to L2.
                const bool ahead = BIG && whole && p.epi == kEpiResid;
                const int n_res = ftile * kTileN + ec.lane_in_tile;
                float g_res = 0.f, hv_cur[8], hv_nxt[8];
                auto load_h = [&](int c0, float (&hv)[8]) {
#pragma unroll
                    for (int j = 0; j < 8; j++)
                        hv[j] = (c0 + j < ec.rows_live && n_res < p.n_out)
                                    ? __ldcg(p.h + (size_t)(ec.row_base + c0 + j) * p.n_out + n_res) : 0.f;
                };
                if (ahead) {
                    g_res = n_res < p.n_out ? __bfloat162float(p.gain_next[n_res]) : 0.f;
                    load_h(0, hv_cur);
                }
                for (int c0 = 0; c0 < rows_acc; c0 += 8) {
                    if (whole && c0 >= ec.rows_live) break;        // rows beyond the live ones: nothing to write
                    float hi[8], lo[8];
                    tmem_ld8(t_addr + c0, hi);
                    if (has_lo) tmem_ld8(t_addr + p.rh + c0, lo);
                    if (ahead) load_h(c0 + 8, hv_nxt);
                    tmem_ld_wait();
                    if (has_lo) {
#pragma unroll
                        for (int j = 0; j < 8; j++) hi[j] += lo[j];
                    }
                    if (whole) {
                        epi_store<8, BIG, MANY>(p, ec, ftile, c0, hi, ahead ? hv_cur : nullptr, ahead ? &g_res : nullptr);
                        if (ahead) {
#pragma unroll
                            for (int j = 0; j < 8; j++) hv_cur[j] = hv_nxt[j];
                        }
                    } else {
                        // partial slot layout [rh/4][feature] of float4 (four token rows of one feature): a warp
                        // stores and loads 512 contiguous bytes per instruction
                        float4* dst = reinterpret_cast<float4*>(my_slot) + (size_t)(c0 >> 2) * kTileN + ec.lane_in_tile;
                        dst[0] = make_float4(hi[0], hi[1], hi[2], hi[3]);
                        dst[kTileN] = make_float4(hi[4], hi[5], hi[6], hi[7]);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acce + 8 * buf);
                if (!whole) {
                    // Any other padding (1..8 rows, 17 and more): the last CTA to deliver its part of the tile sums all
                    // parts in k order.  The barrier orders every thread's partial stores before thread 0's
                    // acq_rel atomic (release is cumulative), and the loads after the second barrier behind
                    // its acquire.
                    epi_bar_g<MANY>(ge);
                    if (et == 0) {
                        if (TRACE && cp.test_stuck && oi == 0 && pc.index != 0) {
                            s_last = 0;             // test hook: this part is never announced, the tile never finishes
                        } else {
                            int prev;
                            asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;"
                                         : "=r"(prev) : "l"(p.tile_counters + pc.tile) : "memory");
                            s_last = (prev == pc.n_pieces - 1);
                            if (s_last) p.tile_counters[pc.tile] = 0;
                        }
                    }
                    epi_bar_g<MANY>(ge);
                    if (et == 0) PASS_TRACE(oi, 5);
                    if (s_last) {
                        tile_done = true;
                        const int c_first = cta - pc.index;
                        const int slot_first = pc.first_slot;
                        for (int c0 = 0; c0 < rows_acc; c0 += 8) {
                            float acc[8];
#pragma unroll
                            for (int j = 0; j < 8; j++) acc[j] = 0.f;
                            // parts are added in k order; loads go out eight parts at a time so that their
                            // latencies overlap
                            for (int q0 = 0; q0 < pc.n_pieces; q0 += 8) {
                                float4 v[8][2];
#pragma unroll
                                for (int qq = 0; qq < 8; qq++) {
                                    const int qi = min(q0 + qq, pc.n_pieces - 1);
                                    const int cq = c_first + qi;
                                    // every contributor but the first starts its own range inside this tile
                                    const int slot = qi == 0 ? slot_first : 0;
                                    const float4* src = reinterpret_cast<const float4*>(
                                        p.partial_ws + ((size_t)cq * 2 + slot) * slot_floats) + (size_t)(c0 >> 2) * kTileN + ec.lane_in_tile;
                                    v[qq][0] = __ldcg(src);
                                    v[qq][1] = __ldcg(src + kTileN);
                                }
#pragma unroll
                                for (int qq = 0; qq < 8; qq++) {
                                    if (q0 + qq < pc.n_pieces) {
                                        acc[0] += v[qq][0].x; acc[1] += v[qq][0].y; acc[2] += v[qq][0].z; acc[3] += v[qq][0].w;
                                        acc[4] += v[qq][1].x; acc[5] += v[qq][1].y; acc[6] += v[qq][1].z; acc[7] += v[qq][1].w;
                                    }
                                }
                            }
                            epi_store<8, BIG, MANY>(p, ec, pc.tile, c0, acc);
                        }
                    }
                }
                }
                if (et == 0 && ge == 0 && tile_done && !whole) PASS_TRACE(oi, 6);
                if ((signal || MANY) && tile_done) {
                    // every thread's stores of this tile happen-before thread 0's release (barrier + cumulativity);
                    // with two groups the barrier also keeps the reset below behind the other group's reads
                    epi_bar_all<MANY>();
                    if (signal && et == 0 && ge == 0)
                        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(cp.op_done + oi) : "memory");
                    if (et == 0 && ge == 0) PASS_TRACE(oi, 7);
                }
                if (ll_peer && ge == 0) ll_reset(ll_peer, 2 * slot_floats, ll_n, p.R);
            }
            if (et == 0 && ge == 0) *(volatile int*)&s_epi_done = oi;
            if (et == 0 && ge == 0) PASS_TRACE(oi, 3);
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (s_abort && threadIdx.x == 0) {
        // let every copy that was requested land before the shared memory is given back
        const int ia = *(volatile int*)&s_issued, ib = *(volatile int*)&s_issued_b;
        const int issued = ia < ib ? ia : ib;       // stages armed by both producers complete
        for (int f = issued - S < 0 ? 0 : issued - S; f < issued; f++) {
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_full + 8 * (f % S), (f / S) & 1))
                if (clock64() - t0 > kWaitCycles) break;
        }
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// (the compiler takes 132 registers of the 168 it may: 136 x 256 threads as allocated, beside the attention CTA's
// 232 x 128, are 64 512 of the SM's 65 536 - PASS_DBG_FOOTPRINT reports both and a test adds them up.  Capped at
// 136 it settles for 116 registers and a step 0.4 % slower.)
__global__ void __maxnreg__(168)
k_gemm_tc(const __grid_constant__ ChainMaps maps, const __grid_constant__ ChainParams cp) {
    gemm_chain_body<false, false, false>(maps, cp);
}
// the same with the %globaltimer stamps, the test hook that withholds partial sums and the held-back weight
// requests compiled in (template flag TRACE): kept out of the kernel above, whose step time follows its code
// size (3.00 -> 2.94 ms per nine-row step without the stamps alone)
__global__ void __maxnreg__(168)
k_gemm_tc_traced(const __grid_constant__ ChainMaps maps, const __grid_constant__ ChainParams cp) {
    gemm_chain_body<false, false, true>(maps, cp);
}
// Steps of ten token rows or more (k >= 5, batches): the many-row epilogue in place of the nine-row one, run by
// kEpiGroups groups of four warps (512 threads: the attention CTA no longer fits beside this one, which at these
// row counts costs less than the extra groups save).
constexpr int kGemmThreadsMany = 128 + kEpiGroups * 128;
__global__ void __launch_bounds__(kGemmThreadsMany, 1)
k_gemm_tc_many(const __grid_constant__ ChainMaps maps, const __grid_constant__ ChainParams cp) {
    gemm_chain_body<false, true, false>(maps, cp);
}
__global__ void __launch_bounds__(kGemmThreadsMany, 1)
k_gemm_tc_many_traced(const __grid_constant__ ChainMaps maps, const __grid_constant__ ChainParams cp) {
    gemm_chain_body<false, true, true>(maps, cp);
}
// prompt chunks: alone on its SM (192 KB of ring), so the register cap of the step's kernel does not apply
__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_tc_big(const __grid_constant__ ChainMaps maps, const __grid_constant__ ChainParams cp) {
    gemm_chain_body<true>(maps, cp);
}

}  // namespace pass
