// C-ABI entry points of the PaSS step library: context, workspace carving, the forward
// schedule, CUDA-graph capture of the step, and the host mirror of the sequence state.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <new>
#include <vector>

#include "attn_fd.cuh"
#include "gemm_tc.cuh"
#include "attn_tc.cuh"
#include "kernels_simt.cuh"
#include "kernels_verify.cuh"
#include "train.cuh"

using namespace pass;

namespace {

constexpr int kMaxCtas = 160;      // upper bound of CTAs of one GEMM launch (one per SM)
constexpr size_t kLLRegionBytes = (size_t)(kMaxCtas + 1) * 2 * kMaxRows * 128 * 4;   // per GEMM of a chain (rows per half up to 128); +1: CTA c reads c+1..

struct Carve {
    size_t off = 0;
    size_t take(size_t bytes) {
        const size_t o = off;
        off += (bytes + 255) & ~(size_t)255;
        return o;
    }
};

struct Layout {
    size_t states, params, unif, status, row_seq, row_pos, tok, cs, invfreq;
    size_t h, xn, qkv, attn, gu, act, logits;
    size_t E, chunk, row_sum, row_max, amax_val, amax_idx, q_logits, q_E, q_sum, scratch;
    size_t xn_bf, attn_bf, act_bf, q_out, sumsq_a, sumsq_b, partial_ws, counters;   // tensor-core path
    size_t ll_ws;
    size_t attn_po, attn_pml, attn_cnt, chain_flags;
    size_t packed, packed_bytes;       // the weights in streaming order (see k_pack_weight)
    size_t total;
};

// Bytes of one weight matrix [N][K] in the packed order: whole boxes of box_rows x 64 elements.
size_t packed_matrix_bytes(size_t N, size_t K, size_t box_rows) {
    return ((N + box_rows - 1) / box_rows) * ((K + 63) / 64) * box_rows * 128;
}

bool config_ok(const pass_config* c) {
    if (!c) return false;
    if (c->n_layers < 1 || c->d_model < 8 || c->n_heads < 1 || c->d_ffn < 8 || c->vocab < 2) return false;
    if (c->d_head != 64 && c->d_head != 128) return false;
    if ((long long)c->n_heads * c->d_head != c->d_model) return false;
    if (c->d_model % 8 || c->d_ffn % 8) return false;
    if (c->k_max < 1 || c->k_max > kMaxLA) return false;
    if (c->max_batch < 1 || c->max_batch > kMaxRows) return false;
    if (c->kv_capacity < 1) return false;
    if (c->dtype != PASS_DTYPE_FP32 && c->dtype != PASS_DTYPE_BF16) return false;
    if (!(c->rms_eps > 0.f) || !(c->rope_theta > 1.f)) return false;
    if (c->dtype == PASS_DTYPE_BF16 && c->d_model % 128) return false;
    return true;
}

size_t esize(int dtype) { return dtype == PASS_DTYPE_FP32 ? 4 : 2; }

Layout make_layout(const pass_config& c) {
    Layout L;
    Carve cv;
    const size_t R = kMaxRows, d = c.d_model, f = c.d_ffn, V = c.vocab, B = c.max_batch;
    // rows of one launch: a prompt chunk of a bf16 model has up to kRowsCap, everything else up to kMaxRows
    const size_t RC = c.dtype == PASS_DTYPE_BF16 ? kRowsCap : kMaxRows;
    L.states = cv.take(B * sizeof(SeqState));
    L.params = cv.take(sizeof(StepParams));
    L.unif = cv.take(B * kUSlots * sizeof(float));
    L.status = cv.take(sizeof(int));
    L.row_seq = cv.take(RC * sizeof(int));
    L.row_pos = cv.take(RC * sizeof(int));
    L.tok = cv.take(RC * sizeof(int));
    L.cs = cv.take(RC * (c.d_head / 2) * sizeof(float2));
    L.invfreq = cv.take((c.d_head / 2) * sizeof(double));
    L.h = cv.take(RC * d * 4);
    L.xn = cv.take(R * d * 4);
    L.qkv = cv.take(R * 3 * d * 4);
    L.attn = cv.take(R * d * 4);
    L.gu = cv.take(R * 2 * f * 4);
    L.act = cv.take(R * f * 4);
    L.logits = cv.take(R * V * 4);
    L.E = cv.take(R * V * 8);
    L.chunk = cv.take(R * kChunks * 8);
    L.row_sum = cv.take(R * kVerifySplits * 8);
    L.row_max = cv.take(R * 4);
    L.amax_val = cv.take(R * kVerifySplits * 4);
    L.amax_idx = cv.take(R * kVerifySplits * 4);
    L.q_logits = cv.take(B * 2 * c.k_max * V * 4);
    L.q_E = cv.take(B * 2 * c.k_max * V * 8);
    L.q_sum = cv.take(B * 2 * c.k_max * kVerifySplits * 8);
    L.scratch = cv.take(B * kChunks * 8);
    L.xn_bf = L.attn_bf = L.act_bf = L.q_out = L.sumsq_a = L.sumsq_b = L.partial_ws = L.counters = 0;
    L.attn_po = L.attn_pml = L.attn_cnt = L.chain_flags = 0;
    L.packed = L.packed_bytes = 0;
    if (c.dtype == PASS_DTYPE_BF16) {
        L.xn_bf = cv.take(RC * d * 2);           // kRowsCap plain rows, or hi rows + lo rows of a step
        L.attn_bf = cv.take(RC * d * 2);
        L.act_bf = cv.take(RC * f * 2);
        L.q_out = cv.take(RC * d * 4);
        L.sumsq_a = cv.take((d / 128 + 1) * RC * 4);
        L.sumsq_b = cv.take((d / 128 + 1) * RC * 4);
        L.partial_ws = cv.take((size_t)kMaxOps * kMaxCtas * 2 * R * kTileN * 4);
        L.counters = cv.take(4096 * 4);
        L.ll_ws = cv.take(kLLRegionBytes * kMaxOps);
        const size_t slices = 2 * kMaxCtas + B * c.n_heads;     // upper bound of B * heads * n_split
        L.attn_po = cv.take(slices * 32 * c.d_head * 4);
        L.attn_pml = cv.take(slices * 32 * 2 * 4);
        L.attn_cnt = cv.take(B * c.n_heads * 4);
        L.chain_flags = cv.take(2 * kMaxOps * 4);
        L.packed_bytes = (size_t)c.n_layers * (4 * packed_matrix_bytes(d, d, 128) + 2 * packed_matrix_bytes(f, d, 64) +
                                               packed_matrix_bytes(d, f, 128)) + packed_matrix_bytes(V, d, 128);
        L.packed = cv.take(L.packed_bytes);
    }
    L.total = cv.off;
    return L;
}

constexpr int kParamRing = 64;

}  // namespace

struct pass_ctx {
    pass_config cfg;
    ModelDims md;
    cudaStream_t stream;
    void *kv_k, *kv_v;
    char* ws;
    Layout L;
    // carved pointers
    SeqState* d_states;
    StepParams* d_params;
    float* d_unif;
    int *d_status, *d_row_seq, *d_row_pos, *d_tok;
    float2* d_cs;
    double* d_invfreq;
    float *d_h, *d_xn, *d_qkv, *d_attn, *d_gu, *d_act, *d_logits;
    VerifyBufs vb;
    double* d_scratch;
    // tensor-core path (bf16 models)
    __nv_bfloat16 *d_xn_bf = nullptr, *d_attn_bf = nullptr, *d_act_bf = nullptr;
    float *d_q_out = nullptr, *d_sumsq_a = nullptr, *d_sumsq_b = nullptr, *d_partial = nullptr;
    float* d_ll = nullptr;             // hand-over slots of the step's GEMMs (EMPTY-or-value words), all bits set when idle
    int* d_counters = nullptr;
    float *d_attn_po = nullptr, *d_attn_pml = nullptr;
    int* d_attn_cnt = nullptr;
    int n_sms = 148;
    bool use_pdl = true;
    bool attn_long = false;       // this step's contexts are long: twice as many attention slices (see step_launch)
    int attn_long_from = 3584;    // PASS_ATTN_LONG_FROM: cached positions from which a step counts as long
    bool attn_tc = true;          // PASS_ATTN_NO_TC: long contexts keep the mma.sync kernel (k_attn_tc otherwise, d_head 128, <= 16 rows)
    bool attn_tc_ready = false, attn_tc_smem_set = false;
    AttnTcMaps attn_tc_maps;      // the key and the value cache as matrices of 128 columns
    bool attn_cluster = true;     // PASS_ATTN_NO_CLUSTER: merge attention slices through global memory
    int attn_debug_stale = 0;     // pass_debug_set(PASS_HOOK_ATTN_STALE, n): attention's early part works from a cache length n short
    int attn_test_stuck = 0;      // pass_debug_set(PASS_HOOK_ATTN_STUCK, 1): k_attn_tc never announces its scores
    int gemm_test_stuck = 0;      // pass_debug_set(PASS_HOOK_GEMM_STUCK, 1): contributors withhold their partial sums
    // Function attributes and occupancy answers belong to the device the context lives on, so they are
    // remembered per context, never per process.
    size_t gemm_smem_set = 0, gemm_big_smem_set = 0, gemm_many_smem_set = 0, gemm_traced_smem_set = 0, gemm_many_traced_smem_set = 0;
    std::map<int, bool> attn_attr_set;         // by kernel instance
    std::map<int, int> attn_cluster_max;       // by kernel instance, slice count and sequences
    cudaError_t launch_err = cudaSuccess;      // first failed launch / attribute call since the last check
    bool use_tc = false;
    bool prompt_plain_bf16 = false;    // pass_set_prompt_precision: long prompts with plain bf16 activations
    // training of the look-ahead embeddings (pass_train_*): everything lives in the caller's training workspace
    struct Train {
        bool ready = false;
        pass_train_config hp;
        int L = 0, max_seqs = 0, step = 0, n_max = 0;
        char* ws = nullptr;
        std::vector<CUtensorMap> tm_qkv_t, tm_o_t, tm_gu_t, tm_d_t;     // transposed weights, packed
        CUtensorMap tm_lm_t;
        float *master = nullptr, *m = nullptr, *v = nullptr, *grad = nullptr;
        float *h_in = nullptr, *qkv = nullptr, *attn = nullptr, *h_mid = nullptr, *gu = nullptr;   // saved per layer
        float *h_last = nullptr, *dh = nullptr, *t0 = nullptr, *t1 = nullptr, *dlogits = nullptr, *loss_row = nullptr, *scratch = nullptr;
        int* targets = nullptr;
        __nv_bfloat16* stage = nullptr;                                 // hi | lo rows of a GEMM's input, any K
        std::map<std::pair<int, int>, CUtensorMap> stage_maps;          // by (K, npad)
        std::map<int, cudaGraphExec_t> graphs;                          // forward + backward over the look-ahead rows, by batch size
        int ng = 0;                                                     // columns of the interleaved gate|up output
        int* pin_targets = nullptr;
        float* pin_loss = nullptr;
    } tr;
    bool packed = false;               // the GEMMs stream the packed copy of the weights (PASS_NO_PACK: the caller's matrices)
    char* d_packed = nullptr;
    bool trace = false;                // PASS_TRACE=1: chain launches leave timestamps (see PASS_DBG_TRACE)
    int trace_launch = 0, attn_trace_launch = 0;
    int chain_done_total[kMaxOps] = {0, 0, 0, 0};   // host mirror of what the counters reach (see launch_chain)
    int* d_chain_flags = nullptr;      // [kMaxOps] tiles done per GEMM position of a chain, growing until the next clear
    std::vector<CUtensorMap> tm_wq, tm_wk, tm_wv, tm_wo, tm_wg, tm_wu, tm_wd;
    std::vector<CUtensorMap> tm_wg_plain, tm_wu_plain;   // 128-row boxes, for running gate or up alone
    CUtensorMap tm_lm;
    struct BMaps { CUtensorMap xn, attn, act; };
    std::map<int, BMaps> bmaps;        // by npad
    // weights
    bool weights_loaded = false;
    const void *tok_emb, *la_emb, *lm_head, *final_norm;
    std::vector<const void*> wq, wk, wv, wo, wg, wu, wd, norm_attn, norm_ffn;
    // host mirror
    std::vector<int> len_ub;
    std::vector<char> prefilled;
    bool have_last = false, params_on_device = false;
    int last_k = -1;
    int top_k = 0, last_top_k = 0;     // top-k sampling: 0 = off (pass_set_top_k)
    int validate_only = 0, dev_validate_only = 0;   // two-call schedule: the current call is a validation call
    bool force_drop = false;           // two-call schedule: the drafting call starts without pending drafts
    float last_T = -1.f;
    int dev_drop = 0;
    bool pending_collect = false;
    int last_rows = 0;
    // pinned staging
    StepParams* pin_params = nullptr;   // ring
    int ring_pos = 0;
    float* pin_unif = nullptr;
    SeqState* pin_states = nullptr;
    int* pin_status = nullptr;
    int* pin_tok = nullptr;
    // graphs
    std::map<int, cudaGraphExec_t> graphs;
    std::map<int, int> graph_launches;
    bool use_graph = true;
    int launches = 0, last_step_launches = 0;
};

#define CUDA_TRY(expr)                                                                     \
    do {                                                                                   \
        cudaError_t e_ = (expr);                                                           \
        if (e_ != cudaSuccess) {                                                           \
            if (getenv("PASS_LOG")) fprintf(stderr, "[pass] %s failed: %s (%s:%d)\n", #expr, \
                                            cudaGetErrorString(e_), __FILE__, __LINE__);   \
            return PASS_ERR_CUDA;                                                          \
        }                                                                                  \
    } while (0)

#define LAUNCH(ctx, kern, grid, block, ...)                           \
    do {                                                              \
        kern<<<(grid), (block), 0, (ctx)->stream>>>(__VA_ARGS__);     \
        (ctx)->launches++;                                            \
    } while (0)

// Launches and attribute calls made deep inside the enqueue helpers report here; the entry points
// turn the first recorded failure into PASS_ERR_CUDA (launch_failed) before they hand anything back.
static void note_err(pass_ctx* c, cudaError_t e, const char* what) {
    if (e == cudaSuccess) return;
    if (c->launch_err == cudaSuccess) c->launch_err = e;
    if (getenv("PASS_LOG")) fprintf(stderr, "[pass] %s failed: %s\n", what, cudaGetErrorString(e));
}
static bool launch_failed(pass_ctx* c) {
    const cudaError_t e = c->launch_err;
    c->launch_err = cudaSuccess;
    return e != cudaSuccess;
}
#define CHECK_LAUNCHES(ctx)                                   \
    do {                                                      \
        if (launch_failed(ctx)) return PASS_ERR_CUDA;         \
        CUDA_TRY(cudaGetLastError());                         \
    } while (0)

// ------------------------------------------------------------------------------- small kernels
__global__ void k_update_state(SeqState* states, int seq, int set_len, int len, int add_len,
                               int set_pending, int pending, int clear_all) {
    SeqState& st = states[seq];
    if (clear_all) {
        st.kv_len = 0; st.pending = 0; st.has_pending = 0; st.m = 0; st.q_sel = 0;
        st.n_out = 0; st.n_acc = 0;
    }
    if (set_len) st.kv_len = len;
    st.kv_len += add_len;
    if (set_pending) { st.pending = pending; st.has_pending = 1; }
    st.m = 0;
}

// Between the caller's [n][d_model] layout and the cache's [head][position][d_head].
template <typename KVT>
__global__ void k_kv_scatter(const KVT* __restrict__ src, ModelDims md, int layer, int seq, int pos0,
                             int n, KVT* __restrict__ cache, int gather) {
    const size_t total = (size_t)n * md.d;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x) {
        const int p = (int)(i / md.d), c = (int)(i % md.d);
        const size_t o = kv_index(md, layer, seq, c / md.dh, pos0 + p) + c % md.dh;
        if (gather) const_cast<KVT*>(src)[i] = cache[o];
        else cache[o] = src[i];
    }
}

// ------------------------------------------------------------------------------- tensor-core path (host)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 matrix [rows][cols] row-major; box = 64 columns (128 bytes, 128B swizzle) x box_rows rows.
static bool make_map(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBlockK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The packed copy of a matrix as a tensor map: n_boxes boxes of box_rows x 64 elements, one after another.
static bool make_map_packed(CUtensorMap* m, const void* base, uint64_t n_boxes, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)kBlockK, n_boxes * box_rows};
    const cuuint64_t strides[1] = {(cuuint64_t)kBlockK * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBlockK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Token rows are padded to a multiple of 8 per half (hi | lo).  Up to 16 rows always take 16 per half: that is
// the padding with the counter-free hand-over of partial sums (see k_gemm_tc), and a one-row step is then as
// fast as a nine-row one (3.10 -> 3.06 ms at the 7B shape) for 2 KB more activation bytes per stage.
// From this many token rows on a step's GEMMs run in k_gemm_tc_many: the passes of eight rows through the epilogue
// are shared by three groups of warps, which beats the nine-row passes of one group from two passes on (k >= 5:
// 3.55 -> 3.46 ms at 13 rows) although the attention CTA no longer fits beside the GEMM CTA.
constexpr int kManyRowsFrom = 10;
static int npad_for(int R) { return R <= 16 ? 32 : ((2 * R + 15) / 16) * 16; }

static int gemm_stages(int npad) {
    const int stage = kATileBytes + npad * 128;
    if (const char* e = getenv("PASS_GEMM_STAGES")) {
        const int s = atoi(e);
        if (s >= 2 && s <= 16 && (size_t)s * stage + 1024 <= 225 * 1024) return s;
    }
    // up to 16 padded rows per half: the step's kernel, which leaves room for one attention CTA (ring of two stages:
    // 64 KB) beside it; more: kernels that have the SM to themselves
    // (measured: more than eight stages make the hand-overs slower again - k = 8: 3.460 / 3.480 ms with 8 / 9)
    int s = npad > 32 ? std::min(8, (206 * 1024 - 1024) / stage) : (142 * 1024 - 1024) / stage;
    if (s < 4) s = std::min(4, (220 * 1024) / stage);
    return std::max(2, std::min(16, s));
}

static const pass_ctx::BMaps* get_bmaps(pass_ctx* c, int npad) {
    auto it = c->bmaps.find(npad);
    if (it != c->bmaps.end()) return &it->second;
    pass_ctx::BMaps bm;
    if (!make_map(&bm.xn, c->d_xn_bf, kRowsCap, c->md.d, npad)) return nullptr;
    if (!make_map(&bm.attn, c->d_attn_bf, kRowsCap, c->md.d, npad)) return nullptr;
    if (!make_map(&bm.act, c->d_act_bf, kRowsCap, c->md.f, npad)) return nullptr;
    return &(c->bmaps[npad] = bm);
}

static GemmParams gemm_base(pass_ctx* c, int R, int npad, int K, int n_tiles, int n_out, int epi) {
    GemmParams p;
    memset(&p, 0, sizeof(p));
    p.n_tiles = n_tiles;
    p.kb_per_tile = (K + kBlockK - 1) / kBlockK;
    p.seg_tiles0 = p.seg_tiles1 = 1 << 30;
    p.npad = npad;
    p.rh = npad / 2;
    p.R = R;
    p.stages = gemm_stages(npad);
    p.epi = epi;
    p.n_out = n_out;
    p.partial_ws = c->d_partial;
    p.ll_ws = c->d_ll;
    p.tile_counters = c->d_counters;
    p.status = c->d_status;
    p.eps = c->md.eps;
    p.md = c->md;
    p.xn_lo_row0 = npad / 2;
    p.packed = c->packed ? 1 : 0;
    p.has_lo = 1;
    return p;
}

// One GEMM of a chain with its four tensor maps (weights 0..2, activations).
struct ChainOp {
    GemmParams p;
    CUtensorMap a0, a1, a2, b;
};

// The tail of the verify scratch (E, [kMaxRows][V] doubles) doubles as the trace buffer: its rows beyond the
// first half are only used by steps of more than 64 rows.  nullptr when E is too small for that.
constexpr int kTraceLaunches = 48;
constexpr size_t kAttnTraceWords = 2048;     // per k_attn_tc launch: [64 heads / 4][16 slices][8 stamps]
static unsigned long long* trace_base(pass_ctx* c) {
    const size_t total = (size_t)kMaxRows * c->md.V;
    const size_t need = (size_t)kTraceLaunches * (kMaxOps * kMaxCtas * 8 + kAttnTraceWords);
    if (need > total / 2) return nullptr;
    return (unsigned long long*)c->vb.E + (total - (size_t)kTraceLaunches * kMaxOps * kMaxCtas * 8);
}
// the long-cache attention kernel's stamps sit in front of the GEMM chain's
static unsigned long long* attn_trace_base(pass_ctx* c) {
    return trace_base(c) ? trace_base(c) - (size_t)kTraceLaunches * kAttnTraceWords : nullptr;
}

// Launch up to kMaxOps dependent GEMMs as ONE kernel (see k_gemm_tc).  GEMM j of the chain gets its own
// partial-sum region and tile counters, because its split tiles may be in flight while GEMM j-1 is
// still being reduced.
static void launch_chain(pass_ctx* c, ChainOp* ops, int n_ops) {
    ChainMaps maps;
    ChainParams cp;
    memset(&cp, 0, sizeof(cp));
    cp.n_ops = n_ops;
    cp.stages = ops[0].p.stages;
    cp.npad = ops[0].p.npad;
    cp.test_stuck = c->gemm_test_stuck;
    cp.hold = getenv("PASS_GEMM_HOLD") ? atoi(getenv("PASS_GEMM_HOLD")) : 0;
    cp.op_done = c->d_chain_flags;
    for (int j = 0; j < kMaxOps; j++) {
        // counters only grow between two clears: each launch waits for the totals that include its own tiles,
        // so nobody has to count the CTAs out and clear them at the end of a launch
        if (j + 1 < n_ops) c->chain_done_total[j] += ops[j].p.n_tiles;      // the last GEMM of a launch signals nobody
        cp.op_target[j] = c->chain_done_total[j];
    }
    cp.status = c->d_status;
    if (c->trace && c->trace_launch < kTraceLaunches && trace_base(c))
        cp.trace = trace_base(c) + (size_t)(c->trace_launch++) * kMaxOps * kMaxCtas * 8;
    const size_t region = (size_t)kMaxCtas * 2 * kMaxRows * kTileN;      // floats per GEMM of the chain
    for (int j = 0; j < n_ops; j++) {
        if (ops[j].p.partial_ws == c->d_partial) {
            ops[j].p.partial_ws = c->d_partial + (size_t)j * region;
            ops[j].p.ll_ws = c->d_ll + (size_t)j * (kLLRegionBytes / 4);
            ops[j].p.tile_counters = c->d_counters + j * 1024;
        }
        cp.op[j] = ops[j].p;
        maps.m[j][0] = ops[j].a0; maps.m[j][1] = ops[j].a1; maps.m[j][2] = ops[j].a2; maps.m[j][3] = ops[j].b;
    }
    for (int j = n_ops; j < kMaxOps; j++)
        for (int q = 0; q < 4; q++) maps.m[j][q] = ops[0].a0;
    const size_t smem = (size_t)cp.stages * (kATileBytes + cp.npad * 128) + 1024;
    const bool big = ops[0].p.whole_only != 0;        // a prompt chunk: the kernel instance with token tiles
    const bool many = !big && ops[0].p.R >= kManyRowsFrom;        // the instance with several epilogue groups
    bool dbg = c->trace || cp.test_stuck || cp.hold;      // stamps, test hook, held-back requests: the instance that has them
    // ... and the schedule arithmetic for CTAs with more pieces than the kernel keeps in shared memory
    for (int j = 0; j < n_ops; j++) dbg |= ops[j].p.n_tiles / c->n_sms + 2 > kPieceCache;
    auto kern = big ? k_gemm_tc_big : many ? (dbg ? k_gemm_tc_many_traced : k_gemm_tc_many) : dbg ? k_gemm_tc_traced : k_gemm_tc;
    size_t& smem_set = big ? c->gemm_big_smem_set : many ? (dbg ? c->gemm_many_traced_smem_set : c->gemm_many_smem_set) : dbg ? c->gemm_traced_smem_set : c->gemm_smem_set;
    if (smem > smem_set) {
        note_err(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem), "k_gemm_tc shared memory size");
        // all of the SM's L1/shared storage as shared memory: lets the CTA of the next launch become
        // resident (and start pulling weights) while this launch's CTA is still running
        note_err(c, cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 100), "k_gemm_tc carveout");
        smem_set = smem;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    long long units = 0;
    for (int j = 0; j < n_ops; j++) units = std::max(units, (long long)ops[j].p.n_tiles * ops[j].p.kb_per_tile);
    // a chain needs every CTA resident at once (they wait for one another's tiles): one CTA per SM
    cfg.gridDim = dim3((unsigned)std::min<long long>(c->n_sms, units));
    cfg.blockDim = dim3(many ? kGemmThreadsMany : kGemmThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = c->stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = c->use_pdl ? 1 : 0;
    note_err(c, cudaLaunchKernelEx(&cfg, kern, maps, cp), "k_gemm_tc launch");
    c->launches++;
}

// Start of a forward: the chain's completion counters go back to zero (on the device, in stream order, and
// in the host's mirror).  Also what makes the next forward right after one that was abandoned on a time-out.
static void chain_counters_clear(pass_ctx* c) {
    note_err(c, cudaMemsetAsync(c->d_chain_flags, 0, sizeof(int) * kMaxOps, c->stream), "chain counter clear");
    for (int j = 0; j < kMaxOps; j++) c->chain_done_total[j] = 0;
}

static void launch_gemm(pass_ctx* c, const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& a2,
                        const CUtensorMap& b, const GemmParams& p) {
    ChainOp op;
    op.p = p; op.a0 = a0; op.a1 = a1; op.a2 = a2; op.b = b;
    launch_chain(c, &op, 1);
}

// The bf16 decoder layers on tensor cores.  Per layer: QKV GEMM (+RMSNorm factor, rotary, KV append),
// attention, O GEMM (+residual, next norm's input), gate/up GEMM (+SwiGLU), down GEMM (+residual).
template <int DH, int MT, bool CL, int ST, int NREG>
static void launch_attn_fd_impl(pass_ctx* c, const AttnParams& ap, int n_seq) {
    constexpr int smem = 2 * ST * kAttnBK * DH * 2;
    bool& set = c->attn_attr_set[NREG * 65536 + ST * 4096 + DH * 8 + MT * 2 + (CL ? 1 : 0)];
    if (!set) {
        note_err(c, cudaFuncSetAttribute(k_attn_fd<DH, MT, CL, true, false, ST, NREG>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem), "k_attn_fd shared memory size");
        note_err(c, cudaFuncSetAttribute(k_attn_fd<DH, MT, CL, true, false, ST, NREG>, cudaFuncAttributePreferredSharedMemoryCarveout, 100), "k_attn_fd carveout");
        set = true;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(c->md.H, n_seq, ap.n_split);
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = c->stream;
    cudaLaunchAttribute at[2];
    int na = 0;
    if (CL) {
        at[na].id = cudaLaunchAttributeClusterDimension;
        at[na].val.clusterDim.x = 1; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = ap.n_split;
        na++;
    }
    if (c->use_pdl) {
        at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[na].val.programmaticStreamSerializationAllowed = 1;
        na++;
    }
    cfg.attrs = at;
    cfg.numAttrs = na;
    note_err(c, cudaLaunchKernelEx(&cfg, k_attn_fd<DH, MT, CL, true, false, ST, NREG>, ap), "k_attn_fd launch");
    c->launches++;
}

// Long caches, d_head 128, at most 16 rows per sequence: scores on tcgen05 (attn_tc.cuh), one CTA per SM.
static void launch_attn_tc(pass_ctx* c, const AttnParams& ap_in, int n_seq) {
    AttnParams ap = ap_in;
    ap.trace = nullptr;
    if (c->trace && c->attn_trace_launch < kTraceLaunches && attn_trace_base(c) && c->md.H <= 64 && n_seq == 1)
        ap.trace = attn_trace_base(c) + (size_t)(c->attn_trace_launch++) * kAttnTraceWords;
    if (!c->attn_tc_smem_set) {
        note_err(c, cudaFuncSetAttribute(k_attn_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem), "k_attn_tc shared memory size");
        c->attn_tc_smem_set = true;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(c->md.H, n_seq, ap.n_split);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = kTcSmem;
    cfg.stream = c->stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = c->use_pdl ? 1 : 0;
    note_err(c, cudaLaunchKernelEx(&cfg, k_attn_tc, c->attn_tc_maps, ap), "k_attn_tc launch");
    c->launches++;
}

// Can the slices of every (sequence, head) run as one cluster each, all at the same time?  Asked once per
// context, kernel instance, slice count and batch; if not (or with more than 8 slices) the merge goes through
// global memory.
template <int DH, int MT, int ST, int NREG>
static bool attn_cluster_ok(pass_ctx* c, int n_split, int n_seq) {
    if (!c->attn_cluster || n_split < 2 || n_split > 8) return false;
    const int key = ((((NREG / 64) * 4 + ST) * 256 + DH) * 8 + MT) * 32 * 256 + n_split * 256 + n_seq;
    auto it = c->attn_cluster_max.find(key);
    if (it == c->attn_cluster_max.end()) {
        constexpr int smem = 2 * ST * kAttnBK * DH * 2;
        note_err(c, cudaFuncSetAttribute(k_attn_fd<DH, MT, true, true, false, ST, NREG>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem), "k_attn_fd shared memory size");
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3(c->md.H, n_seq, n_split);
        cfg.blockDim = dim3(128);
        cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = n_split;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, k_attn_fd<DH, MT, true, true, false, ST, NREG>, &cfg) != cudaSuccess) { n = 0; cudaGetLastError(); }
        it = c->attn_cluster_max.emplace(key, n).first;
    }
    return it->second >= c->md.H * n_seq;
}

template <int DH, int MT, int ST, int NREG>
static void launch_attn_fd(pass_ctx* c, const AttnParams& ap, int n_seq) {
    if (attn_cluster_ok<DH, MT, ST, NREG>(c, ap.n_split, n_seq)) launch_attn_fd_impl<DH, MT, true, ST, NREG>(c, ap, n_seq);
    else launch_attn_fd_impl<DH, MT, false, ST, NREG>(c, ap, n_seq);
}

// GEMMs of the decoder layers as chain entries.
// Prompt chunks (big): the rows are plain bf16, cut into token tiles of 256 rows; every (feature tile, token
// tile) unit is computed whole by one CTA.
static void set_big(pass_ctx* c, GemmParams& p, int R, int feat_tiles) {
    p.has_lo = c->prompt_plain_bf16 ? 0 : 1;
    p.whole_only = 1;
    const int tile_tokens = p.has_lo ? kTokTile / 2 : kTokTile;     // hi | lo rows: 128 tokens fill the MMA's 256 columns
    p.n_tok_tiles = (R + tile_tokens - 1) / tile_tokens;
    p.n_tiles = feat_tiles * p.n_tok_tiles;
}
static ChainOp op_qkv(pass_ctx* c, int R, int npad, const pass_ctx::BMaps* bm, int l, bool big) {
    typedef __nv_bfloat16 bf;
    const int d = c->md.d, dt = d / kTileN;
    ChainOp o;
    o.p = gemm_base(c, R, npad, d, 3 * dt, 3 * d, kEpiQKV);
    o.p.seg_tiles0 = o.p.seg_tiles1 = dt;
    o.p.sumsq_in = c->d_sumsq_a; o.p.n_parts_in = dt; o.p.inv_d_in = 1.f / d;
    o.p.q_out = c->d_q_out; o.p.rope_cs = c->d_cs; o.p.row_seq = c->d_row_seq; o.p.row_pos = c->d_row_pos;
    o.p.layer = l; o.p.kc = (bf*)c->kv_k; o.p.vc = (bf*)c->kv_v;
    o.a0 = c->tm_wq[l]; o.a1 = c->tm_wk[l]; o.a2 = c->tm_wv[l]; o.b = bm->xn;
    if (big) set_big(c, o.p, R, 3 * dt);
    return o;
}
// O-projection -> gate|up -> down of layer l, then the next layer's QKV, or the output head (head = true)
// after the last layer, or nothing.  Returns the number of entries written.
static int build_layer_chain(pass_ctx* c, int R, int npad, const pass_ctx::BMaps* bm, int l, bool head, ChainOp* ch,
                             bool big = false) {
    typedef __nv_bfloat16 bf;
    const ModelDims& md = c->md;
    const int d = md.d, f = md.f, dt = d / kTileN;
    int n = 0;
    {   // attention output projection + residual; prepares the input of the feed-forward norm
        ChainOp& o = ch[n++];
        o.p = gemm_base(c, R, npad, d, dt, d, kEpiResid);
        o.p.h = c->d_h; o.p.gain_next = (const bf*)c->norm_ffn[l]; o.p.xn_out = c->d_xn_bf; o.p.sumsq_out = c->d_sumsq_b;
        o.a0 = o.a1 = o.a2 = c->tm_wo[l]; o.b = bm->attn;
        if (big) set_big(c, o.p, R, dt);
    }
    {   // gate | up, interleaved by 64 rows, SwiGLU in the epilogue
        ChainOp& o = ch[n++];
        o.p = gemm_base(c, R, npad, d, (f + 63) / 64, f, kEpiSwiGLU);
        o.p.interleave = 1;
        o.p.sumsq_in = c->d_sumsq_b; o.p.n_parts_in = dt; o.p.inv_d_in = 1.f / d;
        o.p.act_out = c->d_act_bf;
        o.a0 = c->tm_wg[l]; o.a1 = o.a2 = c->tm_wu[l]; o.b = bm->xn;
        if (big) set_big(c, o.p, R, (f + 63) / 64);
    }
    {   // down projection + residual; prepares the input of the next norm
        ChainOp& o = ch[n++];
        o.p = gemm_base(c, R, npad, f, dt, d, kEpiResid);
        o.p.h = c->d_h;
        o.p.gain_next = (const bf*)(l + 1 < md.n_layers ? c->norm_attn[l + 1] : c->final_norm);
        o.p.xn_out = c->d_xn_bf; o.p.sumsq_out = c->d_sumsq_a;
        o.a0 = o.a1 = o.a2 = c->tm_wd[l]; o.b = bm->act;
        if (big) set_big(c, o.p, R, dt);
    }
    if (l + 1 < md.n_layers) {
        ch[n++] = op_qkv(c, R, npad, bm, l + 1, big);
    } else if (head) {
        ChainOp& o = ch[n++];
        o.p = gemm_base(c, R, npad, d, (md.V + kTileN - 1) / kTileN, md.V, kEpiLogits);
        o.p.sumsq_in = c->d_sumsq_a; o.p.n_parts_in = dt; o.p.inv_d_in = 1.f / d;
        o.p.logits = c->d_logits;
        o.a0 = o.a1 = o.a2 = c->tm_lm; o.b = bm->xn;
        if (big) set_big(c, o.p, R, (md.V + kTileN - 1) / kTileN);
    }
    return n;
}

static void launch_ops(pass_ctx* c, ChainOp* ch, int n) {
    if (getenv("PASS_NO_CHAIN")) for (int j = 0; j < n; j++) launch_chain(c, ch + j, 1);
    else launch_chain(c, ch, n);
}

// Rows of ONE sequence as a prompt chunk: causal flash attention, a CTA per head and block of 64 rows.
template <int DH, bool HL>
static void launch_attn_chunk(pass_ctx* c, AttnParams ap) {
    ap.n_split = 1;
    ap.rows_per_block = 64;
    constexpr int smem = 2 * kAttnStages * kAttnBK * DH * 2;
    bool& set = c->attn_attr_set[DH * 8 + 4 * 2 + (HL ? 64 : 32)];
    if (!set) {
        note_err(c, cudaFuncSetAttribute(k_attn_fd<DH, 4, false, HL, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem), "k_attn_fd shared memory size");
        set = true;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(c->md.H, (ap.M + 63) / 64, 1);
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = c->stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = c->use_pdl ? 1 : 0;
    note_err(c, cudaLaunchKernelEx(&cfg, k_attn_fd<DH, 4, false, HL, true>, ap), "k_attn_fd (chunk) launch");
    c->launches++;
}

// R rows = n_seq sequences x M rows each (M = R when n_seq == 1).
// input_ready: the rotary table and the first layer's norm input have been produced already (k_step_input).
// big: a prompt chunk of up to kRowsCap rows of one sequence in plain bf16 (see set_big).
static int enqueue_layers_tc(pass_ctx* c, int R, int n_seq, bool head, bool input_ready = false, bool big = false) {
    const ModelDims& md = c->md;
    const int d = md.d, npad = big ? kTokTile : npad_for(R), rh = npad / 2;
    const pass_ctx::BMaps* bm = get_bmaps(c, npad);
    if (!bm) return PASS_ERR_CUDA;
    typedef __nv_bfloat16 bf;
    chain_counters_clear(c);
    if (!input_ready) {
        LAUNCH(c, k_rope_table, R, 64, c->d_row_pos, c->d_invfreq, md.dh / 2, c->d_cs);
        const bool plain = big && c->prompt_plain_bf16;
        LAUNCH(c, k_split_norm_input, R, 128, c->d_h, (const bf*)c->norm_attn[0], d, c->d_xn_bf, plain ? -1 : rh, c->d_sumsq_a,
               big && !plain ? rh : 0);
    }
    ChainOp chain[kMaxOps];
    // Kernels of a step: QKV_0 | per layer: attention, then ONE launch running
    // O-projection -> gate|up -> down -> (next layer's QKV, or the output head after the last layer).
    chain[0] = op_qkv(c, R, npad, bm, 0, big);
    launch_ops(c, chain, 1);
    for (int l = 0; l < md.n_layers; l++) {
        const int M = R / n_seq;
        AttnParams ap;
        ap.q = c->d_q_out; ap.ldq = d; ap.row_seq = c->d_row_seq; ap.row_pos = c->d_row_pos; ap.md = md;
        ap.layer = l; ap.kc = (const bf*)c->kv_k; ap.vc = (const bf*)c->kv_v; ap.M = M;
        ap.part_o = c->d_attn_po; ap.part_ml = c->d_attn_pml; ap.counters = c->d_attn_cnt;
        const bool plain = big && c->prompt_plain_bf16;
        ap.out = c->d_attn_bf; ap.lo_row0 = plain ? -1 : rh; ap.debug_stale = c->attn_debug_stale;
        ap.rows_per_block = 0;
        ap.status = c->d_status;
        ap.debug_stuck = c->attn_test_stuck;
        ap.out_tile_rows = big && !plain ? rh : 0;
        if (M <= 16 && md.dh == kTcDH && c->attn_long && c->attn_tc && c->attn_tc_ready) {
            ap.n_split = std::max(1, std::min(kAttnMaxSplit, c->n_sms / (md.H * n_seq)));
            launch_attn_tc(c, ap, n_seq);
        } else if (M <= 32 && R >= kManyRowsFrom) {
            // A step of ten rows or more: its GEMM kernel (k_gemm_tc_many) leaves no room for an attention CTA on its
            // SM, so the attention kernel has the SMs to itself: a ring of two stages (64 KB at d_head 128), three
            // CTAs per SM, and as many slices per (sequence, head) pair as fill those (at most 8, a cluster's worth).
            const int pairs = md.H * n_seq;
            ap.n_split = std::max(1, std::min(8, 3 * c->n_sms / pairs));
            ap.n_split = std::min(ap.n_split, (2 * kMaxCtas + pairs) / pairs);      // what the slices' workspace holds
            if (md.dh == 128) { if (M <= 16) launch_attn_fd<128, 1, 2, 168>(c, ap, n_seq); else launch_attn_fd<128, 2, 2, 168>(c, ap, n_seq); }
            else              { if (M <= 16) launch_attn_fd<64, 1, 2, 168>(c, ap, n_seq); else launch_attn_fd<64, 2, 2, 168>(c, ap, n_seq); }
        } else if (M <= 32) {
            // at most one CTA per SM: the next GEMM's CTA then fits beside it and prefetches weights
            ap.n_split = std::max(1, std::min(kAttnMaxSplit, c->n_sms / (md.H * n_seq)));
            // Long contexts: the key loop (tensor-core work of 4 warps) outweighs everything that one CTA per
            // SM buys at short contexts, so the slices are doubled - two CTAs per SM, 8 warps on the keys.
            // (at most nine rows here: one 16-row tile)
            if (c->attn_long && ap.n_split * 2 <= 8) {
                ap.n_split *= 2;
                if (md.dh == 128) launch_attn_fd<128, 1, 3, 232>(c, ap, n_seq); else launch_attn_fd<64, 1, 3, 232>(c, ap, n_seq);
            } else {
                if (md.dh == 128) launch_attn_fd<128, 1, 2, 232>(c, ap, n_seq); else launch_attn_fd<64, 1, 2, 232>(c, ap, n_seq);
            }
        } else {
            // more than 32 rows: one sequence's prompt chunk (pass_forward_tokens, pass_prefill)
            ap.debug_stale = 0;
            if (md.dh == 128) { if (plain) launch_attn_chunk<128, false>(c, ap); else launch_attn_chunk<128, true>(c, ap); }
            else              { if (plain) launch_attn_chunk<64, false>(c, ap); else launch_attn_chunk<64, true>(c, ap); }
        }
        launch_ops(c, chain, build_layer_chain(c, R, npad, bm, l, head, chain, big));
    }
    return PASS_OK;
}

// ------------------------------------------------------------------------------- forward
template <typename WT>
static void enqueue_layers(pass_ctx* c, int R) {
    const ModelDims& md = c->md;
    const int d = md.d, f = md.f;
    const WT* dummy = nullptr;
    (void)dummy;
    LAUNCH(c, k_rope_table, R, 64, c->d_row_pos, c->d_invfreq, md.dh / 2, c->d_cs);
    const int gw = 8;   // warps (features) per GEMM block
    for (int l = 0; l < md.n_layers; l++) {
        LAUNCH(c, (k_rmsnorm<WT>), R, 256, c->d_h, (const WT*)c->norm_attn[l], d, md.eps, c->d_xn);
        LAUNCH(c, (k_gemm_simt<WT, 16>), (d + gw - 1) / gw, gw * 32, c->d_xn, d, (const WT*)c->wq[l], d, d, R, c->d_qkv, 3 * d, 0);
        LAUNCH(c, (k_gemm_simt<WT, 16>), (d + gw - 1) / gw, gw * 32, c->d_xn, d, (const WT*)c->wk[l], d, d, R, c->d_qkv + d, 3 * d, 0);
        LAUNCH(c, (k_gemm_simt<WT, 16>), (d + gw - 1) / gw, gw * 32, c->d_xn, d, (const WT*)c->wv[l], d, d, R, c->d_qkv + 2 * d, 3 * d, 0);
        LAUNCH(c, (k_rope_kv<WT>), R, 256, c->d_qkv, c->d_cs, c->d_row_seq, c->d_row_pos, md, l, (WT*)c->kv_k, (WT*)c->kv_v);
        if (md.dh == 128)
            LAUNCH(c, (k_attn_simple<WT, 128, false>), dim3(md.H, R), 128, c->d_qkv, 3 * d, c->d_row_seq, c->d_row_pos, md, l, (const WT*)c->kv_k, (const WT*)c->kv_v, (void*)c->d_attn, 0);
        else
            LAUNCH(c, (k_attn_simple<WT, 64, false>), dim3(md.H, R), 128, c->d_qkv, 3 * d, c->d_row_seq, c->d_row_pos, md, l, (const WT*)c->kv_k, (const WT*)c->kv_v, (void*)c->d_attn, 0);
        LAUNCH(c, (k_gemm_simt<WT, 16>), (d + gw - 1) / gw, gw * 32, c->d_attn, d, (const WT*)c->wo[l], d, d, R, c->d_h, d, 1);
        LAUNCH(c, (k_rmsnorm<WT>), R, 256, c->d_h, (const WT*)c->norm_ffn[l], d, md.eps, c->d_xn);
        LAUNCH(c, (k_gemm_simt<WT, 16>), (f + gw - 1) / gw, gw * 32, c->d_xn, d, (const WT*)c->wg[l], f, d, R, c->d_gu, 2 * f, 0);
        LAUNCH(c, (k_gemm_simt<WT, 16>), (f + gw - 1) / gw, gw * 32, c->d_xn, d, (const WT*)c->wu[l], f, d, R, c->d_gu + f, 2 * f, 0);
        LAUNCH(c, k_swiglu, dim3((f + 255) / 256, R), 256, c->d_gu, f, c->d_act);
        LAUNCH(c, (k_gemm_simt<WT, 16>), (d + gw - 1) / gw, gw * 32, c->d_act, f, (const WT*)c->wd[l], d, f, R, c->d_h, d, 1);
    }
}

template <typename WT>
static void enqueue_head(pass_ctx* c, int R) {
    const ModelDims& md = c->md;
    const int gw = 8;
    LAUNCH(c, (k_rmsnorm<WT>), R, 256, c->d_h, (const WT*)c->final_norm, md.d, md.eps, c->d_xn);
    LAUNCH(c, (k_gemm_simt<WT, 16>), (md.V + gw - 1) / gw, gw * 32, c->d_xn, md.d, (const WT*)c->lm_head, md.V, md.d, R, c->d_logits, md.V, 0);
}

template <typename WT>
static void enqueue_step(pass_ctx* c, int k) {
    const ModelDims& md = c->md;
    const int M = 1 + 2 * k, R = md.B * M;
    if (c->use_tc) {
        typedef __nv_bfloat16 bf;
        LAUNCH(c, k_step_input, dim3(R, (md.d + 1023) / 1024), 256, (const bf*)c->tok_emb, (const bf*)c->la_emb,
               c->d_states, c->d_params, M, md.d, md.V, c->d_h, c->d_row_seq, c->d_row_pos, c->d_invfreq, md.dh / 2,
               c->d_cs, (const bf*)c->norm_attn[0], c->d_xn_bf, npad_for(R) / 2, c->d_sumsq_a);
        enqueue_layers_tc(c, R, md.B, true, true);
    } else {
        LAUNCH(c, (k_assemble_step<WT>), R, 256, (const WT*)c->tok_emb, (const WT*)c->la_emb, c->d_states,
               c->d_params, M, md.d, md.V, c->d_h, c->d_row_seq, c->d_row_pos);
        enqueue_layers<WT>(c, R);
        enqueue_head<WT>(c, R);
    }
    LAUNCH(c, k_verify_stats, dim3(R, kVerifySplits), kVerifyThreads, c->vb, c->d_states, c->d_params, M, md.V, md.k_max);
    LAUNCH(c, k_verify_decide, md.B, 1024, c->vb, c->d_states, c->d_params, c->d_unif, M, md.V, md.k_max, c->d_scratch);
}

static void enqueue_step_any(pass_ctx* c, int k) {
    if (c->md.dtype == PASS_DTYPE_FP32) enqueue_step<float>(c, k);
    else enqueue_step<__nv_bfloat16>(c, k);
}

// big: a prompt chunk of more than kMaxRows rows of a bf16 model on the tensor-core path (plain bf16 rows).
static int run_tokens(pass_ctx* c, int seq, const int32_t* tokens, int n, bool want_logits, bool big = false) {
    memcpy(c->pin_tok, tokens, sizeof(int) * n);
    CUDA_TRY(cudaMemcpyAsync(c->d_tok, c->pin_tok, sizeof(int) * n, cudaMemcpyHostToDevice, c->stream));
    if (c->md.dtype == PASS_DTYPE_FP32) {
        LAUNCH(c, (k_assemble_tokens<float>), n, 256, (const float*)c->tok_emb, (const float*)c->la_emb,
               c->d_states, c->d_tok, seq, c->md.d, c->md.V, c->d_h, c->d_row_seq, c->d_row_pos);
        enqueue_layers<float>(c, n);
        if (want_logits) enqueue_head<float>(c, n);
    } else {
        LAUNCH(c, (k_assemble_tokens<__nv_bfloat16>), n, 256, (const __nv_bfloat16*)c->tok_emb,
               (const __nv_bfloat16*)c->la_emb, c->d_states, c->d_tok, seq, c->md.d, c->md.V, c->d_h,
               c->d_row_seq, c->d_row_pos);
        if (c->use_tc) {
            const int rc = enqueue_layers_tc(c, n, 1, want_logits, false, big);
            if (rc != PASS_OK) return rc;
        } else {
            enqueue_layers<__nv_bfloat16>(c, n);
            if (want_logits) enqueue_head<__nv_bfloat16>(c, n);
        }
    }
    c->last_rows = n;
    CHECK_LAUNCHES(c);
    return PASS_OK;
}

// ------------------------------------------------------------------------------- C ABI
extern "C" {

size_t pass_kv_bytes(const pass_config* cfg) {
    if (!config_ok(cfg)) return 0;
    return (size_t)cfg->n_layers * cfg->max_batch * cfg->kv_capacity * cfg->d_model * esize(cfg->dtype);
}

size_t pass_workspace_bytes(const pass_config* cfg) {
    if (!config_ok(cfg)) return 0;
    return make_layout(*cfg).total;
}

int pass_create(const pass_config* cfg, void* kv_k, void* kv_v, size_t kv_bytes, void* workspace,
                size_t workspace_bytes, void* cuda_stream, pass_ctx** out) {
    if (!out) return PASS_ERR_INVALID_ARG;
    *out = nullptr;
    if (!config_ok(cfg) || !kv_k || !kv_v || !workspace) return PASS_ERR_INVALID_ARG;
    if (((uintptr_t)kv_k | (uintptr_t)kv_v | (uintptr_t)workspace) & 255) return PASS_ERR_INVALID_ARG;
    if (kv_bytes < pass_kv_bytes(cfg)) return PASS_ERR_CAPACITY;
    const Layout L = make_layout(*cfg);
    if (workspace_bytes < L.total) return PASS_ERR_CAPACITY;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return PASS_ERR_CUDA;
    pass_ctx* c = new (std::nothrow) pass_ctx();
    if (!c) return PASS_ERR_CUDA;
    c->cfg = *cfg;
    c->md = ModelDims{cfg->n_layers, cfg->d_model, cfg->n_heads, cfg->d_head, cfg->d_ffn, cfg->vocab,
                      cfg->k_max, cfg->max_batch, cfg->kv_capacity, cfg->dtype, cfg->rms_eps,
                      cfg->rope_theta};
    c->stream = (cudaStream_t)cuda_stream;
    c->kv_k = kv_k;
    c->kv_v = kv_v;
    c->ws = (char*)workspace;
    c->L = L;
    char* w = c->ws;
    c->d_states = (SeqState*)(w + L.states);
    c->d_params = (StepParams*)(w + L.params);
    c->d_unif = (float*)(w + L.unif);
    c->d_status = (int*)(w + L.status);
    c->d_row_seq = (int*)(w + L.row_seq);
    c->d_row_pos = (int*)(w + L.row_pos);
    c->d_tok = (int*)(w + L.tok);
    c->d_cs = (float2*)(w + L.cs);
    c->d_invfreq = (double*)(w + L.invfreq);
    c->d_h = (float*)(w + L.h);
    c->d_xn = (float*)(w + L.xn);
    c->d_qkv = (float*)(w + L.qkv);
    c->d_attn = (float*)(w + L.attn);
    c->d_gu = (float*)(w + L.gu);
    c->d_act = (float*)(w + L.act);
    c->d_logits = (float*)(w + L.logits);
    c->vb.logits = c->d_logits;
    c->vb.E = (double*)(w + L.E);
    c->vb.chunk = (double*)(w + L.chunk);
    c->vb.row_sum = (double*)(w + L.row_sum);
    c->vb.row_max = (float*)(w + L.row_max);
    c->vb.amax_val = (float*)(w + L.amax_val);
    c->vb.amax_idx = (int*)(w + L.amax_idx);
    c->vb.q_logits = (float*)(w + L.q_logits);
    c->vb.q_E = (double*)(w + L.q_E);
    c->vb.q_sum = (double*)(w + L.q_sum);
    c->vb.status = c->d_status;
    c->d_scratch = (double*)(w + L.scratch);
    if (cfg->dtype == PASS_DTYPE_BF16) {
        c->d_xn_bf = (__nv_bfloat16*)(w + L.xn_bf);
        c->d_attn_bf = (__nv_bfloat16*)(w + L.attn_bf);
        c->d_act_bf = (__nv_bfloat16*)(w + L.act_bf);
        c->d_q_out = (float*)(w + L.q_out);
        c->d_sumsq_a = (float*)(w + L.sumsq_a);
        c->d_sumsq_b = (float*)(w + L.sumsq_b);
        c->d_partial = (float*)(w + L.partial_ws);
        c->d_ll = (float*)(w + L.ll_ws);
        c->d_counters = (int*)(w + L.counters);
        c->d_attn_po = (float*)(w + L.attn_po);
        c->d_attn_pml = (float*)(w + L.attn_pml);
        c->d_attn_cnt = (int*)(w + L.attn_cnt);
        c->d_chain_flags = (int*)(w + L.chain_flags);
        c->d_packed = w + L.packed;
        c->packed = getenv("PASS_NO_PACK") == nullptr;
        c->use_tc = getenv("PASS_FORCE_SIMT") == nullptr;
        c->use_pdl = getenv("PASS_NO_PDL") == nullptr;
        c->attn_cluster = getenv("PASS_ATTN_NO_CLUSTER") == nullptr;
        c->attn_tc = getenv("PASS_ATTN_NO_TC") == nullptr;
        if (c->md.dh == kTcDH) {
            const uint64_t cache_rows = (uint64_t)c->md.n_layers * c->md.B * c->md.H * c->md.cap;
            c->attn_tc_ready = cache_rows < (1ull << 31) && make_map(&c->attn_tc_maps.k, kv_k, cache_rows, kTcDH, kTcBK) &&
                               make_map(&c->attn_tc_maps.v, kv_v, cache_rows, kTcDH, kTcBK);
        }
        if (const char* e = getenv("PASS_ATTN_LONG_FROM")) c->attn_long_from = std::max(0, atoi(e));
        c->trace = getenv("PASS_TRACE") != nullptr;
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
            c->n_sms = std::min(sms, kMaxCtas);
    }
    c->len_ub.assign(cfg->max_batch, 0);
    c->prefilled.assign(cfg->max_batch, 0);
    c->use_graph = getenv("PASS_NO_GRAPH") == nullptr;

    auto fail = [&](int code) { pass_destroy(c); return code; };
    if (cudaMallocHost((void**)&c->pin_params, sizeof(StepParams) * kParamRing) != cudaSuccess) return fail(PASS_ERR_CUDA);
    if (cudaMallocHost((void**)&c->pin_unif, sizeof(float) * cfg->max_batch * kUSlots) != cudaSuccess) return fail(PASS_ERR_CUDA);
    if (cudaMallocHost((void**)&c->pin_states, sizeof(SeqState) * cfg->max_batch) != cudaSuccess) return fail(PASS_ERR_CUDA);
    if (cudaMallocHost((void**)&c->pin_status, sizeof(int)) != cudaSuccess) return fail(PASS_ERR_CUDA);
    if (cudaMallocHost((void**)&c->pin_tok, sizeof(int) * kRowsCap) != cudaSuccess) return fail(PASS_ERR_CUDA);

    // zero the small state region; rotary frequencies theta^(-2i/d_head) in float64
    if (cudaMemsetAsync(w, 0, L.h, c->stream) != cudaSuccess) return fail(PASS_ERR_CUDA);
    if (cfg->dtype == PASS_DTYPE_BF16 &&
        cudaMemsetAsync(w + L.xn_bf, 0, L.packed - L.xn_bf, c->stream) != cudaSuccess) return fail(PASS_ERR_CUDA);
    // the hand-over slots of the step's GEMMs are EMPTY (all bits set) whenever no launch is using them
    if (cfg->dtype == PASS_DTYPE_BF16 &&
        cudaMemsetAsync(w + L.ll_ws, 0xFF, kLLRegionBytes * kMaxOps, c->stream) != cudaSuccess) return fail(PASS_ERR_CUDA);
    // stamps are told from empty slots by being non-zero
    if (c->trace && attn_trace_base(c) &&
        cudaMemsetAsync(attn_trace_base(c), 0, (size_t)kTraceLaunches * (kMaxOps * kMaxCtas * 8 + kAttnTraceWords) * 8, c->stream) != cudaSuccess)
        return fail(PASS_ERR_CUDA);
    std::vector<double> inv(cfg->d_head / 2);
    for (int i = 0; i < cfg->d_head / 2; i++)
        inv[i] = std::pow((double)cfg->rope_theta, -2.0 * i / cfg->d_head);
    if (cudaMemcpyAsync(c->d_invfreq, inv.data(), inv.size() * 8, cudaMemcpyHostToDevice, c->stream) != cudaSuccess) return fail(PASS_ERR_CUDA);
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return fail(PASS_ERR_CUDA);
    *out = c;
    return PASS_OK;
}

int pass_load_weights(pass_ctx* c, const pass_weights* w) {
    if (!c || !w) return PASS_ERR_INVALID_ARG;
    const void* singles[] = {w->tok_emb, w->la_emb, w->lm_head, w->final_norm};
    for (const void* p : singles)
        if (!p || ((uintptr_t)p & 15)) return PASS_ERR_INVALID_ARG;
    const void* const* arrays[] = {w->wq, w->wk, w->wv, w->wo, w->wg, w->wu, w->wd, w->norm_attn, w->norm_ffn};
    for (auto a : arrays) {
        if (!a) return PASS_ERR_INVALID_ARG;
        for (int l = 0; l < c->md.n_layers; l++)
            if (!a[l] || ((uintptr_t)a[l] & 15)) return PASS_ERR_INVALID_ARG;
    }
    c->tok_emb = w->tok_emb; c->la_emb = w->la_emb; c->lm_head = w->lm_head; c->final_norm = w->final_norm;
    const int nl = c->md.n_layers;
    c->wq.assign(w->wq, w->wq + nl); c->wk.assign(w->wk, w->wk + nl); c->wv.assign(w->wv, w->wv + nl);
    c->wo.assign(w->wo, w->wo + nl); c->wg.assign(w->wg, w->wg + nl); c->wu.assign(w->wu, w->wu + nl);
    c->wd.assign(w->wd, w->wd + nl);
    c->norm_attn.assign(w->norm_attn, w->norm_attn + nl);
    c->norm_ffn.assign(w->norm_ffn, w->norm_ffn + nl);
    for (auto& g : c->graphs) cudaGraphExecDestroy(g.second);
    c->graphs.clear();
    if (c->use_tc) {
        const int d = c->md.d, f = c->md.f;
        std::vector<CUtensorMap>* tms[] = {&c->tm_wq, &c->tm_wk, &c->tm_wv, &c->tm_wo, &c->tm_wg, &c->tm_wu, &c->tm_wd};
        const std::vector<const void*>* ws[] = {&c->wq, &c->wk, &c->wv, &c->wo, &c->wg, &c->wu, &c->wd};
        const int rows[] = {d, d, d, d, f, f, d}, cols[] = {d, d, d, d, d, d, f};
        // With packing on, every matrix is first copied into streaming order inside the workspace and
        // the map is laid over the copy; the caller's matrices stay as they are.
        char* pk = c->d_packed;
        auto weight_map = [&](CUtensorMap* m, const void* W, int N, int K, int box_rows) -> bool {
            if (!c->packed) return make_map(m, W, N, K, box_rows);
            const int n_tiles = (N + box_rows - 1) / box_rows, kbpt = (K + kBlockK - 1) / kBlockK;
            const size_t bytes = packed_matrix_bytes(N, K, box_rows);
            if (pk + bytes > c->d_packed + c->L.packed_bytes) return false;
            const int blocks = (int)std::min<size_t>(148 * 16, (bytes / 16 + 255) / 256);
            LAUNCH(c, k_pack_weight, blocks, 256, (const __nv_bfloat16*)W, N, K, box_rows, n_tiles, kbpt, (__nv_bfloat16*)pk);
            const bool ok = make_map_packed(m, pk, (uint64_t)n_tiles * kbpt, box_rows);
            pk += bytes;
            return ok;
        };
        for (int i = 0; i < 7; i++) {
            tms[i]->resize(nl);
            for (int l = 0; l < nl; l++)
                if (!weight_map(&(*tms[i])[l], (*ws[i])[l], rows[i], cols[i], (i == 4 || i == 5) ? 64 : 128)) return PASS_ERR_CUDA;
        }
        if (!weight_map(&c->tm_lm, c->lm_head, c->md.V, d, 128)) return PASS_ERR_CUDA;
        CHECK_LAUNCHES(c);
        CUDA_TRY(cudaStreamSynchronize(c->stream));
        c->tm_wg_plain.resize(nl);
        c->tm_wu_plain.resize(nl);
        for (int l = 0; l < nl; l++) {
            if (!make_map(&c->tm_wg_plain[l], c->wg[l], f, d, 128)) return PASS_ERR_CUDA;
            if (!make_map(&c->tm_wu_plain[l], c->wu[l], f, d, 128)) return PASS_ERR_CUDA;
        }
    }
    c->weights_loaded = true;
    return PASS_OK;
}

int pass_reset(pass_ctx* c, int seq) {
    if (!c || seq < 0 || seq >= c->md.B) return PASS_ERR_INVALID_ARG;
    LAUNCH(c, k_update_state, 1, 1, c->d_states, seq, 0, 0, 0, 0, 0, 1);
    CHECK_LAUNCHES(c);
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    c->len_ub[seq] = 0;
    c->prefilled[seq] = 0;
    return PASS_OK;
}

int pass_set_top_k(pass_ctx* c, int top_k) {
    if (!c || top_k < 0 || top_k > PASS_MAX_TOP_K) return PASS_ERR_INVALID_ARG;
    c->top_k = top_k;
    return PASS_OK;
}

int pass_set_state(pass_ctx* c, int seq, int len, int32_t pending) {
    if (!c || seq < 0 || seq >= c->md.B || len < 0 || pending < 0 || pending >= c->md.V) return PASS_ERR_INVALID_ARG;
    if (len > c->md.cap) return PASS_ERR_CAPACITY;
    LAUNCH(c, k_update_state, 1, 1, c->d_states, seq, 1, len, 0, 1, (int)pending, 0);
    CHECK_LAUNCHES(c);
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    c->len_ub[seq] = len;
    c->prefilled[seq] = 1;
    return PASS_OK;
}

int pass_forward_tokens(pass_ctx* c, int seq, const int32_t* tokens, int n, float* logits_out_device,
                        int commit) {
    if (!c || !tokens || seq < 0 || seq >= c->md.B || n < 1 || n > kMaxRows || commit < 0 || commit > n)
        return PASS_ERR_INVALID_ARG;
    if (!c->weights_loaded) return PASS_ERR_STATE;
    for (int i = 0; i < n; i++)
        if (tokens[i] < 0 || tokens[i] >= c->md.V + c->md.k_max) return PASS_ERR_INVALID_ARG;
    if (c->pending_collect) {
        const int rc = pass_step_collect(c, nullptr, nullptr);
        if (rc != PASS_OK) return rc;
    }
    if (c->len_ub[seq] + n > c->md.cap) return PASS_ERR_CAPACITY;
    int rc = run_tokens(c, seq, tokens, n, logits_out_device != nullptr);
    if (rc != PASS_OK) return rc;
    if (logits_out_device)
        CUDA_TRY(cudaMemcpyAsync(logits_out_device, c->d_logits, sizeof(float) * (size_t)n * c->md.V,
                                 cudaMemcpyDeviceToDevice, c->stream));
    LAUNCH(c, k_update_state, 1, 1, c->d_states, seq, 0, 0, commit, 0, 0, 0);
    CHECK_LAUNCHES(c);
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    c->len_ub[seq] += commit;
    return PASS_OK;
}

int pass_prefill(pass_ctx* c, int seq, const int32_t* tokens, int n) {
    if (!c || !tokens || seq < 0 || seq >= c->md.B || n < 1) return PASS_ERR_INVALID_ARG;
    if (!c->weights_loaded) return PASS_ERR_STATE;
    for (int i = 0; i < n; i++)
        if (tokens[i] < 0 || tokens[i] >= c->md.V) return PASS_ERR_INVALID_ARG;
    if (n - 1 > c->md.cap) return PASS_ERR_CAPACITY;
    if (c->pending_collect) {
        const int rc = pass_step_collect(c, nullptr, nullptr);
        if (rc != PASS_OK) return rc;
    }
    int rc = pass_reset(c, seq);
    if (rc != PASS_OK) return rc;
    // The prompt goes through the layers in chunks.  bf16 models on the tensor-core path: chunks of up to
    // kRowsCap rows as large GEMMs over (feature tile, token tile) units with plain bf16 activations and causal
    // flash attention, as long as more than kMaxRows rows remain; the last rows (and every other model) in
    // chunks of up to kMaxRows rows through the step's own kernels.
    const bool can_big = c->use_tc && getenv("PASS_NO_BIG_PREFILL") == nullptr;
    for (int s = 0; s < n - 1;) {
        const int left = n - 1 - s;
        const bool big = can_big && left > kMaxRows;
        const int big_rows = c->prompt_plain_bf16 ? kRowsCap : kRowsCap / 2;    // hi + lo parts take two buffer rows per token
        const int rows = std::min(big ? big_rows : kMaxRows, left);
        rc = run_tokens(c, seq, tokens + s, rows, false, big);
        if (rc != PASS_OK) return rc;
        s += rows;
        LAUNCH(c, k_update_state, 1, 1, c->d_states, seq, 0, 0, rows, 0, 0, 0);
        CUDA_TRY(cudaStreamSynchronize(c->stream));   // pin_tok is reused by the next chunk
    }
    LAUNCH(c, k_update_state, 1, 1, c->d_states, seq, 0, 0, 0, 1, (int)tokens[n - 1], 0);
    CHECK_LAUNCHES(c);
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    c->len_ub[seq] = n - 1;
    c->prefilled[seq] = 1;
    return PASS_OK;
}

// A launch that gave up on a bounded wait may leave its cross-CTA scratch half used: hand-over words
// that are not EMPTY, arrival counters of split tiles and of attention slices that are not zero.  All of
// it goes back to the idle state, in stream order, before the next launch.
static cudaError_t scrub_after_timeout(pass_ctx* c) {
    cudaError_t e = cudaMemsetAsync(c->d_ll, 0xFF, kLLRegionBytes * kMaxOps, c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->d_counters, 0, 4096 * sizeof(int), c->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->d_attn_cnt, 0, (size_t)c->md.B * c->md.H * sizeof(int), c->stream);
    return e;
}

static int step_checks(pass_ctx* c, int k, float T, const void* uniforms) {
    if (!c || k < 0 || k > c->md.k_max || !(T >= 0.f) || !std::isfinite(T)) return PASS_ERR_INVALID_ARG;
    if (!uniforms && T != 0.f) return PASS_ERR_INVALID_ARG;
    if (!c->weights_loaded) return PASS_ERR_STATE;
    if (c->md.B * (1 + 2 * k) > kMaxRows) return PASS_ERR_CAPACITY;
    for (int b = 0; b < c->md.B; b++) {
        if (!c->prefilled[b]) return PASS_ERR_STATE;
        if (c->len_ub[b] + 1 + 2 * k > c->md.cap) return PASS_ERR_CAPACITY;
    }
    return PASS_OK;
}

static int step_launch(pass_ctx* c, int k, float T) {
    // step parameters: only re-sent when they differ from what the device holds
    const bool changed = k != c->last_k || T != c->last_T || c->top_k != c->last_top_k;
    const int drop = ((c->have_last && changed) || c->force_drop) ? 1 : 0;
    if (!c->params_on_device || !c->have_last || changed || drop != c->dev_drop ||
        c->validate_only != c->dev_validate_only) {
        if (c->ring_pos == kParamRing) {
            CUDA_TRY(cudaStreamSynchronize(c->stream));
            c->ring_pos = 0;
        }
        StepParams* p = c->pin_params + c->ring_pos++;
        p->temperature = T; p->k = k; p->drop_drafts = drop; p->top_k = c->top_k;
        p->validate_only = c->validate_only; p->pad_[0] = p->pad_[1] = p->pad_[2] = 0;
        CUDA_TRY(cudaMemcpyAsync(c->d_params, p, sizeof(StepParams), cudaMemcpyHostToDevice, c->stream));
        c->params_on_device = true;
        c->dev_drop = drop;
        c->dev_validate_only = c->validate_only;
    }
    c->have_last = true; c->last_k = k; c->last_T = T; c->last_top_k = c->top_k;
    c->launches = 0;
    // one graph per (k, short / long contexts): the number of attention slices is part of the launch shape
    c->attn_long = false;
    for (int b = 0; b < c->md.B; b++) c->attn_long |= c->len_ub[b] >= c->attn_long_from;
    const int gkey = k + (c->attn_long ? 1000 : 0);
    if (c->use_graph) {
        auto it = c->graphs.find(gkey);
        if (it == c->graphs.end()) {
            cudaGraph_t g = nullptr;
            CUDA_TRY(cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
            enqueue_step_any(c, k);
            cudaError_t e = cudaStreamEndCapture(c->stream, &g);
            if (e != cudaSuccess || !g || launch_failed(c)) {
                if (g) cudaGraphDestroy(g);
                return PASS_ERR_CUDA;
            }
            cudaGraphExec_t ge = nullptr;
            e = cudaGraphInstantiate(&ge, g, 0);
            cudaGraphDestroy(g);
            if (e != cudaSuccess) return PASS_ERR_CUDA;
            c->graphs[gkey] = ge;
            c->graph_launches[gkey] = c->launches;
            it = c->graphs.find(gkey);
        }
        CUDA_TRY(cudaGraphLaunch(it->second, c->stream));
        c->last_step_launches = c->graph_launches[gkey];
    } else {
        enqueue_step_any(c, k);
        CHECK_LAUNCHES(c);
        c->last_step_launches = c->launches;
    }
    c->last_rows = c->md.B * (1 + 2 * k);
    for (int b = 0; b < c->md.B; b++) c->len_ub[b] += k + 1;
    c->pending_collect = true;
    return PASS_OK;
}

int pass_step_enqueue(pass_ctx* c, int k, float T, const float* uniforms_device) {
    int rc = step_checks(c, k, T, uniforms_device);
    if (rc != PASS_OK) return rc;
    if (uniforms_device)
        CUDA_TRY(cudaMemcpy2DAsync(c->d_unif, kUSlots * sizeof(float), uniforms_device,
                                   (2 * k + 1) * sizeof(float), (2 * k + 1) * sizeof(float), c->md.B,
                                   cudaMemcpyDeviceToDevice, c->stream));
    return step_launch(c, k, T);
}

int pass_step_collect(pass_ctx* c, int32_t* out_tokens, int32_t* n_out) {
    if (!c) return PASS_ERR_INVALID_ARG;
    if (!c->pending_collect) return PASS_ERR_STATE;
    CUDA_TRY(cudaMemcpyAsync(c->pin_states, c->d_states, sizeof(SeqState) * c->md.B, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(cudaMemcpyAsync(c->pin_status, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    c->pending_collect = false;
    for (int b = 0; b < c->md.B; b++) c->len_ub[b] = c->pin_states[b].kv_len;
    const int status = *c->pin_status;
    if (status != 0) {
        CUDA_TRY(cudaMemsetAsync(c->d_status, 0, sizeof(int), c->stream));
        if ((status & kStatusTimeout) && c->d_ll) CUDA_TRY(scrub_after_timeout(c));
        CUDA_TRY(cudaStreamSynchronize(c->stream));
        if (status & kStatusTimeout) return PASS_ERR_TIMEOUT;
        if (status & kStatusNonFinite) return PASS_ERR_NONFINITE;
        return PASS_ERR_STATE;
    }
    for (int b = 0; b < c->md.B; b++) {
        if (n_out) n_out[b] = c->pin_states[b].n_out;
        if (out_tokens)
            for (int j = 0; j <= c->md.k_max; j++)
                out_tokens[b * (c->md.k_max + 1) + j] = j < c->pin_states[b].n_out ? c->pin_states[b].out_tokens[j] : -1;
    }
    return PASS_OK;
}

int pass_step(pass_ctx* c, int k, float T, const float* uniforms, int32_t* out_tokens, int32_t* n_out) {
    if (!out_tokens || !n_out) return PASS_ERR_INVALID_ARG;
    int rc = step_checks(c, k, T, uniforms);
    if (rc != PASS_OK) return rc;
    if (c->pending_collect) {
        rc = pass_step_collect(c, nullptr, nullptr);
        if (rc != PASS_OK) return rc;
        rc = step_checks(c, k, T, uniforms);
        if (rc != PASS_OK) return rc;
    }
    if (uniforms) {
        for (int b = 0; b < c->md.B; b++)
            for (int j = 0; j < 2 * k + 1; j++) {
                const float u = uniforms[b * (2 * k + 1) + j];
                if (!(u >= 0.f && u < 1.f)) return PASS_ERR_INVALID_ARG;
                c->pin_unif[b * kUSlots + j] = u;
            }
        CUDA_TRY(cudaMemcpyAsync(c->d_unif, c->pin_unif, sizeof(float) * c->md.B * kUSlots, cudaMemcpyHostToDevice, c->stream));
    }
    rc = step_launch(c, k, T);
    if (rc != PASS_OK) return rc;
    return pass_step_collect(c, out_tokens, n_out);
}

int pass_step_two_call(pass_ctx* c, int L, float T, const float* uniforms, int32_t* out_tokens, int32_t* n_out) {
    if (!c || !out_tokens || !n_out || L < 0 || L > c->md.k_max) return PASS_ERR_INVALID_ARG;
    if (!uniforms && T != 0.f) return PASS_ERR_INVALID_ARG;
    const int B = c->md.B, km = c->md.k_max, nu = 2 * L + 2;
    std::vector<float> u1((size_t)B * (2 * L + 1), 0.f), u2((size_t)B * (2 * L + 1), 0.f);
    std::vector<int32_t> t1((size_t)B * (km + 1)), t2((size_t)B * (km + 1)), n1(B), n2(B);
    if (uniforms) {
        for (int b = 0; b < B; b++) {
            const float* U = uniforms + (size_t)b * nu;
            for (int j = 0; j < nu; j++)
                if (!(U[j] >= 0.f && U[j] < 1.f)) return PASS_ERR_INVALID_ARG;
            float* a = u1.data() + (size_t)b * (2 * L + 1);
            float* v = u2.data() + (size_t)b * (2 * L + 1);
            a[L] = U[0];                                         // x_{n+1}
            for (int t = 0; t < L; t++) a[L + 1 + t] = U[1 + t];  // drafts
            for (int j = 0; j < L; j++) v[j] = U[L + 1 + j];      // accept tests
            v[L] = U[2 * L + 1];                                  // residual / extra token
        }
    }
    // drafting call: [x_n, LA_1..LA_L], no pending drafts
    c->force_drop = true;
    c->validate_only = 0;
    int rc = pass_step(c, L, T, uniforms ? u1.data() : nullptr, t1.data(), n1.data());
    c->force_drop = false;
    if (rc != PASS_OK) return rc;
    // validation call: [x_{n+1}, d_1..d_L]
    c->validate_only = 1;
    rc = pass_step(c, L, T, uniforms ? u2.data() : nullptr, t2.data(), n2.data());
    c->validate_only = 0;
    if (rc != PASS_OK) return rc;
    for (int b = 0; b < B; b++) {
        int32_t* o = out_tokens + (size_t)b * (km + 2);
        o[0] = t1[(size_t)b * (km + 1)];
        for (int j = 0; j < n2[b]; j++) o[1 + j] = t2[(size_t)b * (km + 1) + j];
        n_out[b] = 1 + n2[b];
    }
    return PASS_OK;
}

static int kv_copy(pass_ctx* c, int seq, int layer, int pos0, int n, void* k, void* v, int gather) {
    if (!c || !k || !v || seq < 0 || seq >= c->md.B || layer < 0 || layer >= c->md.n_layers || pos0 < 0 || n < 1)
        return PASS_ERR_INVALID_ARG;
    if (pos0 + n > c->md.cap) return PASS_ERR_CAPACITY;
    if (c->pending_collect) {
        const int rc = pass_step_collect(c, nullptr, nullptr);
        if (rc != PASS_OK) return rc;
    }
    const size_t es = esize(c->md.dtype), rowb = (size_t)c->md.d * es;
    const size_t stage_bytes = (size_t)kMaxRows * c->md.V * 8;     // the E buffer doubles as staging
    const int chunk = (int)std::max<size_t>(1, std::min<size_t>(n, stage_bytes / rowb));
    void* stage = c->vb.E;
    void* host[2] = {k, v};
    void* cache[2] = {c->kv_k, c->kv_v};
    for (int which = 0; which < 2; which++)
        for (int s = 0; s < n; s += chunk) {
            const int cn = std::min(chunk, n - s);
            char* hp = (char*)host[which] + (size_t)s * rowb;
            if (!gather) CUDA_TRY(cudaMemcpyAsync(stage, hp, cn * rowb, cudaMemcpyHostToDevice, c->stream));
            const int blocks = (int)std::min<size_t>(1024, ((size_t)cn * c->md.d + 255) / 256);
            if (es == 4)
                LAUNCH(c, (k_kv_scatter<float>), blocks, 256, (const float*)stage, c->md, layer, seq, pos0 + s, cn, (float*)cache[which], gather);
            else
                LAUNCH(c, (k_kv_scatter<__nv_bfloat16>), blocks, 256, (const __nv_bfloat16*)stage, c->md, layer, seq, pos0 + s, cn, (__nv_bfloat16*)cache[which], gather);
            if (gather) CUDA_TRY(cudaMemcpyAsync(hp, stage, cn * rowb, cudaMemcpyDeviceToHost, c->stream));
            CUDA_TRY(cudaStreamSynchronize(c->stream));
        }
    CHECK_LAUNCHES(c);
    return PASS_OK;
}

int pass_set_kv(pass_ctx* c, int seq, int layer, int pos0, int n, const void* k, const void* v) {
    return kv_copy(c, seq, layer, pos0, n, const_cast<void*>(k), const_cast<void*>(v), 0);
}
int pass_get_kv(pass_ctx* c, int seq, int layer, int pos0, int n, void* k, void* v) {
    return kv_copy(c, seq, layer, pos0, n, k, v, 1);
}

int pass_get_debug(pass_ctx* c, int what, void* dst, size_t bytes) {
    if (!c || !dst) return PASS_ERR_INVALID_ARG;
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    const int B = c->md.B, V = c->md.V, km = c->md.k_max;
    auto need = [&](size_t n) { return bytes >= n; };
    if (what == PASS_DBG_LOGITS || what == PASS_DBG_HIDDEN) {
        const size_t n = (size_t)c->last_rows * (what == PASS_DBG_LOGITS ? V : c->md.d) * 4;
        if (!need(n)) return PASS_ERR_CAPACITY;
        CUDA_TRY(cudaMemcpy(dst, what == PASS_DBG_LOGITS ? c->d_logits : c->d_h, n, cudaMemcpyDeviceToHost));
        return PASS_OK;
    }
    if (what == PASS_DBG_TRACE) {
        if (!trace_base(c)) return PASS_ERR_STATE;
        const size_t n = std::min(bytes, (size_t)kTraceLaunches * kMaxOps * kMaxCtas * 8 * 8);
        CUDA_TRY(cudaMemcpy(dst, trace_base(c), n, cudaMemcpyDeviceToHost));
        c->trace_launch = 0;
        return PASS_OK;
    }
    if (what == PASS_DBG_ATTN_TRACE) {
        if (!attn_trace_base(c)) return PASS_ERR_STATE;
        const size_t n = std::min(bytes, (size_t)kTraceLaunches * kAttnTraceWords * 8);
        CUDA_TRY(cudaMemcpy(dst, attn_trace_base(c), n, cudaMemcpyDeviceToHost));
        c->attn_trace_launch = 0;
        return PASS_OK;
    }
    if (what == PASS_DBG_FOOTPRINT) {
        // shared memory of the step's two big kernels (bf16 models): they are meant to share an SM
        if (!need(6 * 4)) return PASS_ERR_CAPACITY;
        if (!c->use_tc) return PASS_ERR_STATE;
        cudaFuncAttributes ag, aa;
        CUDA_TRY(cudaFuncGetAttributes(&ag, k_gemm_tc));
        if (c->md.dh == 128) CUDA_TRY(cudaFuncGetAttributes(&aa, k_attn_fd<128, 1, true, true, false, 2, 232>));
        else CUDA_TRY(cudaFuncGetAttributes(&aa, k_attn_fd<64, 1, true, true, false, 2, 232>));
        int dev = 0, sm_total = 0, reserved = 0;
        CUDA_TRY(cudaGetDevice(&dev));
        CUDA_TRY(cudaDeviceGetAttribute(&sm_total, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev));
        CUDA_TRY(cudaDeviceGetAttribute(&reserved, cudaDevAttrReservedSharedMemoryPerBlock, dev));
        int* o = (int*)dst;
        o[0] = (int)ag.sharedSizeBytes;
        o[1] = gemm_stages(32) * (kATileBytes + 32 * 128) + 1024;
        o[2] = (int)aa.sharedSizeBytes;
        o[3] = 2 * 2 * kAttnBK * c->md.dh * 2;          // ring of two stages
        o[4] = sm_total;
        o[5] = reserved;
        if (bytes >= 9 * 4) {
            // registers: allocated in units of 8 per thread; the two CTAs must fit the SM's register file together
            int regs_total = 0;
            CUDA_TRY(cudaDeviceGetAttribute(&regs_total, cudaDevAttrMaxRegistersPerMultiprocessor, dev));
            o[6] = ((ag.numRegs + 7) / 8) * 8 * kGemmThreads;
            o[7] = ((aa.numRegs + 7) / 8) * 8 * 128;
            o[8] = regs_total;
        }
        return PASS_OK;
    }
    if (what == PASS_DBG_STATUS) {
        if (!need(4)) return PASS_ERR_CAPACITY;
        CUDA_TRY(cudaMemcpy(dst, c->d_status, 4, cudaMemcpyDeviceToHost));
        return PASS_OK;
    }
    std::vector<SeqState> st(B);
    CUDA_TRY(cudaMemcpy(st.data(), c->d_states, sizeof(SeqState) * B, cudaMemcpyDeviceToHost));
    int* o = (int*)dst;
    switch (what) {
        case PASS_DBG_DRAFT_LOGITS: {
            if (!need((size_t)B * km * V * 4)) return PASS_ERR_CAPACITY;
            for (int b = 0; b < B; b++)
                CUDA_TRY(cudaMemcpy((float*)dst + (size_t)b * km * V,
                                    c->vb.q_logits + ((size_t)b * 2 + st[b].q_sel) * km * V,
                                    (size_t)km * V * 4, cudaMemcpyDeviceToHost));
            return PASS_OK;
        }
        case PASS_DBG_KV_LEN: if (!need(4 * B)) return PASS_ERR_CAPACITY; for (int b = 0; b < B; b++) o[b] = st[b].kv_len; return PASS_OK;
        case PASS_DBG_N_DRAFT: if (!need(4 * B)) return PASS_ERR_CAPACITY; for (int b = 0; b < B; b++) o[b] = st[b].m; return PASS_OK;
        case PASS_DBG_PENDING: if (!need(4 * B)) return PASS_ERR_CAPACITY; for (int b = 0; b < B; b++) o[b] = st[b].pending; return PASS_OK;
        case PASS_DBG_N_ACCEPTED: if (!need(4 * B)) return PASS_ERR_CAPACITY; for (int b = 0; b < B; b++) o[b] = st[b].n_acc; return PASS_OK;
        case PASS_DBG_DRAFTS:
            if (!need((size_t)4 * B * km)) return PASS_ERR_CAPACITY;
            for (int b = 0; b < B; b++)
                for (int j = 0; j < km; j++) o[b * km + j] = j < st[b].m ? st[b].drafts[j] : -1;
            return PASS_OK;
        default: return PASS_ERR_INVALID_ARG;
    }
}

static int enqueue_debug_linear(pass_ctx* c, int which, int layer, int R, float* y_device) {
    const int d = c->md.d, f = c->md.f, npad = npad_for(R);
    const pass_ctx::BMaps* bm = get_bmaps(c, npad);
    if (!bm) return PASS_ERR_CUDA;
    const int K = which == 6 ? f : d;
    const CUtensorMap* a0 = nullptr;
    const CUtensorMap* a1 = nullptr;
    int N = d;
    switch (which) {
        case 0: a0 = &c->tm_wq[layer]; break;
        case 1: a0 = &c->tm_wk[layer]; break;
        case 2: a0 = &c->tm_wv[layer]; break;
        case 3: a0 = &c->tm_wo[layer]; break;
        case 4: a0 = &c->tm_wg_plain[layer]; N = f; break;
        case 5: a0 = &c->tm_wu_plain[layer]; N = f; break;
        case 6: a0 = &c->tm_wd[layer]; break;
        case 7: a0 = &c->tm_lm; N = c->md.V; break;
        default: a0 = &c->tm_wg[layer]; a1 = &c->tm_wu[layer]; N = ((f + 63) / 64) * 128; break;
    }
    const int n_tiles = which == 8 ? (f + 63) / 64 : (N + kTileN - 1) / kTileN;
    GemmParams p = gemm_base(c, R, npad, K, n_tiles, N, kEpiLogits);
    p.interleave = which == 8;
    if (which == 4 || which == 5) p.packed = 0;     // gate or up alone: 128-row boxes over the caller's matrix
    p.logits = y_device;
    launch_gemm(c, *a0, a1 ? *a1 : *a0, *a0, which == 6 ? bm->act : bm->xn, p);
    return PASS_OK;
}

static int debug_status(pass_ctx* c) {
    int status = 0;
    CUDA_TRY(cudaMemcpy(&status, c->d_status, 4, cudaMemcpyDeviceToHost));
    if (status) {
        CUDA_TRY(cudaMemset(c->d_status, 0, 4));
        if ((status & kStatusTimeout) && c->d_ll) {
            CUDA_TRY(scrub_after_timeout(c));
            CUDA_TRY(cudaStreamSynchronize(c->stream));
        }
        return (status & kStatusTimeout) ? PASS_ERR_TIMEOUT : PASS_ERR_STATE;
    }
    return PASS_OK;
}

int pass_debug_linear(pass_ctx* c, int which, int layer, const float* x_device, int R, float* y_device) {
    if (!c || !x_device || !y_device || which < 0 || which > 8 || R < 1 || R > kMaxRows) return PASS_ERR_INVALID_ARG;
    if (!c->weights_loaded || !c->use_tc) return PASS_ERR_STATE;
    if (which != 7 && (layer < 0 || layer >= c->md.n_layers)) return PASS_ERR_INVALID_ARG;
    if (c->pending_collect) {
        const int rc = pass_step_collect(c, nullptr, nullptr);
        if (rc != PASS_OK) return rc;
    }
    const int K = which == 6 ? c->md.f : c->md.d;
    LAUNCH(c, k_split_rows, dim3((K + 255) / 256, R), 256, x_device, K, which == 6 ? c->d_act_bf : c->d_xn_bf, npad_for(R) / 2);
    const int rc = enqueue_debug_linear(c, which, layer, R, y_device);
    if (rc != PASS_OK) return rc;
    CHECK_LAUNCHES(c);
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    return debug_status(c);
}

int pass_debug_time_linear(pass_ctx* c, int which, int R, int n_launches, float* ms_total) {
    if (!c || !ms_total || which < 0 || which > 9 || which == 7 || R < 1 || R > kMaxRows || n_launches < 1)
        return PASS_ERR_INVALID_ARG;
    if (!c->weights_loaded || !c->use_tc) return PASS_ERR_STATE;
    const int N = which == 8 ? ((c->md.f + 63) / 64) * 128 : (which == 4 || which == 5 ? c->md.f : c->md.d);
    if (which != 9 && N > c->md.V) return PASS_ERR_CAPACITY;          // results land in the logits buffer
    if (which == 9 && c->md.n_layers < 2) return PASS_ERR_INVALID_ARG;
    if (c->pending_collect) {
        const int rc = pass_step_collect(c, nullptr, nullptr);
        if (rc != PASS_OK) return rc;
    }
    const int npad = npad_for(R), nl = c->md.n_layers;
    const pass_ctx::BMaps* bm = get_bmaps(c, npad);
    if (!bm) return PASS_ERR_CUDA;
    auto one = [&](int i) {
        if (which == 9) {          // the step's dominant launch: O-proj -> gate|up -> down -> next layer's QKV
            ChainOp chain[kMaxOps];
            const int l = i % (nl - 1);
            launch_ops(c, chain, build_layer_chain(c, R, npad, bm, l, false, chain));
        } else {
            enqueue_debug_linear(c, which, i % nl, R, c->d_logits);
        }
    };
    if (which == 9) {              // rows at position 0 of sequence 0: the QKV epilogue needs valid row tables
        chain_counters_clear(c);
        CUDA_TRY(cudaMemsetAsync(c->d_row_seq, 0, sizeof(int) * kMaxRows, c->stream));
        CUDA_TRY(cudaMemsetAsync(c->d_row_pos, 0, sizeof(int) * kMaxRows, c->stream));
    }
    cudaEvent_t e0, e1;
    CUDA_TRY(cudaEventCreate(&e0));
    CUDA_TRY(cudaEventCreate(&e1));
    for (int i = 0; i < std::min(n_launches, nl); i++) one(i);        // warm-up pass
    CUDA_TRY(cudaEventRecord(e0, c->stream));
    for (int i = 0; i < n_launches; i++) one(i);
    CUDA_TRY(cudaEventRecord(e1, c->stream));
    CHECK_LAUNCHES(c);
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    CUDA_TRY(cudaEventElapsedTime(ms_total, e0, e1));
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return debug_status(c);
}

// ------------------------------------------------------------------------------- no-allocation linear
// Scratch of the split-K GEMM (the words through which CTAs that share an output tile hand their
// partial sums to the one that finishes it) kept inside the library image instead of in
// caller-provided memory.  Sized for at most kStaticMaxRows token rows; every GPU that loads the
// library carries these bytes until exit.
//
// Only ONE hand-over protocol ever touches the array: EMPTY-or-value words.  The GEMM kernel picks
// that protocol when the token rows are padded to 16 per half (rh == 16) and arrival counters with
// float4 partial slots otherwise, so this entry point pads EVERY call to 16 rows per half, whatever its
// row count.  A counter-protocol launch would leave its partial sums in the words, and a later finisher
// that polls a word before its contributor's store has landed would take such a leftover for the value.
constexpr int kStaticMaxRows = 16;
constexpr size_t kStaticPartialBytes = (size_t)kMaxCtas * 2 * kStaticMaxRows * kTileN * sizeof(float);
constexpr size_t kStaticCounterBytes = 4096 * sizeof(int);      // not used any more; keeps the array's size
static __device__ __align__(256) unsigned char g_static_scratch[kStaticPartialBytes + kStaticCounterBytes];

// Device address of g_static_scratch per device ordinal.  In host code the symbol's name is only a
// handle; the address a kernel can use has to be asked for, with that device current.
static void* g_static_scratch_addr[64] = {nullptr};

int pass_linear_noalloc(pass_ctx* c, int which, int layer, const float* x_device, int R, float* y_device) {
    if (!c || !x_device || !y_device || which < 0 || which > 8 || R < 1) return PASS_ERR_INVALID_ARG;
    if (R > kStaticMaxRows) {
        if (getenv("PASS_LOG"))
            fprintf(stderr, "[pass] pass_linear_noalloc: %d rows exceed the built-in scratch (max %d rows)\n", R, kStaticMaxRows);
        return PASS_ERR_CAPACITY;
    }
    if (!c->weights_loaded || !c->use_tc) return PASS_ERR_STATE;
    if (which != 7 && (layer < 0 || layer >= c->md.n_layers)) return PASS_ERR_INVALID_ARG;
    if (c->pending_collect) {
        const int rc = pass_step_collect(c, nullptr, nullptr);
        if (rc != PASS_OK) return rc;
    }
    int dev = -1;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return PASS_ERR_INVALID_ARG;
    if (!g_static_scratch_addr[dev]) {          // first call on this device
        void* ptr = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        // the hand-over words start out EMPTY (all bits set); every call leaves them that way
        CUDA_TRY(cudaMemsetAsync(ptr, 0xFF, kStaticPartialBytes, c->stream));
        g_static_scratch_addr[dev] = ptr;
    }
    char* scratch = (char*)g_static_scratch_addr[dev];

    const int d = c->md.d, f = c->md.f;
    const int npad = 2 * kStaticMaxRows;        // always 16 rows per half: the EMPTY-or-value protocol (see above)
    const pass_ctx::BMaps* bm = get_bmaps(c, npad);
    if (!bm) return PASS_ERR_CUDA;
    const int K = which == 6 ? f : d;
    LAUNCH(c, k_split_rows, dim3((K + 255) / 256, R), 256, x_device, K, which == 6 ? c->d_act_bf : c->d_xn_bf, npad / 2);
    const CUtensorMap* a0 = nullptr;
    const CUtensorMap* a1 = nullptr;
    int N = d;
    switch (which) {
        case 0: a0 = &c->tm_wq[layer]; break;
        case 1: a0 = &c->tm_wk[layer]; break;
        case 2: a0 = &c->tm_wv[layer]; break;
        case 3: a0 = &c->tm_wo[layer]; break;
        case 4: a0 = &c->tm_wg_plain[layer]; N = f; break;
        case 5: a0 = &c->tm_wu_plain[layer]; N = f; break;
        case 6: a0 = &c->tm_wd[layer]; break;
        case 7: a0 = &c->tm_lm; N = c->md.V; break;
        default: a0 = &c->tm_wg[layer]; a1 = &c->tm_wu[layer]; N = ((f + 63) / 64) * 128; break;
    }
    const int n_tiles = which == 8 ? (f + 63) / 64 : (N + kTileN - 1) / kTileN;
    GemmParams p = gemm_base(c, R, npad, K, n_tiles, N, kEpiLogits);
    p.interleave = which == 8;
    if (which == 4 || which == 5) p.packed = 0;
    p.logits = y_device;
    p.partial_ws = nullptr;                  // the counter protocol is never taken with rh == 16
    p.tile_counters = nullptr;
    p.ll_ws = (float*)scratch;
    launch_gemm(c, *a0, a1 ? *a1 : *a0, *a0, which == 6 ? bm->act : bm->xn, p);
    CHECK_LAUNCHES(c);
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    const int rc = debug_status(c);
    if (rc == PASS_ERR_TIMEOUT)     // an abandoned launch may have left words in the shared slots
        CUDA_TRY(cudaMemset(scratch, 0xFF, kStaticPartialBytes));
    return rc;
}

int pass_set_prompt_precision(pass_ctx* c, int mode) {
    if (!c || (mode != PASS_PROMPT_HI_LO && mode != PASS_PROMPT_BF16)) return PASS_ERR_INVALID_ARG;
    c->prompt_plain_bf16 = mode == PASS_PROMPT_BF16;
    return PASS_OK;
}

int pass_debug_set(pass_ctx* c, int hook, int value) {
    if (!c || value < 0) return PASS_ERR_INVALID_ARG;
    if (c->pending_collect) {
        const int rc = pass_step_collect(c, nullptr, nullptr);
        if (rc != PASS_OK) return rc;
    }
    switch (hook) {
        case PASS_HOOK_GEMM_STUCK: c->gemm_test_stuck = value ? 1 : 0; break;
        case PASS_HOOK_ATTN_STALE: c->attn_debug_stale = value; break;
        case PASS_HOOK_ATTN_LONG_FROM: c->attn_long_from = value; break;
        case PASS_HOOK_ATTN_STUCK: c->attn_test_stuck = value ? 1 : 0; break;
        default: return PASS_ERR_INVALID_ARG;
    }
    // the hooks are part of the launch parameters, which captured graphs hold by value
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    for (auto& g : c->graphs) cudaGraphExecDestroy(g.second);
    c->graphs.clear();
    c->graph_launches.clear();
    return PASS_OK;
}

int pass_debug_schedule(int n_tiles, int kb_per_tile, int n_ctas, int cta, int it, int32_t* out) {
    if (n_tiles < 1 || kb_per_tile < 1 || n_ctas < 1 || cta < 0 || cta >= n_ctas || it < 0 || !out) return -1;
    GemmParams p;
    memset(&p, 0, sizeof(p));
    p.n_tiles = n_tiles;
    p.kb_per_tile = kb_per_tile;
    Piece pc;
    if (!get_piece(p, cta, n_ctas, it, pc)) return 0;
    out[0] = pc.tile; out[1] = pc.kb0; out[2] = pc.kb1; out[3] = pc.n_pieces; out[4] = pc.index;
    out[5] = pc.slot; out[6] = pc.first_slot;
    return 1;
}

int pass_last_step_launches(pass_ctx* c) { return c ? c->last_step_launches : 0; }
void* pass_stream(pass_ctx* c) { return c ? (void*)c->stream : nullptr; }

void pass_destroy(pass_ctx* c) {
    if (!c) return;
    cudaStreamSynchronize(c->stream);
    for (auto& g : c->graphs) cudaGraphExecDestroy(g.second);
    for (auto& g : c->tr.graphs) cudaGraphExecDestroy(g.second);
    if (c->pin_params) cudaFreeHost(c->pin_params);
    if (c->pin_unif) cudaFreeHost(c->pin_unif);
    if (c->pin_states) cudaFreeHost(c->pin_states);
    if (c->pin_status) cudaFreeHost(c->pin_status);
    if (c->pin_tok) cudaFreeHost(c->pin_tok);
    if (c->tr.pin_targets) cudaFreeHost(c->tr.pin_targets);
    if (c->tr.pin_loss) cudaFreeHost(c->tr.pin_loss);
    delete c;
}

const char* pass_strerror(int code) {
    switch (code) {
        case PASS_OK: return "ok";
        case PASS_ERR_INVALID_ARG: return "invalid argument";
        case PASS_ERR_CAPACITY: return "capacity exceeded (KV cache, workspace or row limit)";
        case PASS_ERR_STATE: return "call not valid in this state";
        case PASS_ERR_CUDA: return "CUDA call failed";
        case PASS_ERR_NONFINITE: return "non-finite logit";
        case PASS_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown error";
    }
}

}  // extern "C"

// ------------------------------------------------------------------------------- look-ahead embedding training
namespace {

struct TrainLayout {
    size_t qkv_t, o_t, gu_t, d_t, lm_t;          // per-layer strides are the matrix sizes
    size_t master, m, v, grad, h_in, qkv, attn, h_mid, gu, h_last, dh, t0, t1, dlogits, loss_row, scratch, targets, stage;
    size_t total;
};

TrainLayout make_train_layout(const pass_config& c, int L, int max_seqs) {
    TrainLayout T;
    Carve cv;
    const size_t d = c.d_model, f = c.d_ffn, V = c.vocab, nl = c.n_layers, R = (size_t)L * max_seqs;
    const size_t ng = ((f + 63) / 64) * 128, wide = std::max(std::max(3 * d, 2 * f), ng);
    T.qkv_t = cv.take(nl * packed_matrix_bytes(d, 3 * d, 128));
    T.o_t = cv.take(nl * packed_matrix_bytes(d, d, 128));
    T.gu_t = cv.take(nl * packed_matrix_bytes(d, 2 * f, 128));
    T.d_t = cv.take(nl * packed_matrix_bytes(f, d, 128));
    T.lm_t = cv.take(packed_matrix_bytes(d, V, 128));
    T.master = cv.take(kMaxLA * d * 4); T.m = cv.take(kMaxLA * d * 4); T.v = cv.take(kMaxLA * d * 4); T.grad = cv.take(kMaxLA * d * 4);
    T.h_in = cv.take(nl * R * d * 4); T.qkv = cv.take(nl * R * 3 * d * 4); T.attn = cv.take(nl * R * d * 4);
    T.h_mid = cv.take(nl * R * d * 4); T.gu = cv.take(nl * R * ng * 4);
    T.h_last = cv.take(R * d * 4); T.dh = cv.take(R * d * 4); T.t0 = cv.take(R * wide * 4); T.t1 = cv.take(R * wide * 4);
    T.dlogits = cv.take(R * V * 4); T.loss_row = cv.take(R * 4);
    T.scratch = cv.take((size_t)max_seqs * c.n_heads * 2 * L * (size_t)(c.kv_capacity) * 4);
    T.targets = cv.take(R * 4);
    T.stage = cv.take((size_t)2 * kMaxRows * std::max(wide, V) * 2);
    T.total = cv.off;
    return T;
}

// One weight-streaming GEMM of the training passes: y [R][N] = x [R][K] (float32) times the matrix behind the
// maps, through the hi | lo staging rows.  n_maps = 3: three matrices of seg rows each one after the other (Q, K, V);
// interleave: gate | up in blocks of 64.
int train_gemm(pass_ctx* c, const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& a2, int seg_tiles,
               bool interleave, int N, int n_tiles, int K, const float* x, int R, float* y) {
    const int npad = npad_for(R);
    auto key = std::make_pair(K, npad);
    auto it = c->tr.stage_maps.find(key);
    if (it == c->tr.stage_maps.end()) {
        CUtensorMap m;
        if (!make_map(&m, c->tr.stage, 2 * kMaxRows, K, npad)) return PASS_ERR_CUDA;
        it = c->tr.stage_maps.emplace(key, m).first;
    }
    LAUNCH(c, k_split_rows, dim3((K + 255) / 256, R), 256, x, K, c->tr.stage, npad / 2);
    GemmParams p = gemm_base(c, R, npad, K, n_tiles, N, kEpiLogits);
    p.packed = 1;
    p.interleave = interleave ? 1 : 0;
    if (seg_tiles > 0) p.seg_tiles0 = p.seg_tiles1 = seg_tiles;
    p.logits = y;
    launch_gemm(c, a0, a1, a2, it->second, p);
    return PASS_OK;
}
int train_gemm1(pass_ctx* c, const CUtensorMap& a, int N, int K, const float* x, int R, float* y) {
    return train_gemm(c, a, a, a, 0, false, N, (N + kTileN - 1) / kTileN, K, x, R, y);
}

}  // namespace

extern "C" {

size_t pass_train_workspace_bytes(const pass_config* cfg, int L, int max_seqs) {
    if (!config_ok(cfg) || cfg->dtype != PASS_DTYPE_BF16 || L < 1 || L > cfg->k_max || max_seqs < 1 ||
        max_seqs > cfg->max_batch || L * max_seqs > kMaxRows)
        return 0;
    return make_train_layout(*cfg, L, max_seqs).total;
}

int pass_train_init(pass_ctx* c, void* train_ws_device, size_t bytes, const pass_train_config* hp, int L, int max_seqs) {
    if (!c || !train_ws_device || !hp || ((uintptr_t)train_ws_device & 255)) return PASS_ERR_INVALID_ARG;
    if (!c->weights_loaded || !c->use_tc || !c->packed) return PASS_ERR_STATE;
    const size_t need = pass_train_workspace_bytes(&c->cfg, L, max_seqs);
    if (need == 0) return PASS_ERR_INVALID_ARG;
    if (bytes < need) return PASS_ERR_CAPACITY;
    if (!(hp->lr > 0.f) || !(hp->beta1 >= 0.f && hp->beta1 < 1.f) || !(hp->beta2 >= 0.f && hp->beta2 < 1.f) ||
        !(hp->eps > 0.f) || hp->weight_decay < 0.f || hp->warmup_steps < 0 || hp->total_steps < 1)
        return PASS_ERR_INVALID_ARG;
    if (c->pending_collect) {
        const int rc = pass_step_collect(c, nullptr, nullptr);
        if (rc != PASS_OK) return rc;
    }
    typedef __nv_bfloat16 bf;
    pass_ctx::Train& t = c->tr;
    const TrainLayout T = make_train_layout(c->cfg, L, max_seqs);
    const int d = c->md.d, f = c->md.f, V = c->md.V, nl = c->md.n_layers;
    char* w = (char*)train_ws_device;
    t.ws = w; t.hp = *hp; t.L = L; t.max_seqs = max_seqs; t.step = 0; t.n_max = c->md.cap;
    t.ng = ((f + 63) / 64) * 128;
    t.master = (float*)(w + T.master); t.m = (float*)(w + T.m); t.v = (float*)(w + T.v); t.grad = (float*)(w + T.grad);
    t.h_in = (float*)(w + T.h_in); t.qkv = (float*)(w + T.qkv); t.attn = (float*)(w + T.attn); t.h_mid = (float*)(w + T.h_mid);
    t.gu = (float*)(w + T.gu); t.h_last = (float*)(w + T.h_last); t.dh = (float*)(w + T.dh); t.t0 = (float*)(w + T.t0);
    t.t1 = (float*)(w + T.t1); t.dlogits = (float*)(w + T.dlogits); t.loss_row = (float*)(w + T.loss_row);
    t.scratch = (float*)(w + T.scratch); t.targets = (int*)(w + T.targets); t.stage = (bf*)(w + T.stage);
    t.stage_maps.clear();
    for (auto& g : t.graphs) cudaGraphExecDestroy(g.second);
    t.graphs.clear();
    if (!t.pin_targets && cudaMallocHost((void**)&t.pin_targets, sizeof(int) * kMaxRows) != cudaSuccess) return PASS_ERR_CUDA;
    if (!t.pin_loss && cudaMallocHost((void**)&t.pin_loss, sizeof(float) * kMaxRows) != cudaSuccess) return PASS_ERR_CUDA;
    // transposed copies of the weights in streaming order (the backward GEMMs multiply by W, not by its transpose)
    auto pack_t = [&](CUtensorMap* m, char* dst, const void* s0, const void* s1, const void* s2, int n_src, int rows_src, int N) -> bool {
        const int K = n_src * rows_src, n_tiles = (N + 127) / 128, kbpt = (K + kBlockK - 1) / kBlockK;
        PackTSources ps;
        ps.src[0] = (const bf*)s0; ps.src[1] = (const bf*)s1; ps.src[2] = (const bf*)s2;
        LAUNCH(c, k_pack_weight_t, n_tiles * kbpt, 128, ps, n_src, rows_src, N, kbpt, (bf*)dst);
        return make_map_packed(m, dst, (uint64_t)n_tiles * kbpt, 128);
    };
    t.tm_qkv_t.resize(nl); t.tm_o_t.resize(nl); t.tm_gu_t.resize(nl); t.tm_d_t.resize(nl);
    for (int l = 0; l < nl; l++) {
        if (!pack_t(&t.tm_qkv_t[l], w + T.qkv_t + l * packed_matrix_bytes(d, 3 * d, 128), c->wq[l], c->wk[l], c->wv[l], 3, d, d)) return PASS_ERR_CUDA;
        if (!pack_t(&t.tm_o_t[l], w + T.o_t + l * packed_matrix_bytes(d, d, 128), c->wo[l], c->wo[l], c->wo[l], 1, d, d)) return PASS_ERR_CUDA;
        if (!pack_t(&t.tm_gu_t[l], w + T.gu_t + l * packed_matrix_bytes(d, 2 * f, 128), c->wg[l], c->wu[l], c->wu[l], 2, f, d)) return PASS_ERR_CUDA;
        if (!pack_t(&t.tm_d_t[l], w + T.d_t + l * packed_matrix_bytes(f, d, 128), c->wd[l], c->wd[l], c->wd[l], 1, d, f)) return PASS_ERR_CUDA;
    }
    if (!pack_t(&t.tm_lm_t, w + T.lm_t, c->lm_head, c->lm_head, c->lm_head, 1, V, d)) return PASS_ERR_CUDA;
    // float32 master rows from the context's look-ahead table, moments at zero
    LAUNCH(c, (k_rows_convert<bf>), (kMaxLA * d + 255) / 256, 256, (const bf*)c->la_emb, t.master, (size_t)c->md.k_max * d, 1);
    CUDA_TRY(cudaMemsetAsync(t.m, 0, sizeof(float) * kMaxLA * d, c->stream));
    CUDA_TRY(cudaMemsetAsync(t.v, 0, sizeof(float) * kMaxLA * d, c->stream));
    CUDA_TRY(cudaMemsetAsync(t.grad, 0, sizeof(float) * kMaxLA * d, c->stream));
    CHECK_LAUNCHES(c);
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    t.ready = true;
    return PASS_OK;
}

// Forward and backward over the look-ahead rows of n_seqs sequences (everything between the prompt passes and
// the update): enqueued on the context's stream, directly or into a graph capture.
static int train_enqueue_rows(pass_ctx* c, int n_seqs) {
    typedef __nv_bfloat16 bf;
    pass_ctx::Train& t = c->tr;
    const ModelDims& md = c->md;
    const int L = t.L, R = n_seqs * L, d = md.d, f = md.f, V = md.V, nl = md.n_layers, dt = d / kTileN;
    // ---- forward over the look-ahead rows, keeping what the backward pass needs
    LAUNCH(c, k_train_rows, R, 256, c->d_states, t.master, L, d, c->d_h, c->d_row_seq, c->d_row_pos);
    LAUNCH(c, k_rope_table, R, 64, c->d_row_pos, c->d_invfreq, md.dh / 2, c->d_cs);
    float* h = c->d_h;
    int rc = PASS_OK;
    for (int l = 0; l < nl && rc == PASS_OK; l++) {
        float* h_in = t.h_in + (size_t)l * R * d; float* qkv = t.qkv + (size_t)l * R * 3 * d;
        float* attn = t.attn + (size_t)l * R * d; float* h_mid = t.h_mid + (size_t)l * R * d; float* gu = t.gu + (size_t)l * R * t.ng;
        CUDA_TRY(cudaMemcpyAsync(h_in, h, sizeof(float) * R * d, cudaMemcpyDeviceToDevice, c->stream));
        LAUNCH(c, (k_rmsnorm<bf>), R, 256, h, (const bf*)c->norm_attn[l], d, md.eps, t.t0);
        rc = train_gemm(c, c->tm_wq[l], c->tm_wk[l], c->tm_wv[l], dt, false, 3 * d, 3 * dt, d, t.t0, R, qkv);
        if (rc != PASS_OK) break;
        LAUNCH(c, (k_rope_kv<bf>), R, 256, qkv, c->d_cs, c->d_row_seq, c->d_row_pos, md, l, (bf*)c->kv_k, (bf*)c->kv_v);
        if (md.dh == 128)
            LAUNCH(c, (k_attn_simple<bf, 128, false>), dim3(md.H, R), 128, qkv, 3 * d, c->d_row_seq, c->d_row_pos, md, l, (const bf*)c->kv_k, (const bf*)c->kv_v, (void*)attn, 0);
        else
            LAUNCH(c, (k_attn_simple<bf, 64, false>), dim3(md.H, R), 128, qkv, 3 * d, c->d_row_seq, c->d_row_pos, md, l, (const bf*)c->kv_k, (const bf*)c->kv_v, (void*)attn, 0);
        rc = train_gemm1(c, c->tm_wo[l], d, d, attn, R, t.t0);
        if (rc != PASS_OK) break;
        LAUNCH(c, k_add_rows, (R * d + 255) / 256, 256, h, t.t0, (size_t)R * d);
        CUDA_TRY(cudaMemcpyAsync(h_mid, h, sizeof(float) * R * d, cudaMemcpyDeviceToDevice, c->stream));
        LAUNCH(c, (k_rmsnorm<bf>), R, 256, h, (const bf*)c->norm_ffn[l], d, md.eps, t.t0);
        rc = train_gemm(c, c->tm_wg[l], c->tm_wu[l], c->tm_wu[l], 0, true, t.ng, (f + 63) / 64, d, t.t0, R, gu);
        if (rc != PASS_OK) break;
        LAUNCH(c, k_swiglu_il, dim3((f + 255) / 256, R), 256, gu, t.ng, f, t.t0);
        rc = train_gemm1(c, c->tm_wd[l], d, f, t.t0, R, t.t1);
        if (rc != PASS_OK) break;
        LAUNCH(c, k_add_rows, (R * d + 255) / 256, 256, h, t.t1, (size_t)R * d);
    }
    if (rc != PASS_OK) return rc;
    CUDA_TRY(cudaMemcpyAsync(t.h_last, h, sizeof(float) * R * d, cudaMemcpyDeviceToDevice, c->stream));
    LAUNCH(c, (k_rmsnorm<bf>), R, 256, h, (const bf*)c->final_norm, d, md.eps, t.t0);
    rc = train_gemm1(c, c->tm_lm, V, d, t.t0, R, c->d_logits);
    if (rc != PASS_OK) return rc;
    // ---- loss on the look-ahead outputs, gradient with respect to the logits (mean over rows)
    LAUNCH(c, k_ce_grad, R, 256, c->d_logits, t.targets, V, 1.f / (float)R, t.dlogits, t.loss_row);
    // ---- backward over the same rows
    rc = train_gemm1(c, t.tm_lm_t, d, V, t.dlogits, R, t.t0);
    if (rc != PASS_OK) return rc;
    LAUNCH(c, (k_rmsnorm_bwd<bf>), R, 256, t.t0, t.h_last, (const bf*)c->final_norm, d, md.eps, (const float*)nullptr, t.dh);
    for (int l = nl - 1; l >= 0 && rc == PASS_OK; l--) {
        float* h_in = t.h_in + (size_t)l * R * d; float* qkv = t.qkv + (size_t)l * R * 3 * d;
        float* h_mid = t.h_mid + (size_t)l * R * d; float* gu = t.gu + (size_t)l * R * t.ng;
        rc = train_gemm1(c, t.tm_d_t[l], f, d, t.dh, R, t.t0);                       // d act
        if (rc != PASS_OK) break;
        LAUNCH(c, k_swiglu_il_bwd, dim3((f + 255) / 256, R), 256, gu, t.ng, f, t.t0, t.t1);   // [d gate | d up]
        rc = train_gemm1(c, t.tm_gu_t[l], d, 2 * f, t.t1, R, t.t0);                  // d (normalised input of the feed-forward)
        if (rc != PASS_OK) break;
        LAUNCH(c, (k_rmsnorm_bwd<bf>), R, 256, t.t0, h_mid, (const bf*)c->norm_ffn[l], d, md.eps, (const float*)t.dh, t.dh);
        rc = train_gemm1(c, t.tm_o_t[l], d, d, t.dh, R, t.t0);                       // d attention output
        if (rc != PASS_OK) break;
        if (md.dh == 128)
            LAUNCH(c, (k_attn_la_bwd<bf, 128>), dim3(md.H, n_seqs), 128, qkv, t.t0, c->d_states, md, l, L, (const bf*)c->kv_k, (const bf*)c->kv_v, t.scratch, t.n_max, t.t1);
        else
            LAUNCH(c, (k_attn_la_bwd<bf, 64>), dim3(md.H, n_seqs), 128, qkv, t.t0, c->d_states, md, l, L, (const bf*)c->kv_k, (const bf*)c->kv_v, t.scratch, t.n_max, t.t1);
        LAUNCH(c, k_rope_bwd, R, 256, t.t1, c->d_cs, d, md.dh);
        rc = train_gemm1(c, t.tm_qkv_t[l], d, 3 * d, t.t1, R, t.t0);                 // d (normalised input of attention)
        if (rc != PASS_OK) break;
        LAUNCH(c, (k_rmsnorm_bwd<bf>), R, 256, t.t0, h_in, (const bf*)c->norm_attn[l], d, md.eps, (const float*)t.dh, t.dh);
    }
    if (rc != PASS_OK) return rc;
    return PASS_OK;
}

static float train_lr(const pass_train_config& hp, int step) {
    if (hp.warmup_steps > 0 && step < hp.warmup_steps) return hp.lr * (float)(step + 1) / (float)hp.warmup_steps;
    if (step >= hp.total_steps) return 0.f;
    const double prog = (double)(step - hp.warmup_steps) / (double)std::max(1, hp.total_steps - hp.warmup_steps);
    return (float)(0.5 * hp.lr * (1.0 + std::cos(3.14159265358979323846 * prog)));
}

int pass_train_step(pass_ctx* c, const int32_t* tokens, int stride, const int32_t* positions, int n_seqs, int apply_update,
                    float* loss_out) {
    if (!c || !tokens || !positions || !loss_out || n_seqs < 1 || stride < 1) return PASS_ERR_INVALID_ARG;
    pass_ctx::Train& t = c->tr;
    if (!t.ready) return PASS_ERR_STATE;
    if (n_seqs > t.max_seqs) return PASS_ERR_CAPACITY;
    typedef __nv_bfloat16 bf;
    const ModelDims& md = c->md;
    const int L = t.L, R = n_seqs * L, d = md.d, f = md.f, V = md.V, nl = md.n_layers, dt = d / kTileN;
    for (int b = 0; b < n_seqs; b++) {
        const int n = positions[b];
        if (n < 0 || n + 1 + L >= stride) return PASS_ERR_INVALID_ARG;        // the targets w_{n+2} .. w_{n+1+L} must exist
        if (n + 1 + L > md.cap) return PASS_ERR_CAPACITY;
        for (int i = 0; i <= n + 1 + L; i++)
            if (tokens[(size_t)b * stride + i] < 0 || tokens[(size_t)b * stride + i] >= V) return PASS_ERR_INVALID_ARG;
    }
    // the prompt part w_0 .. w_n of every sequence: keys and values into the cache, through the prompt pass
    for (int b = 0; b < n_seqs; b++) {
        const int rc = pass_prefill(c, b, tokens + (size_t)b * stride, positions[b] + 2);
        if (rc != PASS_OK) return rc;
        for (int t_ = 0; t_ < L; t_++) t.pin_targets[b * L + t_] = tokens[(size_t)b * stride + positions[b] + 2 + t_];
    }
    CUDA_TRY(cudaMemcpyAsync(t.targets, t.pin_targets, sizeof(int) * R, cudaMemcpyHostToDevice, c->stream));
    // ---- forward and backward over the look-ahead rows: one CUDA graph per batch size
    int rc = PASS_OK;
    if (c->use_graph) {
        auto it = t.graphs.find(n_seqs);
        if (it == t.graphs.end()) {
            cudaGraph_t g = nullptr;
            CUDA_TRY(cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
            rc = train_enqueue_rows(c, n_seqs);
            const cudaError_t e = cudaStreamEndCapture(c->stream, &g);
            if (rc != PASS_OK || e != cudaSuccess || !g || launch_failed(c)) {
                if (g) cudaGraphDestroy(g);
                return rc != PASS_OK ? rc : PASS_ERR_CUDA;
            }
            cudaGraphExec_t ge = nullptr;
            const cudaError_t e2 = cudaGraphInstantiate(&ge, g, 0);
            cudaGraphDestroy(g);
            if (e2 != cudaSuccess) return PASS_ERR_CUDA;
            it = t.graphs.emplace(n_seqs, ge).first;
        }
        CUDA_TRY(cudaGraphLaunch(it->second, c->stream));
    } else {
        rc = train_enqueue_rows(c, n_seqs);
        if (rc != PASS_OK) return rc;
    }
    // ---- gradient of the look-ahead rows (sum over sequences; the 1 / rows factor is in the loss) and the update
    const float lr = train_lr(t.hp, t.step);
    const float b1 = 1.f - std::pow(t.hp.beta1, (float)(t.step + 1)), b2 = 1.f - std::pow(t.hp.beta2, (float)(t.step + 1));
    LAUNCH(c, k_la_grad_adamw, (L * d + 255) / 256, 256, t.dh, n_seqs, L, d, t.grad, t.master, t.m, t.v, lr, t.hp.beta1,
           t.hp.beta2, t.hp.eps, t.hp.weight_decay, b1, b2, apply_update ? 1 : 0);
    CUDA_TRY(cudaMemcpyAsync(t.pin_loss, t.loss_row, sizeof(float) * R, cudaMemcpyDeviceToHost, c->stream));
    CHECK_LAUNCHES(c);
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    const int st = debug_status(c);
    if (st != PASS_OK) return st;
    double sum = 0.0;
    for (int r = 0; r < R; r++) sum += t.pin_loss[r];
    *loss_out = (float)(sum / R);
    if (apply_update) t.step++;
    return PASS_OK;
}

int pass_train_get(pass_ctx* c, int what, float* dst_host, size_t bytes) {
    if (!c || !dst_host) return PASS_ERR_INVALID_ARG;
    pass_ctx::Train& t = c->tr;
    if (!t.ready) return PASS_ERR_STATE;
    const size_t n = (size_t)t.L * c->md.d * sizeof(float);
    if (bytes < n) return PASS_ERR_CAPACITY;
    const float* src = what == PASS_TRAIN_LA ? t.master : what == PASS_TRAIN_GRAD ? t.grad : nullptr;
    if (!src) return PASS_ERR_INVALID_ARG;
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    CUDA_TRY(cudaMemcpy(dst_host, src, n, cudaMemcpyDeviceToHost));
    return PASS_OK;
}

int pass_train_export(pass_ctx* c, void* la_emb_device) {
    if (!c || !la_emb_device) return PASS_ERR_INVALID_ARG;
    pass_ctx::Train& t = c->tr;
    if (!t.ready) return PASS_ERR_STATE;
    typedef __nv_bfloat16 bf;
    LAUNCH(c, (k_rows_convert<bf>), (t.L * c->md.d + 255) / 256, 256, (const bf*)la_emb_device, t.master, (size_t)t.L * c->md.d, 0);
    CHECK_LAUNCHES(c);
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    return PASS_OK;
}

}  // extern "C"

