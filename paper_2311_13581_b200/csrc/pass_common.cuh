// Shared device-side declarations of the PaSS step library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/pass.h"

namespace pass {

constexpr int kMaxLA = PASS_MAX_LOOKAHEAD;          // 8
constexpr int kMaxRows = PASS_MAX_ROWS;             // 128: rows of one step or one pass_forward_tokens call
constexpr int kRowsCap = 2048;                      // rows of one launch at most (a prompt chunk): row tables, strides
constexpr int kUSlots = 2 * kMaxLA + 1;             // uniforms per sequence and step
constexpr int kVerifySplits = 8;                    // CTAs per logits row in the stats kernel
constexpr int kVerifyThreads = 256;
constexpr int kChunks = kVerifySplits * kVerifyThreads;   // CDF chunks per row

// Status bits written by kernels, read by the host after a step.
constexpr int kStatusNonFinite = 1;
constexpr int kStatusTimeout = 2;
constexpr int kStatusBadState = 4;

// Per-sequence decoding state, resident on the device so that a captured step can be
// replayed unchanged (Algorithm 1 bookkeeping: n, the pending token, the drafts).
struct SeqState {
    int kv_len;        // cached positions
    int pending;       // last emitted token, not yet in the cache
    int has_pending;   // 0 before prefill
    int m;             // pending drafts: 0 or k
    int q_sel;         // which half of the draft-law store holds the laws of the drafts
    int drafts[kMaxLA];
    // result of the last step
    int n_out;
    int n_acc;
    int out_tokens[kMaxLA + 1];
    int pad_[2];
};

// Inputs of one step, copied in before the graph launch.
struct StepParams {
    float temperature;
    int k;
    int drop_drafts;   // k, temperature or top_k changed: pending drafts are void
    int top_k;         // > 0: every law is the softmax over the top_k largest logits of its row only
    int validate_only; // 1: validation call of the two-call schedule - the look-ahead rows' outputs are not used
    int pad_[3];
    // followed by float u[max_batch][kUSlots]
};

struct ModelDims {
    int n_layers, d, H, dh, f, V;
    int k_max, B, cap;
    int dtype;
    float eps, theta;
};

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) {
    return __bfloat162float(v);
}
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
    return __float2bfloat16_rn(v);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// KV cache layout, the same for K and V: [layer][seq][head][position][d_head].
// Contiguous per head so that one CTA streams its head's keys as one run.
__host__ __device__ __forceinline__ size_t kv_index(const ModelDims& md, int layer, int seq, int head,
                                                    int pos) {
    return ((((size_t)layer * md.B + seq) * md.H + head) * (size_t)md.cap + pos) * md.dh;
}

}  // namespace pass
