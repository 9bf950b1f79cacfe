// Speculative-sampling verify of the PaSS step (Algorithm 1, validation phase; the same rule
// as Algorithm 2): temperature softmax of the target rows and of the look-ahead rows, accept
// tests against the stored draft laws, residual resample or extra token, next drafts, and the
// commit / rollback of the sequence state.  All probabilities are float64 on the device so
// that decisions agree with a float64 reading of the same logits.
//
// Two kernels:
//   k_verify_stats  - grid (rows, kVerifySplits): e_i = exp((z_i - max z)/T) per row, written
//                     out together with per-chunk sums (chunks in vocabulary order, so that a
//                     prefix over chunks is a CDF); look-ahead rows are also copied into the
//                     other half of the draft-law store.
//   k_verify_decide - grid (batch): the sequential accept loop on scalars, one inverse-CDF
//                     search for the final token, k searches for the next drafts, state update.
#pragma once
#include "pass_common.cuh"

namespace pass {

struct VerifyBufs {
    const float* logits;      // [rows][V]
    double* E;                // [rows][V]      exp((z - max)/T) of the current rows
    double* chunk;            // [rows][kChunks] per-chunk sums of E
    double* row_sum;          // [rows][kVerifySplits] per-split sums (fixed-order partials)
    float* row_max;           // [rows]
    float* amax_val;          // [rows][kVerifySplits]   greedy: per-split maximum
    int* amax_idx;            // [rows][kVerifySplits]   and its first index
    // draft-law store, two halves per sequence: [B][2][k_max]...
    float* q_logits;          // [B][2][k_max][V]
    double* q_E;              // [B][2][k_max][V]
    double* q_sum;            // [B][2][k_max][kVerifySplits]
    int* status;
};

__device__ __forceinline__ double block_sum_256(double v, double* sh) {
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0) {
        for (int w = 0; w < (int)(blockDim.x >> 5); w++) t += sh[w];
        sh[0] = t;
    }
    __syncthreads();
    t = sh[0];
    __syncthreads();
    return t;
}

// Elements of a row are cut into kChunks contiguous chunks of `cl` elements; chunk c belongs to
// split c / kVerifyThreads, thread c % kVerifyThreads.
__global__ void __launch_bounds__(kVerifyThreads)
k_verify_stats(VerifyBufs vb, const SeqState* __restrict__ states,
               const StepParams* __restrict__ sp, int M, int V, int k_max) {
    __shared__ double sh[8];
    __shared__ float shf[8];
    __shared__ int shi[8];
    const int r = blockIdx.x, split = blockIdx.y, b = r / M, i = r % M;
    const int k = sp->k;
    const SeqState& st = states[b];
    const int m = (sp->drop_drafts || st.m != k) ? 0 : st.m;
    if (i > m + k) return;                                   // pad row
    const float T = sp->temperature;
    const float* z = vb.logits + (size_t)r * V;
    const int cl = (V + kChunks - 1) / kChunks;
    const int c = split * kVerifyThreads + threadIdx.x;
    const int lo = min(c * cl, V), hi = min(lo + cl, V);
    const bool la_row = i > m;                               // candidate law of the next drafts
    const int t = i - m - 1;
    const size_t qrow = (((size_t)b * 2 + (st.q_sel ^ 1)) * k_max + (la_row ? t : 0));

    bool bad = false;
    if (T == 0.f) {
        // greedy: first argmax of this split's range
        float bv = -INFINITY;
        int bi = V;
        for (int e = lo; e < hi; e++) {
            const float v = z[e];
            bad |= !isfinite(v);
            if (v > bv) { bv = v; bi = e; }
            if (la_row) vb.q_logits[qrow * V + e] = v;
        }
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if ((threadIdx.x & 31) == 0) { shf[threadIdx.x >> 5] = bv; shi[threadIdx.x >> 5] = bi; }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < 8; w++)
                if (shf[w] > bv || (shf[w] == bv && shi[w] < bi)) { bv = shf[w]; bi = shi[w]; }
            vb.amax_val[r * kVerifySplits + split] = bv;
            vb.amax_idx[r * kVerifySplits + split] = bi;
        }
    } else {
        // every split needs the row maximum: each computes it over the whole row (L2 reads)
        float mx = -INFINITY;
        for (int e = threadIdx.x; e < V; e += kVerifyThreads) {
            const float v = z[e];
            bad |= !isfinite(v);
            mx = fmaxf(mx, v);
        }
        mx = warp_max(mx);
        if ((threadIdx.x & 31) == 0) shf[threadIdx.x >> 5] = mx;
        __syncthreads();
        mx = shf[0];
        for (int w = 1; w < 8; w++) mx = fmaxf(mx, shf[w]);
        // Top-k sampling (Experiments, setup): the law keeps the top_k largest logits of the row, equal
        // values ranked by index.  (thr, thr_idx) is the last kept element in that order, found by top_k
        // rounds of "largest element after the previous one"; every split of the row finds it for itself.
        float thr = -INFINITY;
        int thr_idx = V;                                     // keeps everything
        const int top_k = sp->top_k;
        if (top_k > 0 && top_k < V) {
            float lv = INFINITY;
            int li = -1;
            for (int it = 0; it < top_k; it++) {
                float bv = -INFINITY;
                int bi = V;
                for (int e = threadIdx.x; e < V; e += kVerifyThreads) {
                    const float v = z[e];
                    const bool after = v < lv || (v == lv && e > li);
                    if (after && (v > bv || (v == bv && e < bi))) { bv = v; bi = e; }
                }
                for (int o = 16; o > 0; o >>= 1) {
                    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
                }
                __syncthreads();                             // shf / shi free
                if ((threadIdx.x & 31) == 0) { shf[threadIdx.x >> 5] = bv; shi[threadIdx.x >> 5] = bi; }
                __syncthreads();
                bv = shf[0];
                bi = shi[0];
                for (int w = 1; w < 8; w++)
                    if (shf[w] > bv || (shf[w] == bv && shi[w] < bi)) { bv = shf[w]; bi = shi[w]; }
                lv = bv;
                li = bi;
            }
            thr = lv;
            thr_idx = li;
        }
        const double invT = 1.0 / (double)T;
        double cs = 0.0;
        for (int e = lo; e < hi; e++) {
            const float v = z[e];
            const bool keep = v > thr || (v == thr && e <= thr_idx);
            const double ev = keep ? exp(((double)v - (double)mx) * invT) : 0.0;
            vb.E[(size_t)r * V + e] = ev;
            if (la_row) { vb.q_logits[qrow * V + e] = v; vb.q_E[qrow * V + e] = ev; }
            cs += ev;
        }
        vb.chunk[(size_t)r * kChunks + c] = cs;
        // per-split sum in a fixed order: warp tree, then warps in order
        const double tot = block_sum_256(cs, sh);
        if (threadIdx.x == 0) {
            vb.row_sum[r * kVerifySplits + split] = tot;
            if (split == 0) vb.row_max[r] = mx;
            if (la_row) vb.q_sum[qrow * kVerifySplits + split] = tot;
        }
    }
    if (bad) atomicOr(vb.status, kStatusNonFinite);
}

// Inverse CDF over chunked weights: smallest index i with w_0 + .. + w_i > u * total.
// `csum` are the chunk sums of this block's threads (kChunks / blockDim.x chunks per thread,
// consecutive), weight(i) gives w_i.  Returns the index to every thread.
template <typename WeightFn>
__device__ int block_invcdf(const double* __restrict__ chunk_sums, int V, double u, WeightFn weight,
                            double* sh_d, int* sh_i) {
    constexpr int CPT = kChunks / 1024;                     // chunks per thread
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cl = (V + kChunks - 1) / kChunks;
    double mine[CPT], tsum = 0.0;
#pragma unroll
    for (int j = 0; j < CPT; j++) { mine[j] = chunk_sums[tid * CPT + j]; tsum += mine[j]; }
    // inclusive scan over threads
    double inc = tsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) sh_d[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        double w = sh_d[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double n = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += n;
        }
        sh_d[32 + lane] = w;                                 // inclusive over warps
    }
    if (tid == 0) sh_i[0] = 1024;
    __syncthreads();
    const double total = sh_d[32 + 31];
    const double woff = warp ? sh_d[32 + warp - 1] : 0.0;
    const double incl = woff + inc, excl = incl - tsum;
    const double target = u * total;
    if (incl > target && tsum > 0.0) atomicMin(&sh_i[0], tid);
    __syncthreads();
    const int owner = sh_i[0];
    __syncthreads();
    if (owner == 1024) {
        // rounding left no crossing: last index with positive weight
        int last = -1;
        for (int e = min((tid + 1) * CPT * cl, V) - 1; e >= tid * CPT * cl; e--)
            if (weight(e) > 0.0) { last = e; break; }
        if (tid == 0) sh_i[1] = -1;
        __syncthreads();
        atomicMax(&sh_i[1], last);
        __syncthreads();
        const int res = max(sh_i[1], 0);
        __syncthreads();
        return res;
    }
    if (tid == owner) {
        double c = excl;
        int res = -1, lastpos = -1;
        const int lo = min(tid * CPT * cl, V), hi = min(lo + CPT * cl, V);
        for (int e = lo; e < hi; e++) {
            const double w = weight(e);
            if (w > 0.0) lastpos = e;
            c += w;
            if (c > target) { res = e; break; }
        }
        sh_i[1] = res >= 0 ? res : max(lastpos, lo);
    }
    __syncthreads();
    const int res = sh_i[1];
    __syncthreads();
    return res;
}

__global__ void __launch_bounds__(1024)
k_verify_decide(VerifyBufs vb, SeqState* __restrict__ states, const StepParams* __restrict__ sp,
                const float* __restrict__ uniforms, int M, int V, int k_max,
                double* __restrict__ scratch /* [B][kChunks] */) {
    __shared__ double sh_d[64];
    __shared__ int sh_i[4];
    __shared__ int s_a;
    __shared__ int s_arg[2 * kMaxLA + 1];
    const int b = blockIdx.x, tid = threadIdx.x;
    SeqState& st = states[b];
    const int k = sp->k;
    const float T = sp->temperature;
    const int m = (sp->drop_drafts || st.m != k) ? 0 : st.m;
    const float* u = uniforms + (size_t)b * kUSlots;
    const int r0 = b * M;
    if (*vb.status != 0) {                                   // leave the sequence untouched
        if (tid == 0) { st.n_out = 0; st.n_acc = 0; }
        return;
    }
    const size_t qbase = ((size_t)b * 2 + st.q_sel) * k_max;        // laws of the pending drafts
    const size_t qnext = ((size_t)b * 2 + (st.q_sel ^ 1)) * k_max;  // laws of the next drafts

    if (T == 0.f) {
        // greedy: one-hot laws.  Draft j is accepted iff it is the argmax of target row j-1;
        // the final token is the argmax of the first row that disagrees (or of row m).
        if (tid < 1 + m + k) {
            const int r = r0 + tid;
            float bv = vb.amax_val[r * kVerifySplits];
            int bi = vb.amax_idx[r * kVerifySplits];
            for (int s = 1; s < kVerifySplits; s++) {
                const float v = vb.amax_val[r * kVerifySplits + s];
                const int ix = vb.amax_idx[r * kVerifySplits + s];
                if (v > bv || (v == bv && ix < bi)) { bv = v; bi = ix; }
            }
            s_arg[tid] = bi;
        }
        __syncthreads();
        if (tid == 0) {
            int a = 0;
            while (a < m && st.drafts[a] == s_arg[a]) a++;
            const int y = s_arg[a];
            for (int j = 0; j < a; j++) st.out_tokens[j] = st.drafts[j];
            st.out_tokens[a] = y;
            st.n_out = a + 1;
            st.n_acc = a;
            st.kv_len += a + 1;
            st.pending = y;
            if (a == m && k > 0 && !sp->validate_only) {
                for (int t = 0; t < k; t++) st.drafts[t] = s_arg[m + 1 + t];
                st.m = k;
                st.q_sel ^= 1;
            } else {
                st.m = 0;
            }
        }
        return;
    }

    // totals of the target rows and of the stored draft laws, summed in a fixed order
    auto total_of = [&](const double* parts) {
        double t = 0.0;
        for (int s = 0; s < kVerifySplits; s++) t += parts[s];
        return t;
    };
    if (tid == 0) {
        int a = 0;
        for (; a < m; a++) {
            const int dj = st.drafts[a];
            const double p = vb.E[(size_t)(r0 + a) * V + dj] / total_of(vb.row_sum + (r0 + a) * kVerifySplits);
            const double q = vb.q_E[(qbase + a) * V + dj] / total_of(vb.q_sum + (qbase + a) * kVerifySplits);
            const double ratio = p / q;
            if (!((double)u[a] < fmin(1.0, ratio))) break;
        }
        s_a = a;
    }
    __syncthreads();
    const int a = s_a;
    int y;
    if (a < m) {
        // residual law max(0, P_tgt,a - Q_dft,a+1): chunk sums first, then the search
        const double* Ep = vb.E + (size_t)(r0 + a) * V;
        const double* Eq = vb.q_E + (qbase + a) * V;
        const double ip = 1.0 / total_of(vb.row_sum + (r0 + a) * kVerifySplits);
        const double iq = 1.0 / total_of(vb.q_sum + (qbase + a) * kVerifySplits);
        auto wres = [&](int e) { return fmax(0.0, Ep[e] * ip - Eq[e] * iq); };
        constexpr int CPT = kChunks / 1024;
        const int cl = (V + kChunks - 1) / kChunks;
        double* cs = scratch + (size_t)b * kChunks;
        double any = 0.0;
        for (int j = 0; j < CPT; j++) {
            const int c = tid * CPT + j;
            const int lo = min(c * cl, V), hi = min(lo + cl, V);
            double s = 0.0;
            for (int e = lo; e < hi; e++) s += wres(e);
            cs[c] = s;
            any += s;
        }
        // no residual mass at all (laws coincide): fall back to the target law
        __syncthreads();
        double tot = warp_sum(any);
        if ((tid & 31) == 0) sh_d[tid >> 5] = tot;
        __syncthreads();
        tot = 0.0;
        for (int w = 0; w < 32; w++) tot += sh_d[w];
        __syncthreads();
        if (tot > 0.0) {
            y = block_invcdf(cs, V, (double)u[k], wres, sh_d, sh_i);
        } else {
            auto wp = [&](int e) { return Ep[e]; };
            y = block_invcdf(vb.chunk + (size_t)(r0 + a) * kChunks, V, (double)u[k], wp, sh_d, sh_i);
        }
    } else {
        const double* Ep = vb.E + (size_t)(r0 + m) * V;
        auto wp = [&](int e) { return Ep[e]; };
        y = block_invcdf(vb.chunk + (size_t)(r0 + m) * kChunks, V, (double)u[k], wp, sh_d, sh_i);
    }
    int nd[kMaxLA];
    if (a == m && !sp->validate_only) {
        for (int t = 0; t < k; t++) {
            const double* Eq = vb.E + (size_t)(r0 + m + 1 + t) * V;
            auto wq = [&](int e) { return Eq[e]; };
            nd[t] = block_invcdf(vb.chunk + (size_t)(r0 + m + 1 + t) * kChunks, V,
                                 (double)u[k + 1 + t], wq, sh_d, sh_i);
        }
    }
    if (tid == 0) {
        for (int j = 0; j < a; j++) st.out_tokens[j] = st.drafts[j];
        st.out_tokens[a] = y;
        st.n_out = a + 1;
        st.n_acc = a;
        st.kv_len += a + 1;
        st.pending = y;
        if (a == m && k > 0 && !sp->validate_only) {
            for (int t = 0; t < k; t++) st.drafts[t] = nd[t];
            st.m = k;
            st.q_sel ^= 1;
        } else {
            st.m = 0;
        }
    }
    (void)qnext;
}

}  // namespace pass
