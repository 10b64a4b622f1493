// Eq. (1) of the paper: P'(v, t), the probability that v is the first output in the window, emitted at offset t.
// Input: the window's logits [B, W, V+1] (fp32, as written by the joint's store epilogue); output, in place:
// natural-log P'(v, t); optionally the K most probable (label, offset) pairs per utterance (the candidates
// Algorithm 3 expands).  One CTA per utterance.  The work is a streaming pass over the logits, bound by memory
// bandwidth, not a contraction: 2 x (V+1) x 4 bytes per window row (read once, written once; the second read of
// the row during the write pass and the top-K passes hit L2: a window is W x (V+1) x 4 bytes = 32 KB at W = 8).
#include <math_constants.h>

#include "wind_internal.cuh"

namespace wind {

constexpr int FO_THREADS = 256;

__device__ __forceinline__ float fo_warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float fo_warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(FO_THREADS) first_output_kernel(float* __restrict__ logp, const int32_t* __restrict__ enc_len,
                                                                  const int32_t* __restrict__ t0, int W, int NV, int blank, int K,
                                                                  int32_t* __restrict__ top_label, int32_t* __restrict__ top_jump,
                                                                  float* __restrict__ top_logp) {
    __shared__ float s_lse[kMaxWindow], s_before[kMaxWindow];   // log-sum-exp of a row; sum of blank log-probs of the rows before it
    __shared__ float s_best_v[FO_THREADS / 32];
    __shared__ int s_best_i[FO_THREADS / 32];
    __shared__ float s_prev_v;
    __shared__ int s_prev_i;
    const int b = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int n = enc_len[b] - t0[b];
    n = n < 0 ? 0 : (n > W ? W : n);
    float* base = logp + (size_t)b * W * NV;
    // ---- log-sum-exp per row, one warp per row (no block-wide synchronisation inside): maximum, then sum of exponentials ----
    for (int w = warp; w < n; w += FO_THREADS / 32) {
        const float* row = base + (size_t)w * NV;
        float mx = -CUDART_INF_F;
        for (int v = lane; v < NV; v += 32) mx = fmaxf(mx, row[v]);
        mx = fo_warp_max(mx);
        float se = 0.f;
        for (int v = lane; v < NV; v += 32) se += expf(row[v] - mx);
        se = fo_warp_sum(se);
        if (lane == 0) s_lse[w] = mx + logf(se);
    }
    __syncthreads();
    // ---- running sum of the blank log-probabilities (the product over earlier frames in Eq. 1) ----
    if (threadIdx.x == 0) {
        float before = 0.f;
        for (int w = 0; w < n; ++w) {
            s_before[w] = before;
            before += base[(size_t)w * NV + blank] - s_lse[w];
        }
    }
    __syncthreads();
    // ---- log P'(v, t) in place, one warp per row ----
    for (int w = warp; w < n; w += FO_THREADS / 32) {
        float* row = base + (size_t)w * NV;
        const float shift = s_before[w] - s_lse[w];
        for (int v = lane; v < NV; v += 32) {
            const float x = row[v] + shift;
            row[v] = (v == blank && w != n - 1) ? -CUDART_INF_F : x;
        }
    }
    if (K <= 0) return;
    __syncthreads();   // the block's own writes above are read below
    // ---- the K most probable (label, offset) pairs, best first; equal values in order of (offset, label) ----
    if (threadIdx.x == 0) { s_prev_v = CUDART_INF_F; s_prev_i = -1; }
    __syncthreads();
    const int total = n * NV;
    constexpr int KLOC = 8;
    if (K <= KLOC) {
        // one pass over the window: every thread keeps the K best of its own elements (sorted, best first), then K
        // rounds pick the best of the threads' current heads; the winning thread moves on to its next one
        float lv[KLOC];
        int li[KLOC];
#pragma unroll
        for (int j = 0; j < KLOC; ++j) { lv[j] = -CUDART_INF_F; li[j] = 0x7fffffff; }
        for (int i = threadIdx.x; i < total; i += FO_THREADS) {
            float x = base[i];
            int xi = i;
            if (x > -CUDART_INF_F) {
#pragma unroll
                for (int j = 0; j < KLOC; ++j) {
                    // i ascends, so on equal values the earlier element stays ahead
                    if (j < K && x > lv[j]) {
                        const float tv = lv[j]; const int ti = li[j];
                        lv[j] = x; li[j] = xi;
                        x = tv; xi = ti;
                    }
                }
            }
        }
        for (int k = 0; k < K; ++k) {
            float bv = lv[0];
            int bi = li[0];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            if (lane == 0) { s_best_v[warp] = bv; s_best_i[warp] = bi; }
            __syncthreads();
            bv = s_best_v[0]; bi = s_best_i[0];
#pragma unroll
            for (int q = 1; q < FO_THREADS / 32; ++q) {
                const float ov = s_best_v[q];
                const int oi = s_best_i[q];
                if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            const bool any = bv > -CUDART_INF_F;
            if (any && li[0] == bi) {   // this thread's head was taken: shift its list
#pragma unroll
                for (int j = 0; j < KLOC - 1; ++j) { lv[j] = lv[j + 1]; li[j] = li[j + 1]; }
                lv[KLOC - 1] = -CUDART_INF_F; li[KLOC - 1] = 0x7fffffff;
            }
            if (threadIdx.x == 0) {
                const int off = any ? bi / NV : -1;
                top_label[(size_t)b * K + k] = any ? bi - off * NV : -1;
                top_jump[(size_t)b * K + k] = off;
                top_logp[(size_t)b * K + k] = any ? bv : -CUDART_INF_F;
            }
            __syncthreads();
        }
        return;
    }
    for (int k = 0; k < K; ++k) {
        const float pv = s_prev_v;
        const int pi = s_prev_i;
        float bv = -CUDART_INF_F;
        int bi = -1;
        for (int i = threadIdx.x; i < total; i += FO_THREADS) {
            const float x = base[i];
            const bool after_prev = x < pv || (x == pv && i > pi);   // not yet taken
            if (after_prev && x > -CUDART_INF_F && (bi < 0 || x > bv)) { bv = x; bi = i; }   // i ascends: first of equals stays
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (oi >= 0 && (bi < 0 || ov > bv || (ov == bv && oi < bi))) { bv = ov; bi = oi; }
        }
        if (lane == 0) { s_best_v[warp] = bv; s_best_i[warp] = bi; }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int q = 1; q < FO_THREADS / 32; ++q) {
                const float ov = s_best_v[q];
                const int oi = s_best_i[q];
                if (oi >= 0 && (bi < 0 || ov > bv || (ov == bv && oi < bi))) { bv = ov; bi = oi; }
            }
            const int off = bi >= 0 ? bi / NV : -1;
            top_label[(size_t)b * K + k] = bi >= 0 ? bi - off * NV : -1;
            top_jump[(size_t)b * K + k] = off;
            top_logp[(size_t)b * K + k] = bi >= 0 ? bv : -CUDART_INF_F;
            if (bi >= 0) { s_prev_v = bv; s_prev_i = bi; }
            else { s_prev_v = -CUDART_INF_F; s_prev_i = 0x7fffffff; }   // nothing left
        }
        __syncthreads();
    }
}

cudaError_t launch_first_output(float* logp, const int32_t* enc_len, const int32_t* t0, int B, int W, int NV, int blank, int K,
                                int32_t* top_label, int32_t* top_jump, float* top_logp, cudaStream_t stream) {
    first_output_kernel<<<B, FO_THREADS, 0, stream>>>(logp, enc_len, t0, W, NV, blank, K, top_label, top_jump, top_logp);
    return cudaGetLastError();
}

}  // namespace wind
