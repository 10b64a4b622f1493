// Plain-ALU (FFMA) kernels: the fp32 path, and the bf16 path for shapes the tensor-core
// kernels do not take.  On the bf16 path the operands are rounded where the tensor path
// rounds them (enc_proj, the joint's activation output and the LSTM's h input go through
// bf16), so both kernel sets compute the same quantities.
#include "wind_internal.cuh"

namespace wind {

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

template <typename T> __device__ __forceinline__ float round_like(float x);
template <> __device__ __forceinline__ float round_like<float>(float x) { return x; }
template <> __device__ __forceinline__ float round_like<__nv_bfloat16>(float x) {
    return __bfloat162float(__float2bfloat16_rn(x));
}
template <typename T> __device__ __forceinline__ void stf(T* p, float x);
template <> __device__ __forceinline__ void stf<float>(float* p, float x) { *p = x; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// n consecutive weights (n a multiple of 8, src 16-byte aligned) into shared memory as floats, 16 bytes per load
__device__ __forceinline__ void load8(const __nv_bfloat16* src, float* dst) {
    const uint4 v = *reinterpret_cast<const uint4*>(src);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(h[i]);
        dst[2 * i] = f.x;
        dst[2 * i + 1] = f.y;
    }
}
__device__ __forceinline__ void load8(const float* src, float* dst) {
    const float4 a = reinterpret_cast<const float4*>(src)[0], b = reinterpret_cast<const float4*>(src)[1];
    dst[0] = a.x; dst[1] = a.y; dst[2] = a.z; dst[3] = a.w; dst[4] = b.x; dst[5] = b.y; dst[6] = b.z; dst[7] = b.w;
}
template <typename T> __device__ __forceinline__ bool aligned_rows(const T* p, int row_elems) {
    return reinterpret_cast<uintptr_t>(p) % 32 == 0 && row_elems % 8 == 0;   // every row then starts on a 16-byte boundary (fp32: 32)
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---------------------------------------------------------------------------
// enc_proj[r, :] = enc[r, :] . W_enc^T + b_enc for valid rows r = b*T + t, t < len[b]
// 64x64 output tile, 16x16 threads, 4x4 outputs each, K tiles of 16.
// ---------------------------------------------------------------------------
template <typename TW>
__global__ void __launch_bounds__(256) enc_proj_simt_kernel(const TW* __restrict__ enc, const int32_t* __restrict__ enc_len,
                                                            const TW* __restrict__ w_enc, const float* __restrict__ b_enc,
                                                            TW* __restrict__ enc_proj, int B, int T, int D, int H) {
    __shared__ float As[16][65];
    __shared__ float Bs[16][65];
    const long long rows = (long long)B * T;
    const long long r0 = (long long)blockIdx.x * 64;
    const int h0 = blockIdx.y * 64;
    // skip tiles without a valid row
    {
        long long rl = r0 + 63 < rows ? r0 + 63 : rows - 1;
        int b0 = (int)(r0 / T), b1 = (int)(rl / T);
        bool any = false;
        for (int b = b0; b <= b1; ++b) {
            long long first = (long long)b * T > r0 ? (long long)b * T : r0;
            if (first <= rl && first - (long long)b * T < enc_len[b]) any = true;
        }
        if (!any) return;
    }
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < D; k0 += 16) {
        for (int e = threadIdx.x; e < 64 * 16; e += 256) {
            int rr = e >> 4, kk = e & 15;
            long long r = r0 + rr;
            float v = 0.f;
            if (r < rows && k0 + kk < D) {
                int b = (int)(r / T);
                int t = (int)(r - (long long)b * T);
                if (t < enc_len[b]) v = ldf(enc + r * D + k0 + kk);
            }
            As[kk][rr] = v;
            int hh = h0 + rr;
            Bs[kk][rr] = (hh < H && k0 + kk < D) ? ldf(w_enc + (size_t)hh * D + k0 + kk) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        long long r = r0 + ty * 4 + i;
        if (r >= rows) continue;
        int b = (int)(r / T);
        int t = (int)(r - (long long)b * T);
        if (t >= enc_len[b]) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int hh = h0 + tx * 4 + j;
            if (hh < H) stf(enc_proj + r * H + hh, acc[i][j] + b_enc[hh]);
        }
    }
}

cudaError_t simt_enc_proj(const Call& c) {
    long long rows = (long long)c.B * c.T;
    dim3 grid((unsigned)((rows + 63) / 64), (unsigned)((c.m.H + 63) / 64));
    if (rows == 0) return cudaSuccess;
    if (c.m.dtype == WIND_DT_BF16)
        enc_proj_simt_kernel<__nv_bfloat16><<<grid, 256, 0, c.stream>>>(
            (const __nv_bfloat16*)c.enc, c.enc_len, (const __nv_bfloat16*)c.m.w_enc, c.m.b_enc,
            (__nv_bfloat16*)c.enc_proj(), c.B, c.T, c.m.D, c.m.H);
    else
        enc_proj_simt_kernel<float><<<grid, 256, 0, c.stream>>>((const float*)c.enc, c.enc_len, (const float*)c.m.w_enc,
                                                                  c.m.b_enc, (float*)c.enc_proj(), c.B, c.T, c.m.D, c.m.H);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// One LSTM layer for all utterances; block j owns hidden unit j (its 4 gate rows).
// x = emb[emit_tok[b]] (layer 0) or the new h of the layer below; utterances with
// emit_tok[b] < 0 keep their state (h copied to the other parity buffer).
// ---------------------------------------------------------------------------
template <typename TW>
__global__ void __launch_bounds__(128) lstm_layer_simt_kernel(const Ctrl* __restrict__ ctrl, const int32_t* __restrict__ emit_tok,
                                                              const TW* __restrict__ emb, const float* __restrict__ x_below,
                                                              const TW* __restrict__ w_ih, const TW* __restrict__ w_hh,
                                                              const float* __restrict__ b_ih, const float* __restrict__ b_hh,
                                                              const float* __restrict__ h_in, float* __restrict__ h_out,
                                                              float* __restrict__ c_state, int B, int n_in, int P) {
    if (ctrl->active == 0) return;
    extern __shared__ float sm[];  // 4 rows x (n_in + P)
    const int j = blockIdx.x;
    const int K = n_in + P;
    if (aligned_rows(w_ih, n_in) && aligned_rows(w_hh, P)) {
        // eight weights per load (a chunk never straddles a row or the boundary between the two matrices)
        for (int c8 = threadIdx.x; c8 < 4 * K / 8; c8 += blockDim.x) {
            const int e = 8 * c8, g = e / K, k = e - g * K;
            const size_t row = (size_t)g * P + j;
            load8(k < n_in ? w_ih + row * n_in + k : w_hh + row * P + (k - n_in), sm + e);
        }
    } else {
        for (int e = threadIdx.x; e < 4 * K; e += blockDim.x) {
            int g = e / K, k = e - g * K;
            size_t row = (size_t)g * P + j;
            sm[e] = (k < n_in) ? ldf(w_ih + row * n_in + k) : ldf(w_hh + row * P + (k - n_in));
        }
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    float bias[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) bias[g] = b_ih[g * P + j] + b_hh[g * P + j];
    for (int b = warp; b < B; b += nw) {
        const int tok = emit_tok[b];
        const float* hb = h_in + (size_t)b * P;
        if (tok < 0) {
            if (lane == 0) h_out[(size_t)b * P + j] = hb[j];
            continue;
        }
        float a[4] = {0.f, 0.f, 0.f, 0.f};
        for (int k = lane; k < K; k += 32) {
            float x;
            if (k < n_in)
                x = x_below ? round_like<TW>(x_below[(size_t)b * P + k]) : ldf(emb + (size_t)tok * n_in + k);
            else
                x = round_like<TW>(hb[k - n_in]);
#pragma unroll
            for (int g = 0; g < 4; ++g) a[g] = fmaf(sm[g * K + k], x, a[g]);
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) a[g] = warp_sum(a[g]);
        if (lane == 0) {
            float gi = 1.f / (1.f + expf(-(a[0] + bias[0])));
            float gf = 1.f / (1.f + expf(-(a[1] + bias[1])));
            float gg = tanhf(a[2] + bias[2]);
            float go = 1.f / (1.f + expf(-(a[3] + bias[3])));
            float cc = gf * c_state[(size_t)b * P + j] + gi * gg;
            c_state[(size_t)b * P + j] = cc;
            h_out[(size_t)b * P + j] = go * tanhf(cc);
        }
    }
}

// pred_proj[b, o] = W_pred[o, :] . h_top[b, :] + b_pred[o]; block o owns output o.
template <typename TW>
__global__ void __launch_bounds__(128) pred_proj_simt_kernel(const Ctrl* __restrict__ ctrl, const TW* __restrict__ w_pred,
                                                             const float* __restrict__ b_pred, const float* __restrict__ h_top,
                                                             float* __restrict__ pred_proj, int B, int P, int H) {
    if (ctrl->active == 0) return;
    extern __shared__ float sm[];
    const int o = blockIdx.x;
    for (int k = threadIdx.x; k < P; k += blockDim.x) sm[k] = ldf(w_pred + (size_t)o * P + k);
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    for (int b = warp; b < B; b += nw) {
        float a = 0.f;
        for (int k = lane; k < P; k += 32) a = fmaf(sm[k], round_like<TW>(h_top[(size_t)b * P + k]), a);
        a = warp_sum(a);
        if (lane == 0) pred_proj[(size_t)b * H + o] = a + b_pred[o];
    }
}

template <typename TW>
static cudaError_t simt_pred_step_t(const Call& c, int parity_in) {
    const int P = c.m.P, B = c.B;
    for (int l = 0; l < c.m.L; ++l) {
        const int n_in = l == 0 ? c.m.E : P;
        const float* x_below = l == 0 ? nullptr : c.h(1 - parity_in) + (size_t)(l - 1) * B * P;
        size_t smem = sizeof(float) * 4 * (size_t)(n_in + P);
        if (smem > 48 * 1024)
            cudaFuncSetAttribute(lstm_layer_simt_kernel<TW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        lstm_layer_simt_kernel<TW><<<P, 128, smem, c.stream>>>(
            c.ctrl(), c.emit_tok(), (const TW*)c.m.emb, x_below, (const TW*)c.w_ih[l], (const TW*)c.w_hh[l], c.b_ih[l],
            c.b_hh[l], c.h(parity_in) + (size_t)l * B * P, c.h(1 - parity_in) + (size_t)l * B * P,
            c.c() + (size_t)l * B * P, B, n_in, P);
    }
    pred_proj_simt_kernel<TW><<<c.m.H, 128, sizeof(float) * P, c.stream>>>(
        c.ctrl(), (const TW*)c.m.w_pred, c.m.b_pred, c.h(1 - parity_in) + (size_t)(c.m.L - 1) * B * P, c.pred_proj(), B, P,
        c.m.H);
    return cudaGetLastError();
}

cudaError_t simt_pred_step(const Call& c, int parity_in) {
    return c.m.dtype == WIND_DT_BF16 ? simt_pred_step_t<__nv_bfloat16>(c, parity_in) : simt_pred_step_t<float>(c, parity_in);
}
int simt_pred_launches(const Call& c) { return c.m.L + 1; }

// ---------------------------------------------------------------------------
// Windowed joint for one utterance per block: z[w] = act(enc_proj[b, t+w] + pred_proj[b]),
// logits[w, v] = W_out[v] . z[w] + b_out[v]; per-row argmax key (or the logits themselves).
// Rows are taken in chunks of 8 so the activation tile stays small.
// ---------------------------------------------------------------------------
//
// WG (window-based greedy decoding): besides the row maximum over the non-blank labels the block gathers each
// row's log-sum-exp and blank logit, picks the most probable (label, offset) pair of Eq. (1) (or "all blank") once
// every row is done, and writes the keys in the form the control step reads: the chosen row carries its label, every
// other row the blank, so that "first non-blank row" is the chosen pair.
template <typename TW, bool WG>
__global__ void __launch_bounds__(256) joint_simt_kernel(const Ctrl* __restrict__ ctrl, const int32_t* __restrict__ t_cur,
                                                         const int32_t* __restrict__ enc_len, const TW* __restrict__ enc_proj,
                                                         const float* __restrict__ pred_proj, const TW* __restrict__ w_out,
                                                         const float* __restrict__ b_out, unsigned long long* __restrict__ keys,
                                                         float* __restrict__ logits_out, int T, int W, int H, int NV, int act,
                                                         int blank) {
    if (ctrl->active == 0) return;
    extern __shared__ float z[];  // [8][H]
    __shared__ unsigned long long skey[8];
    // window mode: per-warp running (maximum, sum of exponentials) of the chunk's rows; per-row results of the window
    __shared__ float s_m[8][8], s_s[8][8];
    __shared__ float s_lse[kMaxWindow], s_blank[kMaxWindow];
    __shared__ unsigned long long s_best[kMaxWindow];
    const int b = blockIdx.x;
    const int t = t_cur[b], len = enc_len[b];
    if (t >= len) return;
    const int n = min(W, len - t);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    for (int w0 = 0; w0 < n; w0 += 8) {
        const int nc = min(8, n - w0);
        __syncthreads();
        if (threadIdx.x < 8) skey[threadIdx.x] = 0ull;
        for (int e = threadIdx.x; e < nc * H; e += blockDim.x) {
            int w = e / H, k = e - w * H;
            float s = ldf(enc_proj + ((size_t)b * T + t + w0 + w) * H + k) + pred_proj[(size_t)b * H + k];
            s = act == WIND_ACT_RELU ? fmaxf(s, 0.f) : tanhf(s);
            z[e] = round_like<TW>(s);
        }
        __syncthreads();
        float run_m[8], run_s[8];
#pragma unroll
        for (int w = 0; w < 8; ++w) { run_m[w] = -INFINITY; run_s[w] = 0.f; }
        for (int v = warp; v < NV; v += nw) {
            float a[8];
#pragma unroll
            for (int w = 0; w < 8; ++w) a[w] = 0.f;
            for (int k = lane; k < H; k += 32) {
                float wv = ldf(w_out + (size_t)v * H + k);
#pragma unroll
                for (int w = 0; w < 8; ++w)
                    if (w < nc) a[w] = fmaf(wv, z[w * H + k], a[w]);
            }
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                if (w < nc) {
                    float s = warp_sum(a[w]) + b_out[v];
                    if (lane == 0) {
                        if (logits_out) logits_out[((size_t)b * W + w0 + w) * NV + v] = s;
                        if (!WG) {
                            atomicMax(&skey[w], pack_key(s, (uint32_t)v));
                        } else {
                            if (v == blank) s_blank[w0 + w] = s;
                            else atomicMax(&skey[w], pack_key(s, (uint32_t)v));
                            if (s > run_m[w]) { run_s[w] = run_s[w] * __expf(run_m[w] - s) + 1.f; run_m[w] = s; }
                            else run_s[w] += __expf(s - run_m[w]);
                        }
                    }
                }
            }
        }
        if (WG && lane == 0) {
#pragma unroll
            for (int w = 0; w < 8; ++w) { s_m[warp][w] = run_m[w]; s_s[warp][w] = run_s[w]; }
        }
        __syncthreads();
        if (!WG) {
            if (threadIdx.x < nc) keys[(size_t)b * W + w0 + threadIdx.x] = skey[threadIdx.x];
        } else if (threadIdx.x < nc) {
            const int w = threadIdx.x;
            float mx = -INFINITY;
            for (int k = 0; k < nw; ++k) mx = fmaxf(mx, s_m[k][w]);
            float se = 0.f;
            for (int k = 0; k < nw; ++k)
                if (s_s[k][w] > 0.f) se += s_s[k][w] * __expf(s_m[k][w] - mx);
            s_lse[w0 + w] = mx + __logf(se);
            s_best[w0 + w] = skey[w];
        }
    }
    if (WG) {
        __syncthreads();
        if (threadIdx.x == 0) {
            // candidates in the order rows ascending (each row's best non-blank label), "all blank" last; first strict maximum
            float before = 0.f, top = -INFINITY;
            int pick = -1;
            for (int j = 0; j < n; ++j) {
                if (s_best[j] != 0ull) {
                    const float sc = before + key_logit(s_best[j]) - s_lse[j];
                    if (sc > top) { top = sc; pick = j; }
                }
                before += s_blank[j] - s_lse[j];
            }
            if (before > top) pick = -1;
            const unsigned long long blank_key = pack_key(0.f, (uint32_t)blank);
            for (int j = 0; j < n; ++j) keys[(size_t)b * W + j] = j == pick ? s_best[j] : blank_key;
        }
    }
}

template <typename TW, bool WG>
static cudaError_t simt_joint_t(const Call& c, float* logits_out) {
    const size_t smem = sizeof(float) * 8 * (size_t)c.m.H;
    if (smem > 48 * 1024) cudaFuncSetAttribute(joint_simt_kernel<TW, WG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    joint_simt_kernel<TW, WG><<<c.B, 256, smem, c.stream>>>(c.ctrl(), c.t(), c.enc_len, (const TW*)c.enc_proj(), c.pred_proj(),
                                                            (const TW*)c.m.w_out, c.m.b_out, c.keys(), logits_out, c.T, c.W,
                                                            c.m.H, c.m.V + 1, c.m.act, c.m.blank_id);
    return cudaGetLastError();
}

// Beam search: the rows are hypotheses of ONE utterance (all read utterance 0's enc_proj rows), there are only a few
// of them, and only the logits are wanted (Eq. (1) is a pass of its own): one block per (vocabulary slice of 16,
// hypothesis), so that the joint of a handful of hypotheses still spreads over the SMs.
template <typename TW>
__global__ void __launch_bounds__(256) joint_logits_shared_kernel(const int32_t* __restrict__ t_cur, const int32_t* __restrict__ enc_len,
                                                                  const TW* __restrict__ enc_proj, const float* __restrict__ pred_proj,
                                                                  const TW* __restrict__ w_out, const float* __restrict__ b_out,
                                                                  float* __restrict__ logits_out, int W, int H, int NV, int act, int stage_w) {
    extern __shared__ float z[];  // [8][H] activations, then (stage_w) [16][H] the block's rows of W_out
    float* wsm = z + 8 * (size_t)H;
    const int b = blockIdx.y;
    const int t = t_cur[b], len = enc_len[b];
    if (t >= len) return;
    const int n = min(W, len - t);
    const int v0 = blockIdx.x * 16, v1 = min(NV, v0 + 16);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    const bool vec = aligned_rows(w_out, H) && aligned_rows(enc_proj, H);
    // the block's rows of W_out, once (all loads in flight together instead of one dependent load per dot-product step)
    if (stage_w && vec) {
        for (int c8 = threadIdx.x; c8 < (v1 - v0) * H / 8; c8 += blockDim.x) load8(w_out + (size_t)v0 * H + 8 * (size_t)c8, wsm + 8 * c8);
    } else if (stage_w) {
        for (int e = threadIdx.x; e < (v1 - v0) * H; e += blockDim.x) wsm[e] = ldf(w_out + (size_t)v0 * H + e);
    }
    for (int w0 = 0; w0 < n; w0 += 8) {
        const int nc = min(8, n - w0);
        __syncthreads();
        if (vec) {
            for (int c8 = threadIdx.x; c8 < nc * H / 8; c8 += blockDim.x) {
                const int e = 8 * c8, w = e / H, k = e - w * H;
                float x[8];
                load8(enc_proj + (size_t)(t + w0 + w) * H + k, x);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float s = x[i] + pred_proj[(size_t)b * H + k + i];
                    s = act == WIND_ACT_RELU ? fmaxf(s, 0.f) : tanhf(s);
                    z[e + i] = round_like<TW>(s);
                }
            }
        } else {
            for (int e = threadIdx.x; e < nc * H; e += blockDim.x) {
                const int w = e / H, k = e - w * H;
                float s = ldf(enc_proj + (size_t)(t + w0 + w) * H + k) + pred_proj[(size_t)b * H + k];
                s = act == WIND_ACT_RELU ? fmaxf(s, 0.f) : tanhf(s);
                z[e] = round_like<TW>(s);
            }
        }
        __syncthreads();
        for (int v = v0 + warp; v < v1; v += nw) {
            float a[8];
#pragma unroll
            for (int w = 0; w < 8; ++w) a[w] = 0.f;
            for (int k = lane; k < H; k += 32) {
                const float wv = stage_w ? wsm[(size_t)(v - v0) * H + k] : ldf(w_out + (size_t)v * H + k);
#pragma unroll
                for (int w = 0; w < 8; ++w)
                    if (w < nc) a[w] = fmaf(wv, z[w * H + k], a[w]);
            }
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                if (w < nc) {
                    const float s = warp_sum(a[w]) + b_out[v];
                    if (lane == 0) logits_out[((size_t)b * W + w0 + w) * NV + v] = s;
                }
            }
        }
    }
}

template <typename TW>
static cudaError_t simt_joint_shared_t(const Call& c, float* logits_out) {
    // eight activation rows and, where they fit, the block's sixteen rows of W_out
    const int stage_w = sizeof(float) * 24 * (size_t)c.m.H <= 160 * 1024;
    const size_t smem = sizeof(float) * (stage_w ? 24 : 8) * (size_t)c.m.H;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(joint_logits_shared_kernel<TW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    dim3 grid((unsigned)((c.m.V + 1 + 15) / 16), (unsigned)c.B);
    joint_logits_shared_kernel<TW><<<grid, 256, smem, c.stream>>>(c.t(), c.enc_len, (const TW*)c.enc_proj(), c.pred_proj(),
                                                                  (const TW*)c.m.w_out, c.m.b_out, logits_out, c.W, c.m.H,
                                                                  c.m.V + 1, c.m.act, stage_w);
    return cudaGetLastError();
}

cudaError_t simt_joint_shared(const Call& c, float* logits_out) {
    if (c.B == 0) return cudaSuccess;
    return c.m.dtype == WIND_DT_BF16 ? simt_joint_shared_t<__nv_bfloat16>(c, logits_out) : simt_joint_shared_t<float>(c, logits_out);
}

cudaError_t simt_joint(const Call& c, float* logits_out) {
    if (c.B == 0) return cudaSuccess;
    const bool wg = c.mode == WIND_MODE_WINDOW && !logits_out;
    if (c.m.dtype == WIND_DT_BF16)
        return wg ? simt_joint_t<__nv_bfloat16, true>(c, logits_out) : simt_joint_t<__nv_bfloat16, false>(c, logits_out);
    return wg ? simt_joint_t<float, true>(c, logits_out) : simt_joint_t<float, false>(c, logits_out);
}

}  // namespace wind
