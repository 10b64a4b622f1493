// Device-resident label-looping control: per-utterance first-non-blank scan over the
// window's argmax keys, jump, emission, max-symbols rule, termination, and the loop
// condition of the CUDA-graph WHILE node.  No host involvement per step.
#include "wind_internal.cuh"

namespace wind {

// Reset all per-call state.  Block 0 also fills the control block.
__global__ void __launch_bounds__(256) init_kernel(Ctrl* ctrl, int32_t* t, unsigned long long* t_pub, int32_t* count, int32_t* emit_tok,
                                                   unsigned long long* keys, float* h, float* c, uint32_t* hb, uint32_t* z,
                                                   uint32_t* trace, size_t n_trace_words, uint32_t* sync_words, size_t n_sync_words, int32_t* out_len, const int32_t* __restrict__ enc_len, int32_t* slot, int N, int B, int T, size_t n_keys,
                                                   size_t n_h, size_t n_c, size_t n_hb_words, size_t n_z_words,
                                                   int blank, int step_cap, int kernels_used, int launches_per_step,
                                                   int launches_setup) {
    const size_t gtid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t gstride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = gtid; i < n_h; i += gstride) h[i] = 0.f;
    for (size_t i = gtid; i < n_c; i += gstride) c[i] = 0.f;
    for (size_t i = gtid; i < n_hb_words; i += gstride) hb[i] = 0u;
    for (size_t i = gtid; i < n_z_words; i += gstride) z[i] = 0u;
    for (size_t i = gtid; i < n_trace_words; i += gstride) trace[i] = 0u;
    for (size_t i = gtid; i < n_sync_words; i += gstride) sync_words[i] = 0u;   // arrival counters and the stamps of pred_proj
    for (size_t i = gtid; i < n_keys; i += gstride) keys[i] = 0ull;
    for (size_t i = gtid; i < (size_t)B; i += gstride) {
        t[i] = 0;
        t[B + i] = 0;
        t_pub[i] = 0ull;
        count[i] = 0;
        emit_tok[i] = blank;  // start of sequence: every decoder is fed the blank id once
        // batch row i starts with utterance i (the first B of N utterances; rows beyond N stay empty)
        const int len = (int)i < N ? min(max(enc_len[i], 0), T) : 0;
        slot[i] = len;
        slot[B + i] = len;
        slot[2 * B + i] = (int)i * T;
        slot[3 * B + i] = (int)i * T;
        slot[4 * B + i] = (int)i < N ? (int)i : 0;
        slot[5 * B + i] = 0;
    }
    for (size_t i = gtid; i < (size_t)N; i += gstride) out_len[i] = 0;
    if (blockIdx.x == 0) {
        __shared__ int s_active, s_bad;
        __shared__ unsigned long long s_frames;
        if (threadIdx.x == 0) { s_active = 0; s_frames = 0ull; s_bad = 0; }
        __syncthreads();
        int a = 0;
        unsigned long long f = 0;
        for (int b = threadIdx.x; b < N; b += blockDim.x) {
            int len = enc_len[b];
            if (len < 0 || len > T) s_bad = 1;   // a caller's mistake: nothing may be read through this length
            a += len > 0;
            f += (unsigned long long)(len > 0 ? len : 0);
        }
        atomicAdd(&s_active, a);
        atomicAdd(&s_frames, f);
        __syncthreads();
        if (threadIdx.x == 0) {
            ctrl->status = s_bad ? WIND_ERR_INVALID_ARG : 0;
            ctrl->bad_input = s_bad;
            ctrl->active = s_bad ? 0 : s_active;
            ctrl->step = 0;
            ctrl->step_cap = step_cap;
            ctrl->joint_rows = 0;
            ctrl->tokens = 0;
            ctrl->forced = 0;
            ctrl->frames = (int64_t)s_frames;
            for (int k = 0; k < 65; ++k) ctrl->jump_hist[k] = 0;
            ctrl->launches_per_step = launches_per_step;
            ctrl->launches_setup = launches_setup;
            ctrl->kernels = kernels_used;
            ctrl->bar = 0u;
            ctrl->abort = 0;
            for (int k = 0; k < 4; ++k) ctrl->phase_cycles[k] = 0;
            ctrl->loop_ns = 0;
            ctrl->timeout_site = 0;
            ctrl->timeout_cta = 0;
            ctrl->next_utt = N < B ? N : B;
            ctrl->n_utt = N;
        }
    }
}

cudaError_t launch_init(const Call& c, int kernels_used, int launches_per_step, int launches_setup) {
    size_t n_h = 2 * (size_t)c.m.L * c.B * c.m.P, n_c = (size_t)c.m.L * c.B * c.m.P;
    const int N = c.N > 0 ? c.N : c.B;
    // every lock step moves some utterance forward (a frame, or one of at most S tokens on a frame), apart from the
    // two steps around an utterance's start; with refilled rows the worst case is one utterance after the other
    long long step_cap = (long long)c.T * (c.S + 1) + 2;
    if (c.N > 0) step_cap = (step_cap + 1) * c.N;
    if (step_cap > 0x7fffffff) step_cap = 0x7fffffff;
    const bool bf = c.m.dtype == WIND_DT_BF16;
    const size_t n_hb_words = bf ? (size_t)c.m.L * c.lay.Bpad * c.m.P : 0;       // 2 parities x bf16 = one word per element
    const size_t n_z_words = bf ? (size_t)c.lay.rows_pad * c.m.H / 2 : 0;
    size_t biggest = n_h > n_z_words ? n_h : n_z_words;
    if (n_hb_words > biggest) biggest = n_hb_words;
    int blocks = (int)((biggest + 255) / 256);
    if (blocks > 592) blocks = 592;
    if (blocks < 1) blocks = 1;
    init_kernel<<<blocks, 256, 0, c.stream>>>(c.ctrl(), c.t(), c.t_pub(), c.count(), c.emit_tok(), c.keys(), c.h(0), c.c(),
                                              reinterpret_cast<uint32_t*>(c.hb(0, 0)), reinterpret_cast<uint32_t*>(c.z()),
                                              reinterpret_cast<uint32_t*>(c.trace()),
                                              bf ? sizeof(TraceEvent) * kTraceRoles * kTraceEvents / 4 : 0,
                                              reinterpret_cast<uint32_t*>(c.flags()), bf ? (c.lay.enc_proj - c.lay.flags) / 4 : 0,   // the counters, pred_pub and the key slots lie side by side, before enc_proj
                                              c.out_len, c.enc_len, c.slot(), N, c.B, c.T, 3 * (size_t)c.lay.rows_pad, n_h, n_c, n_hb_words,
                                              n_z_words, c.m.blank_id, (int)step_cap, kernels_used, launches_per_step,
                                              launches_setup);
    return cudaGetLastError();
}

// One lock-step control update (Algorithm 2's branch, per utterance):
//   all rows blank -> t += n; else i = first non-blank row, emit (label, t + i), t += i.
// Consumes and clears the keys.  Single block; thread per utterance (strided).
__global__ void __launch_bounds__(256) control_kernel(Ctrl* ctrl, int32_t* __restrict__ t_cur, int32_t* __restrict__ count,
                                                      int32_t* __restrict__ emit_tok, unsigned long long* __restrict__ keys,
                                                      const int32_t* __restrict__ enc_len, int32_t* __restrict__ out_tokens,
                                                      int32_t* __restrict__ out_frames, int32_t* __restrict__ out_len, int B,
                                                      int W, int S, int max_out, int blank, int NV,
                                                      cudaGraphConditionalHandle handle, int use_handle) {
    __shared__ int s_active, s_tokens, s_forced, s_rows, s_err;
    __shared__ int s_hist[65];
    if (ctrl->active == 0) {
        if (use_handle && threadIdx.x == 0) cudaGraphSetConditional(handle, 0);
        return;
    }
    if (threadIdx.x == 0) { s_active = 0; s_tokens = 0; s_forced = 0; s_rows = 0; s_err = 0; }
    for (int k = threadIdx.x; k < 65; k += blockDim.x) s_hist[k] = 0;
    __syncthreads();
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        int t = t_cur[b];
        const int len = enc_len[b];
        int emit = -1;
        if (t < len) {
            const int n = min(W, len - t);
            int i = -1, label = blank;
            for (int w = 0; w < n; ++w) {
                unsigned long long key = keys[(size_t)b * W + w];
                keys[(size_t)b * W + w] = 0ull;
                if (i < 0) {
                    if (key == 0ull) s_err = WIND_ERR_INTERNAL;  // a valid row was never evaluated
                    uint32_t lab = key_label(key);
                    if (lab >= (uint32_t)NV) { s_err = WIND_ERR_INTERNAL; lab = (uint32_t)blank; }
                    if ((int)lab != blank) { i = w; label = (int)lab; }
                }
            }
            atomicAdd(&s_rows, n);
            int cnt = count[b];
            if (i < 0) {
                atomicAdd(&s_hist[n], 1);
                t += n;
                cnt = 0;
            } else {
                atomicAdd(&s_hist[i], 1);
                if (i > 0) cnt = 0;
                t += i;
                int pos = out_len[b];
                if (pos < max_out) {
                    out_tokens[(size_t)b * max_out + pos] = label;
                    out_frames[(size_t)b * max_out + pos] = t;
                    out_len[b] = pos + 1;
                    emit = label;
                    atomicAdd(&s_tokens, 1);
                    cnt += 1;
                    if (cnt == S) { t += 1; cnt = 0; atomicAdd(&s_forced, 1); }
                } else {
                    s_err = WIND_ERR_OUTPUT_OVERFLOW;  // this utterance stops here
                    t = len;
                }
            }
            t_cur[b] = t;
            count[b] = cnt;
            if (t < len) atomicAdd(&s_active, 1);
        }
        emit_tok[b] = emit;
    }
    __syncthreads();
    for (int k = threadIdx.x; k < 65; k += blockDim.x)
        if (s_hist[k]) ctrl->jump_hist[k] += s_hist[k];
    if (threadIdx.x == 0) {
        int active = s_active;
        ctrl->joint_rows += s_rows;
        ctrl->tokens += s_tokens;
        ctrl->forced += s_forced;
        int step = ctrl->step + 1;
        ctrl->step = step;
        if (s_err) set_status(ctrl, s_err);
        if (step >= ctrl->step_cap && active > 0) { set_status(ctrl, WIND_ERR_INTERNAL); active = 0; }
        if (s_err == WIND_ERR_INTERNAL) active = 0;
        ctrl->active = active;
        if (use_handle) cudaGraphSetConditional(handle, active > 0 ? 1u : 0u);
    }
}

cudaError_t launch_control(const Call& c, cudaGraphConditionalHandle handle, int use_handle) {
    control_kernel<<<1, 256, 0, c.stream>>>(c.ctrl(), c.t(), c.count(), c.emit_tok(), c.keys(), c.enc_len, c.out_tokens,
                                            c.out_frames, c.out_len, c.B, c.W, c.S, c.max_out, c.m.blank_id, c.m.V + 1, handle,
                                            use_handle);
    return cudaGetLastError();
}

// Teacher forcing (wind_eval_joint_window): token u of each prefix, -1 past its end.  A token outside [0, V] is a
// caller's mistake: the blank is fed instead and the call reports WIND_ERR_INVALID_ARG.
__global__ void force_tokens_kernel(Ctrl* ctrl, int32_t* emit_tok, const int32_t* __restrict__ prefix, int U,
                                    const int32_t* __restrict__ prefix_len, int u, int B, int NV, int blank) {
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b == 0 && !ctrl->bad_input) ctrl->active = B;
    if (b < B) {
        int tok = (u < prefix_len[b]) ? prefix[(size_t)b * U + u] : -1;
        if (tok >= NV || tok < -1) { tok = blank; set_status(ctrl, WIND_ERR_INVALID_ARG); }
        emit_tok[b] = tok;
    }
}
cudaError_t launch_force_tokens(const Call& c, const int32_t* prefix, int U, const int32_t* prefix_len, int u) {
    force_tokens_kernel<<<(c.B + 127) / 128, 128, 0, c.stream>>>(c.ctrl(), c.emit_tok(), prefix, U, prefix_len, u, c.B, c.m.V + 1,
                                                                 c.m.blank_id);
    return cudaGetLastError();
}

// Window start of every utterance (teacher forcing, beam search).  A start outside [0, len] is a caller's mistake: it
// is moved inside, so that nothing is read out of range, and the call reports WIND_ERR_INVALID_ARG.
__global__ void set_t_kernel(Ctrl* ctrl, int32_t* t, const int32_t* __restrict__ t0, const int32_t* __restrict__ enc_len, int B) {
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b == 0 && !ctrl->bad_input) ctrl->active = B;
    if (b < B) {
        int v = t0[b];
        if (enc_len) {
            const int len = enc_len[b] > 0 ? enc_len[b] : 0;
            if (v < 0 || v > len) { v = v < 0 ? 0 : len; set_status(ctrl, WIND_ERR_INVALID_ARG); }
        }
        t[b] = v;
        t[B + b] = v;
    }
}
cudaError_t launch_set_t(const Call& c, const int32_t* t0) {
    set_t_kernel<<<(c.B + 127) / 128, 128, 0, c.stream>>>(c.ctrl(), c.t(), t0, c.enc_len, c.B);
    return cudaGetLastError();
}

// Measurement aid: joint activations of a plausible size in every row (a hash of the index mapped to [0, 2), as after a
// ReLU), so that the joint phase can be timed alone on fixed operands.
__global__ void fill_z_kernel(__nv_bfloat16* z, size_t n) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        uint32_t x = (uint32_t)i * 2654435761u + 12345u;
        x ^= x >> 15; x *= 2246822519u; x ^= x >> 13;
        z[i] = __float2bfloat16_rn((float)(x & 0xFFFFu) * (2.f / 65536.f));
    }
}
cudaError_t launch_fill_z(const Call& c) {
    fill_z_kernel<<<296, 256, 0, c.stream>>>(c.z(), (size_t)c.lay.rows_pad * c.m.H);
    return cudaGetLastError();
}

}  // namespace wind
