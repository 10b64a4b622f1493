// Internal declarations shared by the translation units of the library:
// workspace layout, device control block, argmax key packing, launch prototypes.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "wind.h"

namespace wind {

constexpr int WIND_MODE_FIRST_NONBLANK = 0;
constexpr int WIND_MODE_WINDOW = 1;
constexpr int kMaxLayers = 8;
constexpr int kMaxWindow = 64;
constexpr size_t kAlign = 256;

// Timeline of the loop kernel (debug aid, off unless a step window is set): one record per event.
struct TraceEvent {
    uint32_t tag;      // phase * 16 + event
    int32_t step;
    long long clock;   // clock64 of the SM that runs CTA 0
};
constexpr int kTraceRoles = 24;    // TMA issuer, MMA issuer, first epilogue thread, barrier: of CTA 0, then of the last CTA;
                                   // 8..23: marks of EVERY CTA in the first traced step (global timer), see trace_mark
constexpr int kTraceEvents = 512;

// Device control block, first thing in the workspace.
struct Ctrl {
    int32_t status;   // wind_status_t, sticky (first error wins)
    int32_t active;   // utterances with t < len after the last control update
    int32_t step;     // loop iterations executed
    int32_t step_cap; // hard bound on step
    int64_t joint_rows;
    int64_t tokens;
    int64_t forced;
    int64_t frames;
    int64_t jump_hist[65];
    int32_t launches_per_step;
    int32_t launches_setup;
    int32_t kernels;
    int32_t bad_input;  // set by the init kernel: a length outside [0, T]; the loops then do not start
    // persistent loop kernel
    uint32_t bar;             // grid barrier: arrivals so far (monotonic within a call)
    int32_t abort;            // some CTA gave up: everybody leaves
    long long phase_cycles[4];  // SM cycles spent in the joint / decoder-update / projection phases (CTA 0), [3] unused
    long long loop_ns;        // wall time of the loop kernel (CTA 0, global timer)
    int32_t timeout_site;     // which wait ran out first (resident-weights loop kernel; 0 = none), and in which CTA
    int32_t timeout_cta;
    int32_t next_utt;         // first utterance that has not been given a batch row yet (more utterances than rows)
    int32_t n_utt;
};

// Byte offsets of every workspace region (all multiples of kAlign).
struct Layout {
    size_t ctrl;       // Ctrl
    size_t t;          // int32 [2][B] current frame per utterance (the loop kernel ping-pongs by step parity)
    size_t t_pub;      // uint64 [B]  (lock step + 2) << 32 | next frame: published early in a step for the projection CTAs
    size_t slot;       // int32 [6][B] the utterance of each batch row: frames [2][B], first enc_proj row [2][B], index, tokens so far
    size_t count;      // int32 [B]   consecutive emissions on the current frame
    size_t emit_tok;   // int32 [B]   token to feed to the decoder this step, -1 = none
    size_t keys;       // uint64 [3][rows_pad] packed (logit, label) argmax keys, 0 = empty ([1]: loop kernel's other step
                       // parity; [2]: best non-blank key per row in window-based decoding)
    size_t jpart;      // float2 [rows_pad][4 * vocabulary tiles] partial (maximum, sum of exponentials) of each row's logits
    size_t jblank;     // fp32 [rows_pad] blank logit of each window row (both: window-based decoding on the tensor path)
    size_t h;          // fp32 [2][L][B][P]  LSTM hidden state, ping-pong by step parity (plain-ALU path)
    size_t c;          // fp32 [L][B][P]     LSTM cell state
    size_t pred_proj;  // fp32 [B][H]        (plain-ALU path)
    size_t hb;         // bf16 [2][L][Bpad][P] LSTM hidden state as tensor-core operand rows (tensor path)
    size_t z;          // bf16 [rows_pad][H] joint activations act(enc_proj + pred_proj), the joint GEMM's operand (tensor path)
    size_t dh;         // fp32 [B][4P] layer 1's recurrent term, handed from its CTAs to the layer's update (tensor path, L >= 2)
    size_t g0;         // fp32 [V+1][4P] layer-0 gate pre-activations of every token: W_ih emb[tok] + b_ih + b_hh (tensor path)
    size_t trace;      // TraceEvent [kTraceRoles][kTraceEvents]: optional timeline of CTA 0 of the loop kernel
    size_t flags;      // uint32 [n_flags] arrival counters between CTA groups of the resident-weights loop kernel
    size_t kslot;      // uint64 [window rows][vocabulary tiles, padded to even] stamped (logit, label) keys, one per window row and vocabulary tile
    size_t pred_pub;   // (bf16 x 2, uint32) [B][H / 2] pred_proj values in pairs, each pair stamped with the projection phase that wrote it
    size_t enc_proj;   // elem [N*T][H] (N utterances; N = B unless rows are refilled)
    size_t total;
    // host staging (wind_decode_greedy_host), placed after `total`
    size_t st_enc, st_len, st_tok, st_frm, st_olen, st_total;
    int32_t Bpad;      // B rounded up to 128 (tensor path operand rows)
    int32_t rows_pad;  // B*W rounded up to 256 (window rows incl. tile padding)
    int32_t n_flags;   // one counter per 16 window rows of the widest window and three per 16 utterances always suffice
};

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

inline Layout make_layout(const wind_model_t& m, int B, int T, int W, int max_out, int N = 0) {
    Layout L{};
    const size_t es = (m.dtype == WIND_DT_BF16) ? 2 : 4;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    L.ctrl = take(sizeof(Ctrl));
    const bool bf = m.dtype == WIND_DT_BF16;
    L.rows_pad = (int32_t)(((size_t)B * W + 255) / 256 * 256);
    L.t = take(sizeof(int32_t) * 2 * B);
    L.t_pub = take(sizeof(uint64_t) * B);
    L.slot = take(sizeof(int32_t) * 6 * B);
    L.count = take(sizeof(int32_t) * B);
    L.emit_tok = take(sizeof(int32_t) * B);
    L.keys = take(sizeof(uint64_t) * 3 * (size_t)L.rows_pad);
    L.h = take(sizeof(float) * 2 * (size_t)m.L * B * m.P);
    L.c = take(sizeof(float) * (size_t)m.L * B * m.P);
    L.pred_proj = take(sizeof(float) * (size_t)B * m.H);
    L.Bpad = (B + 127) / 128 * 128;
    L.hb = take(bf ? 2 * (size_t)m.L * L.Bpad * m.P * 2 : 0);
    L.z = take(bf ? (size_t)L.rows_pad * m.H * 2 : 0);
    L.dh = take(bf && m.L >= 2 ? sizeof(float) * (size_t)B * 4 * m.P : 0);
    L.g0 = take(bf ? sizeof(float) * (size_t)(m.V + 1) * 4 * m.P : 0);
    L.trace = take(bf ? sizeof(TraceEvent) * kTraceRoles * kTraceEvents : 0);
    L.jpart = take(bf ? sizeof(float) * 2 * (size_t)L.rows_pad * 4 * ((size_t)(m.V + 1 + 127) / 128) : 0);
    L.jblank = take(bf ? sizeof(float) * (size_t)L.rows_pad : 0);
    L.n_flags = B * (kMaxWindow / 16) + 16 + 3 * (B / 16 + 1);   // independent of W: row groups have at least 16 rows
    L.flags = take(bf ? sizeof(uint32_t) * (size_t)L.n_flags : 0);
    L.pred_pub = take(bf ? 4 * (size_t)B * m.H : 0);
    L.kslot = take(bf ? 8 * ((size_t)L.rows_pad + 256) * (((size_t)(m.V + 1 + 127) / 128 + 1) & ~(size_t)1) : 0);
    L.enc_proj = take(es * (size_t)(N > B ? N : B) * T * m.H);
    L.total = off;
    L.st_enc = take(es * (size_t)B * T * m.D);
    L.st_len = take(sizeof(int32_t) * B);
    L.st_tok = take(sizeof(int32_t) * (size_t)B * (max_out > 0 ? max_out : 1));
    L.st_frm = take(sizeof(int32_t) * (size_t)B * (max_out > 0 ? max_out : 1));
    L.st_olen = take(sizeof(int32_t) * B);
    L.st_total = off - L.total;
    return L;
}

// Everything a kernel launcher needs for one call (host-side bundle, passed by value).
struct Call {
    wind_model_t m;
    const void* w_ih[kMaxLayers];
    const void* w_hh[kMaxLayers];
    const float* b_ih[kMaxLayers];
    const float* b_hh[kMaxLayers];
    const void* enc;
    const int32_t* enc_len;
    int32_t B, T, W, S, max_out;
    int32_t N;        // utterances when batch rows are refilled (wind_decode_greedy_refill), else 0: row b = utterance b
    int32_t mode;     // WIND_MODE_FIRST_NONBLANK (Algorithm 2) or WIND_MODE_WINDOW (best pair of Eq. (1) per step)
    int32_t joint_iters;   // wind_bench_joint: run only the joint phase of the loop kernel, this many times
    int32_t* out_tokens;
    int32_t* out_frames;
    int32_t* out_len;
    uint8_t* ws;
    Layout lay;
    cudaStream_t stream;
    const void* tc;   // tensor maps of this call (host memory owned by the tensor-kernel module)

    Ctrl* ctrl() const { return reinterpret_cast<Ctrl*>(ws + lay.ctrl); }
    int32_t* t() const { return reinterpret_cast<int32_t*>(ws + lay.t); }   // [2][B]; the per-phase kernels use [0]
    unsigned long long* t_pub() const { return reinterpret_cast<unsigned long long*>(ws + lay.t_pub); }
    int32_t* slot() const { return reinterpret_cast<int32_t*>(ws + lay.slot); }
    int32_t* count() const { return reinterpret_cast<int32_t*>(ws + lay.count); }
    int32_t* emit_tok() const { return reinterpret_cast<int32_t*>(ws + lay.emit_tok); }
    unsigned long long* keys() const { return reinterpret_cast<unsigned long long*>(ws + lay.keys); }  // [2][rows_pad]
    float* h(int parity) const {
        return reinterpret_cast<float*>(ws + lay.h) + (size_t)parity * m.L * B * m.P;
    }
    float* c() const { return reinterpret_cast<float*>(ws + lay.c); }
    float* pred_proj() const { return reinterpret_cast<float*>(ws + lay.pred_proj); }
    void* enc_proj() const { return ws + lay.enc_proj; }
    __nv_bfloat16* z() const { return reinterpret_cast<__nv_bfloat16*>(ws + lay.z); }
    float* g0() const { return reinterpret_cast<float*>(ws + lay.g0); }
    float* dh() const { return reinterpret_cast<float*>(ws + lay.dh); }
    float2* jpart() const { return reinterpret_cast<float2*>(ws + lay.jpart); }
    float* jblank() const { return reinterpret_cast<float*>(ws + lay.jblank); }
    TraceEvent* trace() const { return reinterpret_cast<TraceEvent*>(ws + lay.trace); }
    uint32_t* flags() const { return reinterpret_cast<uint32_t*>(ws + lay.flags); }
    unsigned long long* pred_pub() const { return reinterpret_cast<unsigned long long*>(ws + lay.pred_pub); }
    unsigned long long* kslot() const { return reinterpret_cast<unsigned long long*>(ws + lay.kslot); }
    __nv_bfloat16* hb(int parity, int l) const {
        return reinterpret_cast<__nv_bfloat16*>(ws + lay.hb) + ((size_t)parity * m.L + l) * lay.Bpad * m.P;
    }
};

// ---------------------------------------------------------------------------
// argmax key: (orderable fp32 logit) << 32 | (0xFFFFFFFF - label); max key = max logit,
// lowest label on equal logits.  0 is "empty".
// ---------------------------------------------------------------------------
__host__ __device__ inline uint32_t orderable_f32(uint32_t bits) {
    return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
}
__device__ inline unsigned long long pack_key(float logit, uint32_t label) {
    return ((unsigned long long)orderable_f32(__float_as_uint(logit)) << 32) | (unsigned long long)(0xFFFFFFFFu - label);
}
__host__ __device__ inline uint32_t key_label(unsigned long long key) {
    return 0xFFFFFFFFu - (uint32_t)(key & 0xFFFFFFFFull);
}
__device__ inline float key_logit(unsigned long long key) {
    const uint32_t hi = (uint32_t)(key >> 32);
    return __uint_as_float((hi & 0x80000000u) ? (hi & 0x7FFFFFFFu) : ~hi);
}

__device__ inline void set_status(Ctrl* ctrl, int32_t s) { atomicCAS(&ctrl->status, 0, s); }

// ---------------------------------------------------------------------------
// launchers (each enqueues on call.stream; returns cudaGetLastError())
// ---------------------------------------------------------------------------
// plain-ALU kernels (fp32 path, and bf16 path when the tensor kernels do not apply)
cudaError_t simt_enc_proj(const Call& c);
cudaError_t simt_pred_step(const Call& c, int parity_in);            // all layers + pred_proj
cudaError_t simt_joint(const Call& c, float* logits_out /*nullable*/);
cudaError_t simt_joint_shared(const Call& c, float* logits_out);   // every row's window comes from utterance 0 (beam search)
int simt_pred_launches(const Call& c);

// control
cudaError_t launch_init(const Call& c, int kernels_used, int launches_per_step, int launches_setup);
cudaError_t launch_control(const Call& c, cudaGraphConditionalHandle handle, int use_handle);
cudaError_t launch_force_tokens(const Call& c, const int32_t* prefix, int U, const int32_t* prefix_len, int u);
cudaError_t launch_set_t(const Call& c, const int32_t* t0);
cudaError_t launch_fill_z(const Call& c);   // measurement aid: fixed joint activations

// first-output distribution of a window (Eq. 1), in place on the window's logits
// beam search (Algorithm 3): workspace regions behind the call's own layout, and the host-driven search
struct BeamLayout {
    size_t h_pool, c_pool, g_pool;   // fp32 [slots][L][P] x 2, [slots][H]: decoder states of live hypotheses and their pred_proj
    size_t ints;                     // int32 [8][K] per-iteration index arrays
    size_t logits;                   // fp32 [K][W][V+1]
    size_t top_label, top_jump, top_logp;   // [K][K]
    size_t total;
    int slots;
};
BeamLayout make_beam_layout(const wind_model_t& m, int T, int W, int K, int S, size_t base);
wind_status_t beam_search_run(Call& cb, const BeamLayout& bl, int K, int prefix_search, int max_hyps, int max_out, int32_t* out_tokens,
                              int32_t* out_frames, int32_t* out_len, double* out_score, int32_t* n_hyps, int64_t* n_steps,
                              cudaError_t* cuda_err);

cudaError_t launch_first_output(float* logp, const int32_t* enc_len, const int32_t* t0, int B, int W, int NV, int blank, int K,
                                int32_t* top_label, int32_t* top_jump, float* top_logp, cudaStream_t stream);

// tensor-core kernels (bf16 path)
bool tc_supported(const wind_model_t& m, int B, int T, int W);
cudaError_t tc_prepare(Call& c);         // builds the tensor maps and the tile plan of this call (host only), sets c.tc
cudaError_t tc_enc_proj(const Call& c);
cudaError_t tc_gate_table(const Call& c);  // g0[tok] = W_ih[0] emb[tok] + b_ih[0] + b_hh[0] for every token
// The whole decoding loop as one persistent cooperative kernel.  prefix == nullptr: greedy
// decoding until every utterance is done.  Otherwise teacher forcing: feed prefix tokens, then
// store the window logits at t (set beforehand in both t buffers) to logits_out.
cudaError_t tc_loop(const Call& c, const int32_t* prefix, int U, const int32_t* prefix_len, float* logits_out,
                    int trace_step);
int tc_setup_launches(const Call& c);

}  // namespace wind
