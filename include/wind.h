/*
 * wind.h -- C ABI of the B200 (sm_100a) library for batched greedy RNN-Transducer
 * decoding with windowed non-blank detection (WIND).
 *
 * The library computes, per utterance, exactly what the sequential greedy procedure
 * computes (Algorithm 1, "RNN-T Inference Algorithm"): scan the encoder frames left to
 * right; at frame t evaluate the joiner on (enc[t], decoder state) and take the argmax;
 * a non-blank label is appended, fed to the decoder and t is kept; blank keeps the
 * decoder state and advances t (rules 1 and 2 of the background section).  With a window
 * W > 1 it follows Algorithm 2 ("WIND Algorithm"): the joiner is evaluated on
 * enc[t : t+n], n = min(W, len - t), against the ONE current decoder state, every row's
 * argmax is taken, and the decoder jumps to the first non-blank row (t += i, label
 * appended) or past the whole window (t += n) when all rows are blank.  W = 1 is the
 * sequential baseline.  The batch runs in lock step (one joiner call and one masked
 * decoder update per step for all utterances), which the paper describes in prose only
 * (method section, last paragraph; CUDA-graph paragraph of the analysis section).
 *
 * Model (the paper leaves decoder and joiner abstract; these are the shapes used here):
 *   decoder : embedding [V+1, E] + L-layer LSTM (hidden P, gate order i,f,g,o, biases
 *             b_ih + b_hh, zero initial state), one token per update; the
 *             start-of-sequence input is blank_id;
 *   joiner  : logits = W_out * act(W_enc*f + b_enc + W_pred*h_top + b_pred) + b_out,
 *             V+1 logits, argmax with the lowest index winning ties.
 * max_symbols (S): after S consecutive emissions on one frame the S-th token is still
 * emitted and fed to the decoder, then t advances by one; the count resets whenever t
 * advances (the safeguard the paper mentions in a footnote of the beam-search section).
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless the parameter comment says "host".
 *   - All buffers are caller-owned and borrowed for the duration of the call; the
 *     library allocates no device memory.  Weight matrices are row-major [out, in].
 *   - dtype WIND_DT_F32: everything fp32, plain FMA arithmetic (no tf32); joint logits agree
 *     with an fp64 evaluation within 1e-4.
 *   - dtype WIND_DT_BF16: enc, emb and all weight matrices are bf16 (uint16 bit patterns),
 *     biases fp32.  Every product is accumulated in fp32 and the LSTM cell state c is kept in
 *     fp32.  Three intermediate quantities are rounded to bf16 (nearest even) because they are
 *     tensor-core operands: enc_proj (stored once per call), the LSTM hidden state h wherever it
 *     is consumed (the recurrent term of the next update, the input of the layer above and
 *     pred_proj -- the recurrence therefore feeds back a bf16 h), and the joint's activations
 *     act(enc_proj + pred_proj).  Both kernel sets (wind_kernels_t) round in the same places; the
 *     tensor-core kernels with on-chip weights also round pred_proj to bf16 before that sum.
 *     The tensor-core kernels evaluate the gate nonlinearities (and tanh activations) with the
 *     hardware tanh approximation (absolute error about 5e-4, below the bf16 rounding of h) when
 *     the weights are resident on chip; the plain-ALU kernels use tanhf / expf.  Joint logits
 *     agree with an fp64 evaluation of the same bf16 weights within 2e-2, also after hundreds
 *     of decoder updates; decisions whose top-two margin is smaller than such differences can
 *     come out differently between kernel sets (AUTO picks the set by shape), never between two
 *     runs of one set, and never between window sizes.
 *   - Calls enqueue work on `stream`, synchronise that stream once at the end to read the
 *     device status word, and return it.  Errors detectable on the host return before
 *     any launch.  Every device-side wait is bounded; a wait that runs out sets
 *     WIND_ERR_TIMEOUT instead of hanging.
 *   - Results are deterministic run to run.
 */
#ifndef WIND_H_
#define WIND_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    WIND_OK = 0,
    WIND_ERR_INVALID_ARG = 1,     /* null pointer, non-positive size, W < 1, blank_id > V, ... */
    WIND_ERR_UNSUPPORTED = 2,     /* shape outside what the kernels handle (see wind_decode_greedy) */
    WIND_ERR_CUDA = 3,            /* a CUDA runtime/driver call failed; see wind_last_cuda_error() */
    WIND_ERR_OUTPUT_OVERFLOW = 4, /* some utterance produced more than max_out tokens */
    WIND_ERR_TIMEOUT = 5,         /* a bounded device-side wait ran out */
    WIND_ERR_INTERNAL = 6,        /* step cap exceeded or inconsistent device state */
    WIND_ERR_WORKSPACE = 7        /* workspace too small or misaligned */
} wind_status_t;

typedef enum { WIND_ACT_RELU = 0, WIND_ACT_TANH = 1 } wind_act_t;
typedef enum { WIND_DT_F32 = 0, WIND_DT_BF16 = 1 } wind_dtype_t;

/* Which kernels run the bf16 path.  AUTO picks the tensor-core (tcgen05/TMA) kernels
 * when the shapes allow (D, E, P, H multiples of 64) and the plain-ALU kernels otherwise. */
typedef enum { WIND_KERNELS_AUTO = 0, WIND_KERNELS_SIMT = 1, WIND_KERNELS_TENSOR = 2 } wind_kernels_t;

typedef struct {
    int32_t D, E, P, L, H, V;  /* V labels; logits are V+1 wide; 1 <= L <= 8 */
    int32_t blank_id;          /* 0..V; also the start-of-sequence decoder input */
    int32_t act;               /* wind_act_t */
    int32_t dtype;             /* wind_dtype_t: element type of enc, emb and the weight matrices */
    int32_t reserved;
    const void* emb;           /* [V+1, E] */
    const void* const* w_ih;   /* HOST array of L device pointers: [4P, E] for l = 0, [4P, P] for l > 0 */
    const void* const* w_hh;   /* HOST array of L device pointers: [4P, P] */
    const float* const* b_ih;  /* HOST array of L device pointers: [4P] fp32 */
    const float* const* b_hh;  /* HOST array of L device pointers: [4P] fp32 */
    const void* w_enc;         /* [H, D] */
    const float* b_enc;        /* [H] */
    const void* w_pred;        /* [H, P] */
    const float* b_pred;       /* [H] */
    const void* w_out;         /* [V+1, H] */
    const float* b_out;        /* [V+1] */
} wind_model_t;

/* Counters of the last decode that used a workspace (read back with wind_read_stats). */
typedef struct {
    int64_t steps;         /* lock-step iterations of the decoding loop */
    int64_t joint_rows;    /* joiner rows evaluated for decisions (sum of n over steps and utterances) */
    int64_t tokens;        /* tokens emitted (= decoder updates after the start-of-sequence one) */
    int64_t forced;        /* forced advances by the max_symbols rule */
    int64_t frames;        /* sum of enc_len */
    int64_t jump_hist[65]; /* jump sizes 0..min(W,64): i on an emission, n on an all-blank window */
    int32_t status;        /* device status word (wind_status_t) */
    int32_t launches_per_step; /* kernel nodes in one loop iteration */
    int32_t launches_setup;    /* kernel launches outside the loop (projection, init, first decoder update) */
    int32_t kernels;           /* wind_kernels_t actually used */
    int32_t timeout_site;      /* after WIND_ERR_TIMEOUT from the resident-weights loop kernel: a code for the wait that ran
                                  out first (a diagnostic: grep the code in the kernel source) and the CTA it ran out in */
    int32_t timeout_cta;
} wind_stats_t;

/*
 * Bytes of device workspace needed by wind_decode_greedy / wind_eval_joint_window for
 * batches up to B utterances of up to T frames and window W.  Holds enc_proj [B,T,H],
 * the decoder state, per window row a few argmax keys, the joint's activations and (for
 * window-based decoding) per-tile softmax statistics -- the window logits themselves,
 * W x (V+1) floats per utterance in the paper's memory analysis, never leave the chip --
 * and control words.  Grows with W only by these per-row arrays.
 */
wind_status_t wind_workspace_bytes(const wind_model_t* m, int32_t B, int32_t T, int32_t W, size_t* bytes);

/*
 * Batched greedy decoding (Algorithm 2; Algorithm 1 when W == 1).
 *   enc        [B, T, D] row-major, element type m->dtype.  Frames t >= enc_len[b] are
 *              never read for a decision (they may hold NaN).
 *   enc_len    [B] int32, 0 <= enc_len[b] <= T.  The values live on the device, so they are checked there, before
 *              the loop starts: if one lies outside [0, T] nothing is decoded (no frame is read through
 *              it), the outputs are undefined and the call returns WIND_ERR_INVALID_ARG.
 *   W          window, 1 <= W <= 64.   max_symbols >= 1.
 *   out_tokens [B, max_out] int32; out_frames [B, max_out] int32 (0-based encoder frame at
 *              which the token was emitted, non-decreasing, each value at most
 *              max_symbols times); out_len [B] int32.  Entries beyond out_len[b] are
 *              left untouched.  max_out = T * max_symbols always suffices; if an utterance
 *              needs more than max_out it stops there, the others finish, and the call
 *              returns WIND_ERR_OUTPUT_OVERFLOW.
 *   workspace  device memory, 256-byte aligned, at least wind_workspace_bytes(m,B,T,W).
 *              Calls sharing a workspace must not overlap in time.
 *   stream     cudaStream_t (0 = default stream).
 * WIND_ERR_UNSUPPORTED: L > 8, W > 64, B*T*H or B*max_out beyond 2^31-1 elements.
 */
wind_status_t wind_decode_greedy(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B,
                                 int32_t T, int32_t W, int32_t max_symbols, int32_t* out_tokens,
                                 int32_t* out_frames, int32_t* out_len, int32_t max_out, void* workspace,
                                 size_t workspace_bytes, void* stream);

/*
 * Greedy decoding (Algorithm 2) of N utterances on B batch rows, B <= N or not: rows 0..B-1 start with utterances
 * 0..B-1, and a row whose utterance is finished takes the next utterance that has none yet, inside the decoding loop
 * (the row's decoder state is cleared in the lock step that finds it finished, the utterance moves in, and the step
 * after that feeds start-of-sequence; two lock steps per change of utterance).  The batch therefore stays full until
 * fewer than B utterances are left -- the length-sorted batches of wind_plan_batches shorten each batch's tail, this
 * removes it.  Every utterance's result is the one wind_decode_greedy gives for it in a batch of B rows (Algorithm 2
 * treats the utterances of a batch independently; a batch size for which the library picks another kernel plan can
 * differ at low-margin decisions, as stated at the top); which row decodes which utterance is not part of the result.
 *   enc [N, T, D], enc_len [N], out_tokens / out_frames [N, max_out], out_len [N]: as in wind_decode_greedy, per
 *   utterance.  Workspace: wind_refill_workspace_bytes (enc_proj of all N utterances, everything else for B rows).
 * Only the tensor-core kernel set refills rows: WIND_ERR_UNSUPPORTED for fp32 models and for shapes outside that set
 * (see wind_decode_greedy), and when N * T * max(D, H) exceeds 2^31 - 1.  wind_read_stats counts over all N utterances.
 * The paper decodes fixed batches; its batched decoding (Section 2.2) leaves the order of utterances to the caller.
 */
wind_status_t wind_refill_workspace_bytes(const wind_model_t* m, int32_t N, int32_t T, int32_t B, int32_t W, size_t* bytes);
wind_status_t wind_decode_greedy_refill(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t N, int32_t T,
                                        int32_t B, int32_t W, int32_t max_symbols, int32_t* out_tokens, int32_t* out_frames,
                                        int32_t* out_len, int32_t max_out, void* workspace, size_t workspace_bytes,
                                        void* stream);

/*
 * Window-based greedy decoding: at every step the window's first-output distribution P'(v, t) of Eq. (1) is
 * formed under the current decoder state and its most probable entry decides the step (the variant sketched
 * beside Algorithm 2, which looks at the whole window instead of stopping at the first frame whose own argmax is
 * not blank):
 *   pair (v != blank, offset j): v is emitted at frame t + j and t += j;
 *   the blank entry (only the window's last row has one: every row blank): t += n.
 * Candidates are compared in the order offsets ascending, labels ascending, the blank entry last; the first
 * strict maximum wins.  log-softmax, the running sum of blank log-probabilities and the comparison are fp32.
 * The max_symbols rule, every argument, the outputs, the workspace (same size) and the status codes are those of
 * wind_decode_greedy.  W == 1 gives Algorithm 1; for W > 1 the result depends on W.
 */
wind_status_t wind_decode_window_greedy(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B,
                                        int32_t T, int32_t W, int32_t max_symbols, int32_t* out_tokens,
                                        int32_t* out_frames, int32_t* out_len, int32_t max_out, void* workspace,
                                        size_t workspace_bytes, void* stream);

/*
 * Extra workspace (added to wind_workspace_bytes) that wind_decode_greedy_host needs for
 * staging enc, enc_len and the three outputs on the device.
 */
wind_status_t wind_host_staging_bytes(const wind_model_t* m, int32_t B, int32_t T, int32_t max_out, size_t* bytes);

/*
 * Same decode, but enc, enc_len, out_tokens, out_frames and out_len are HOST pointers
 * (pinned memory gives asynchronous copies).  The call copies enc_len and the valid frames
 * of enc to the device, decodes, copies the lengths and then the token and frame columns up
 * to the longest transcript back (entries of a row beyond its out_len are unspecified), and
 * synchronises the stream.  enc_len_host is also read on the host: a value outside [0, T] is
 * WIND_ERR_INVALID_ARG.  The model's
 * weights stay device pointers.  workspace: device, at least wind_workspace_bytes +
 * wind_host_staging_bytes.
 */
wind_status_t wind_decode_greedy_host(const wind_model_t* m, const void* enc_host, const int32_t* enc_len_host,
                                      int32_t B, int32_t T, int32_t W, int32_t max_symbols,
                                      int32_t* out_tokens_host, int32_t* out_frames_host, int32_t* out_len_host,
                                      int32_t max_out, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Teacher-forced window logits, for parity checks: runs the same projection, decoder and
 * fused joiner kernels as the decode, with the argmax epilogue replaced by a store.
 *   prefix [B, U] int32, prefix_len [B] (tokens fed after the start-of-sequence blank;
 *   U >= max prefix_len), t0 [B] window start (0 <= t0[b] <= enc_len[b]).
 *   logits [B, W, V+1] fp32; rows w >= min(W, enc_len[b] - t0[b]) are left untouched.
 * A length outside [0, T] is handled as in wind_decode_greedy.  A prefix token outside [0, V] is replaced
 * by the blank and a window start outside [0, enc_len[b]] is moved inside (so that nothing is read out of
 * range); in both cases the call returns WIND_ERR_INVALID_ARG and the logits are undefined.
 */
wind_status_t wind_eval_joint_window(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B,
                                     int32_t T, int32_t W, const int32_t* prefix, int32_t U,
                                     const int32_t* prefix_len, const int32_t* t0, float* logits, void* workspace,
                                     size_t workspace_bytes, void* stream);

/*
 * Eq. (1) of the paper's beam-search section: P'(v, t), the probability that v is the FIRST output in the window that
 * starts at frame t0[b], emitted at frame t0[b] + t, given the decoder state after `prefix`:
 *     v != blank:  P(v | t0 + t) * prod_{t' < t} P(blank | t0 + t')
 *     v == blank:  0 for t < n - 1;  prod_{t' <= n - 1} P(blank | t0 + t') for t = n - 1
 * with P(. | frame) the softmax of the joint's logits and n = min(W, enc_len[b] - t0[b]) (the truncated window of
 * Algorithm 3, line "n = min(N, T - t)").  Same inputs as wind_eval_joint_window.
 *   logp       [B, W, V+1] fp32 out: natural-log P'(v, t), -inf for the zero entries; rows w >= n are left untouched.
 *   K          0, or how many of the most probable (label, offset) pairs to return per utterance: the expansions
 *              Algorithm 3 takes "from all |V| x n combinations".  top_label, top_jump [B, K] int32, top_logp [B, K] fp32,
 *              best first; equal values in order of (offset, label); -1 / -inf when the window has fewer than K entries.
 * The logits stay in `logp` between the joint's store epilogue and the in-place pass; errors as wind_eval_joint_window.
 */
wind_status_t wind_window_first_output(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B, int32_t T,
                                       int32_t W, const int32_t* prefix, int32_t U, const int32_t* prefix_len,
                                       const int32_t* t0, float* logp, int32_t K, int32_t* top_label, int32_t* top_jump,
                                       float* top_logp, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Largest workspace, in bytes, that wind_eval_joint_window_static can serve: the size of the
 * scratch array compiled into the library.
 */
#define WIND_STATIC_WORKSPACE_BYTES (16u * 1024u * 1024u)

/*
 * wind_eval_joint_window for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this entry point exists only for the sake of such callers.)
 *
 * Some callers of this library run where cudaMalloc is off limits: inside a stream-ordered
 * section that must not synchronise the device, in a process whose memory pool is owned and
 * fully handed out by another component, or in a real-time loop that is not allowed to touch
 * the driver's allocator.  They cannot size and allocate the `workspace` the other entry points
 * ask for.  This variant takes the same inputs and writes the same `logits`, but keeps all of
 * its scratch (enc_proj, decoder state, keys, control words) in one array of
 * WIND_STATIC_WORKSPACE_BYTES that is part of the library image: every GPU on which the
 * library's kernels are loaded holds those bytes until the process exits.
 *
 *   - The call makes no cudaMalloc / cudaFree and uses no library routine that allocates.
 *   - If wind_workspace_bytes(m, B, T, W) exceeds WIND_STATIC_WORKSPACE_BYTES the call returns
 *     WIND_ERR_WORKSPACE before any launch; use wind_eval_joint_window with your own workspace.
 *   - The first call on each device is a set-up step: with that device current it looks up the
 *     device address of the array.  With CUDA's lazy loading this is also the moment the driver
 *     loads the library's image on that device, which reserves the array's bytes and may
 *     synchronise the device; if the device has no room left the call fails with WIND_ERR_CUDA.
 *     Make that first call at start-up, outside any stream capture and before memory gets tight;
 *     later calls on the device only read the cached address.  The address belongs to the
 *     device's primary context: after cudaDeviceReset it is stale and this entry point must not
 *     be used again in the process.
 *   - All calls on one device share the one array, which still holds what the previous call
 *     left; every call re-initialises the parts that must start from zero.  Two calls that
 *     overlap on the GPU (different streams, or different host threads) race on it: serialise them.
 * Arguments, results and error codes are otherwise those of wind_eval_joint_window.
 */
wind_status_t wind_eval_joint_window_static(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B,
                                            int32_t T, int32_t W, const int32_t* prefix, int32_t U,
                                            const int32_t* prefix_len, const int32_t* t0, float* logits, void* stream);

/* Per-kernel device times of one decode (milliseconds summed over launches, and launch counts):
 * CUDA events recorded on `stream` around every launch on the plain-ALU path; on the tensor-core
 * path the loop's phases as timed inside the persistent kernel. */
typedef struct {
    double enc_proj_ms, joint_ms, control_ms, pred_ms;
    int64_t enc_proj_launches, joint_launches, control_launches, pred_launches;
    /* tensor-core path only (zero otherwise): the decoding loop is one persistent kernel; loop_ms is its
     * duration between two CUDA events, split into joint_ms + lstm_ms + proj_ms (= pred_ms) in proportion to
     * the SM cycles its first CTA spent in each phase (barrier waits included); gate_table_ms is the one-shot
     * GEMM that tabulates layer 0's input term for every token */
    double loop_ms, lstm_ms, proj_ms, gate_table_ms;
} wind_profile_t;

/*
 * Measurement aid: the same decode as wind_decode_greedy (same kernels, same results) with the
 * time attributed to its parts.  On the plain-ALU path the loop is driven from the host in bursts
 * of steps so that every launch can be bracketed by a pair of CUDA events on `stream` (slower than
 * wind_decode_greedy: events and one synchronisation per burst).  The paper has no counterpart; its
 * timing is wall clock only.
 */
wind_status_t wind_profile_decode(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B,
                                  int32_t T, int32_t W, int32_t max_symbols, int32_t* out_tokens,
                                  int32_t* out_frames, int32_t* out_len, int32_t max_out, void* workspace,
                                  size_t workspace_bytes, void* stream, wind_profile_t* host_out);

/*
 * WIND beam search (Algorithm 3) for ONE utterance, beam K, window W.
 * A map from frames to partial hypotheses is worked off in frame order: the hypotheses of the smallest frame t are
 * recombined and pruned to K, the joint is evaluated over the window of n = min(W, T - t) frames for each of them,
 * P'(v, t) of Eq. (1) is formed and every hypothesis is expanded by its K most probable entries (a label at an
 * offset: appended, continues at t + offset; the blank entry: continues at t + n).  The most probable hypotheses
 * that reached frame T are returned, best first.
 * Recombination: hypotheses with the same tokens (and the same count of emissions on the current frame) become one
 * with their probabilities summed; then the K most probable stay.  prefix_search != 0 adds the step between the
 * two as the paper states it: for every pair (A, B) of the frame's hypotheses with A's tokens a proper prefix of B's,
 * P(A) times the probability of emitting B's extra tokens at the current frame (each under the decoder state after
 * the tokens before it) is added to B, then every such A is removed; completions use the probabilities the
 * hypotheses had when the step began.  (The paper refers to another paper for the details of this step; what is
 * built is its own sentence, taken literally.  It costs one more round of kernels and one synchronisation per extra
 * token and K pairs.)
 * max_symbols: as in wind_decode_greedy (the paper leaves its safeguard for this algorithm to its code).
 * Entries of P' are ranked by probability, then offset, then label.  Scores are natural-log probabilities; the
 * window's log-softmax is fp32, sums over steps are fp64.  K = 1 gives wind_decode_window_greedy's result.
 * The map, recombination and pruning run on the host; the model arithmetic (encoder projection, decoder updates of
 * surviving hypotheses, windowed joint, Eq. (1) and its K best entries) runs in kernels on `stream`, which the call
 * synchronises once per iteration to read K x K (label, offset, log-probability) triples.
 *   enc        DEVICE [T, D], element type m->dtype.    T >= 1, 1 <= W <= 64, 1 <= K <= 16.
 *   out_*      HOST: tokens/frames [max_hyps, max_out], lengths and scores [max_hyps], *n_hyps = hypotheses written
 *              (at most max_hyps, best first); a hypothesis longer than max_out is cut in the token arrays, its
 *              length is reported in full.  n_steps (may be null): iterations of the loop.
 *   workspace  DEVICE, at least wind_beam_workspace_bytes(m, T, W, K, max_symbols); 256-byte aligned.
 * WIND_ERR_WORKSPACE also when the pool of decoder states (sized for K (W + 2) (min(max_symbols, 32) + 2) live
 * hypotheses) runs out.
 */
wind_status_t wind_beam_workspace_bytes(const wind_model_t* m, int32_t T, int32_t W, int32_t K, int32_t max_symbols,
                                        size_t* bytes);
wind_status_t wind_beam_search(const wind_model_t* m, const void* enc, int32_t T, int32_t W, int32_t K,
                               int32_t max_symbols, int32_t prefix_search, int32_t max_hyps, int32_t max_out,
                               int32_t* out_tokens_host,
                               int32_t* out_frames_host, int32_t* out_len_host, double* out_score_host,
                               int32_t* n_hyps_host, int64_t* n_steps_host, void* workspace, size_t workspace_bytes,
                               void* stream);

/*
 * Length-aware batching of a set of N utterances (host-only; no CUDA call).  The lock-step loop of a batch runs until
 * its longest utterance is done, so batches of mixed lengths leave most rows idle for most steps: the paper's batched
 * gain shrinks as the batch grows for the same reason.  The plan sorts the utterances by length, longest first (equal
 * lengths keep their order), and cuts the sorted list into batches of B (the last one may be smaller), which
 * minimises the sum over batches of the longest length.  With several GPUs, rank r of R takes batches r, r + R, ...
 * (longest first, so that the ranks' loads differ by at most one batch of the shortest utterances).
 *   enc_len  HOST [N] int32, each >= 0.     order    HOST [N] out: utterance indices, batch after batch.
 *   batch_T  HOST [ceil(N / B)] out, may be null: longest length of each batch (the T to pack it with).
 *   n_batches HOST out.
 * WIND_ERR_INVALID_ARG: null pointer, N < 0, B < 1, a negative length.
 */
wind_status_t wind_plan_batches(const int32_t* enc_len, int32_t N, int32_t B, int32_t* order, int32_t* batch_T,
                                int32_t* n_batches);

/* Copies the counters of the last decode that used `workspace` to host memory (synchronises `stream`). */
wind_status_t wind_read_stats(const void* workspace, void* stream, wind_stats_t* host_out);

/*
 * Timeline of the persistent loop kernel (tensor-core path), a debugging and measurement aid.
 * wind_set_trace(s) makes later decodes record, for lock steps s and s + 1 (s = -1 is the start of
 * sequence), when the role threads of CTA 0 pass fixed points of each phase; s < -1 switches it off
 * (default).  Returns the previous setting.  Recording costs a few stores and does not change results.
 * wind_read_trace copies the records of the last decode that used `workspace` (same m, B, T, W).
 *   role:  0 TMA issuer, 1 MMA issuer, 2 first epilogue thread, 3 grid barrier (4..7: the same of the last CTA);
 *          8 + k: mark k of EVERY CTA in lock step s; for these records `step` holds the CTA index and `clock` the
 *          global timer in nanoseconds, which is comparable across SMs (who is last is what bounds a phase).  Marks:
 *          joint 0 entered, 1 copies of the window's enc_proj rows issued, 2 pred_proj arrived, 3 operand handed to the
 *          issuing threads, 4 accumulator ready, 5 keys out; decoder update 6 keys of the CTA's utterances complete,
 *          7 tokens known, 8 accumulator ready, 9 state written; projection 10 state counters seen, 11 accumulator
 *          ready, 12 pred_proj published, 13 / 14 the GEMM issued ahead of the decoder update (counters seen /
 *          issued), 15 done.  (The streaming mode records 5, 9 and 15: its barrier arrivals.)
 *   phase: 0 joint, 1 decoder update, 2 projection
 *   event: 0 phase entered, 1 first / 2 last TMA issued, 3 first operands arrived, 4 accumulator
 *          committed, 5 epilogue inputs requested (token known), 6 accumulator ready, 7 epilogue
 *          done, 8 barrier arrival, 9 barrier release
 *   clock: SM cycle counter of the recording CTA's SM (roles 0..7)
 */
typedef struct {
    int32_t role, phase, event, step;
    int64_t clock;
} wind_trace_event_t;
int32_t wind_set_trace(int32_t first_step);
wind_status_t wind_read_trace(const wind_model_t* m, int32_t B, int32_t T, int32_t W, const void* workspace, void* stream,
                              wind_trace_event_t* host_out, int32_t capacity, int32_t* n_out);

/*
 * Measurement aid: the joint phase of the decoding loop by itself.  The loop kernel (the one that reads the joint's
 * activations from the workspace: resident weights with grid barriers, or streamed weights, as the planner chooses for
 * the shapes) runs ONLY its joint phase, `iters` times back to back, every CTA for itself, on fixed activations of all
 * B * W window rows: the W_out contraction on tensor cores, the per-row argmax and the 64-bit key combine, exactly the
 * code of a lock step's joint phase without the phases around it.  Timed with two CUDA events on `stream` around one
 * launch (a short untimed launch goes first).  The paper has no counterpart; it is how the share of the tensor peak the
 * joint can reach at a given size is told apart from the latency chain of the loop.
 *   workspace  device, at least wind_workspace_bytes(m, B, 1, W); the model needs valid weight pointers.
 *   host_out   ms for the timed launch; rows = B * W (algorithmic), rows_issued / labels_issued = what the tiles cover
 *              (padding included); resident = which kernel ran; ctas = CTAs that had a joint item.
 * flop per iteration: 2 * H * (V + 1) * rows (algorithmic), 2 * H * labels_issued * rows_issued (issued).
 */
typedef struct {
    double ms;
    int64_t rows, rows_issued, labels_issued;
    int32_t iters, resident, ctas, reserved;
} wind_joint_bench_t;
wind_status_t wind_bench_joint(const wind_model_t* m, int32_t B, int32_t W, int32_t iters, void* workspace, size_t workspace_bytes,
                               void* stream, wind_joint_bench_t* host_out);

/*
 * Test hook for the failure path of the persistent loop kernel: with extra_arrivals > 0 its grid barrier waits
 * for that many arrivals more than there are CTAs, so the first barrier of the next decode can never fill.  Every
 * wait in the kernel is bounded (about two seconds), so the decode then ends by itself: the CTAs give up, free
 * their tensor memory and return, and the call reports WIND_ERR_TIMEOUT with undefined outputs; the CUDA context
 * stays usable.  0 restores normal operation.  Returns the previous value.  The paper has no counterpart (its only
 * mention of a safeguard is the beam-search footnote about not staying on one frame forever).
 */
int32_t wind_debug_stall_barrier(int32_t extra_arrivals);

/*
 * Options of the tensor-core loop's tile planner, process-wide (defaults: 1, -1, 4, -1).  Meant for tests and
 * measurements, which use them to reach every mode of the loop kernels on one shape; results do not depend on them.
 *   resident         0: never choose the resident-weights mode (weights then stream through shared memory every
 *                    step, as for shapes whose tiles do not fit on chip)
 *   joint_placement  streaming mode only: where a CTA keeps its W_out tile when it owns one joint item: -1 the
 *                    planner's choice, 0 streamed every step, 1 shared memory, 2 tensor memory (taken when feasible)
 *   max_joint_waves  resident mode: most passes over row groups the joint may take per step (1..4)
 *   dataflow         resident mode: which of its two kernels runs.  0: the phases of a lock step are separated by grid
 *                    barriers.  1: no grid barrier; CTAs hand results on through per-group arrival counters and stamped
 *                    data, and a joint CTA builds its own operand from pred_proj and prefetched enc_proj rows.
 *                    -1: the planner's choice (the second for one-layer models and batches up to 64 utterances,
 *                    where it measures faster; the first beyond).  The two give the same transcripts.
 */
void wind_set_loop_options(int32_t resident, int32_t joint_placement, int32_t max_joint_waves, int32_t dataflow);

/*
 * The tile plan the tensor-core loop would use for a model and batch on a device with `sms` multiprocessors and
 * `smem_optin` bytes of opt-in shared memory per block: host arithmetic only, no CUDA call, so that the plan's
 * invariants (every shared-memory region inside smem_bytes, tensor-memory columns within 512, disjoint CTA sets
 * inside the grid) can be checked over many shapes without a GPU.  WIND_ERR_UNSUPPORTED: the shapes are outside the
 * tensor-core path (dimensions not multiples of 64, fewer than 128 logits) or nothing fits.
 * Resident mode (resident = 1; dataflow: which of its two kernels): CTAs [0, l_sets * l_items) hold decoder tiles (l_items = ut_count unit tiles x ql_count
 * utterance groups of nl), the last p_items = ht_count x qp_count CTAs hold W_pred tiles (np utterances each), CTAs
 * [w_first, w_first + w_count) record the steps; shared memory of a CTA: tile_bytes at 0, the state box at buf_off, the
 * joint's operand (nj rows x H) at z_off (z_off_p in W_pred CTAs), staging from stage_off to smem_bytes - 1024.
 * Streaming mode: rings of stages_lp x stage_lp and stages_j x stage_j bytes behind tile_bytes.
 */
typedef struct {
    int32_t grid, resident, dataflow, smem_bytes;
    int32_t nj, vt_count, rg_count, rg_stride, j_mode;
    int32_t tm_j, tm_l, tm_p;
    int32_t nl, np, ut_count, ht_count, ql_count, qp_count, l_items, p_items, w_first, w_count, l_sets;
    int32_t tile_bytes, buf_off, z_off, z_off_p, stage_off;
    int32_t slots, ul, ug_count, mt_count, hg_count, stages_lp, stages_j, stage_lp, stage_j;
} wind_plan_t;
wind_status_t wind_debug_plan(const wind_model_t* m, int32_t B, int32_t W, int32_t sms, int32_t smem_optin, wind_plan_t* out);

/* Process-wide choice of kernels for the bf16 path (default AUTO).  Returns the previous value. */
int32_t wind_set_kernels(int32_t kernels);

/* Human-readable name of a status code (static string). */
const char* wind_status_string(wind_status_t s);

/* Text of the last CUDA error seen by this thread inside the library (static/thread-local string). */
const char* wind_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* WIND_H_ */
