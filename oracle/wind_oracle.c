/*
 * CPU oracle for greedy RNN-Transducer decoding: the sequential frame-by-frame
 * procedure (Algorithm 1, "RNN-T Inference Algorithm") and windowed decoding
 * (Algorithm 2, "WIND Algorithm").
 *
 * THIS IS TEST INFRASTRUCTURE.  It is deliberately plain and slow: nested loops,
 * every sum accumulated in fp64 in index order, no blocking, no SIMD, no BLAS.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may call
 * it; the CUDA library shares no code with it.
 *
 * Model (the paper treats decoder and joiner as black boxes; Section "Background:
 * RNN-T" only fixes their roles):
 *   decoder  = embedding table + L-layer LSTM (gate order i,f,g,o; two bias
 *              vectors; zero initial state), fed ONE token per update; the
 *              start-of-sequence input is the blank id;
 *   joiner   = W_out * act(W_enc*f + b_enc + W_pred*h_top + b_pred) + b_out,
 *              act = ReLU or tanh; argmax is taken on the logits (softmax is
 *              monotone), lowest index winning ties.
 *
 * Safeguard against staying on one frame forever ("max symbols per frame", S):
 * a counter of consecutive emissions on the current frame; when it reaches S
 * the S-th token is still emitted and fed to the decoder, then t advances by
 * one.  The counter resets whenever t advances.
 *
 * The file also holds Eq. (1) (first-output distribution of a window) and window-based greedy decoding, which
 * takes the most probable (label, offset) pair of Eq. (1) at every step; their pins: the distribution sums to
 * one, closed forms, W = 1 equals Algorithm 1, a step-by-step recomputation from Eq. (1) in the tests, and a
 * hand-worked example where it differs from Algorithm 2; and Algorithm 3 (beam search for one utterance), pinned
 * by: beam 1 equals window-based greedy decoding, an unpruned beam gives every token sequence its total probability
 * over all alignments for every window (brute force on independently evaluated logits), hand-worked examples, and
 * the optional prefix step against independently evaluated completions.
 *
 * Precision: fp64 throughout by default.  With round_bf16 set in the model, enc_proj, the LSTM hidden state and the joint's
 * activations are rounded to bf16 where they are produced and everything else stays fp64 (the paper runs its models under
 * bf16 autocast and names no rounding points; these three are the matrix operands of a bf16 implementation).  Pins of this
 * mode: the rounding against a library conversion, and each of the three places against a step-by-step recomputation.
 *
 * Pins (see tests): WIND(W) == sequential for every W; brute-force tabulation
 * of joint argmaxes on tiny models; LSTM / linear layers against library fp64
 * routines and closed forms; S honoured; jump-size support.
 * The paper prints no worked numeric example, so token-level agreement with the
 * paper's own runs is "parity unpinned"; the pins above are what fixes this code.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t D, E, P, L, H, V;
    int32_t blank_id;
    int32_t act; /* 0 = ReLU, 1 = tanh */
    const float* emb;         /* [V+1, E] */
    const float* const* w_ih; /* L x [4P, in_l], in_0 = E, in_l = P */
    const float* const* w_hh; /* L x [4P, P] */
    const float* const* b_ih; /* L x [4P] */
    const float* const* b_hh; /* L x [4P] */
    const float* w_enc;       /* [H, D] */
    const float* b_enc;       /* [H] */
    const float* w_pred;      /* [H, P] */
    const float* b_pred;      /* [H] */
    const float* w_out;       /* [V+1, H] */
    const float* b_out;       /* [V+1] */
    int32_t round_bf16;       /* 0: fp64 throughout.  1: the three intermediate quantities that a bf16 implementation keeps
                                 as matrix operands -- enc_proj, the LSTM hidden state h, and the joint's activations
                                 act(enc_proj + pred_proj) -- are rounded to bf16 (nearest even) where they are produced;
                                 everything else (sums, cell state c, pred_proj, logits) stays fp64.  The paper runs its
                                 models under bf16 autocast and fixes no rounding points; these are the ones a decision
                                 taken "in the kernel's precision" has to share. */
} oracle_model_t;

typedef struct {
    int64_t steps;          /* loop iterations (joint evaluations) */
    int64_t joint_rows;     /* joint rows evaluated */
    int64_t pred_updates;   /* decoder updates, excluding the start-of-sequence one */
    int64_t forced;         /* forced advances by the S rule */
    int64_t low_margin;     /* decisions whose top-2 logit margin < margin_thr */
    int64_t decisions;      /* frame-level decisions taken (Alg. 1 sense) */
    int64_t emit_frames;    /* frames with at least one emission */
    int64_t jump_hist[65];  /* jump sizes 0..64 (WIND only; W <= 64 recorded) */
} oracle_stats_t;

/* ------------------------------------------------------------------------- */
/* y = W x + b, W [n_out, n_in] fp32 row-major, x fp64, fp64 accumulate       */
/* ------------------------------------------------------------------------- */
void oracle_linear(const float* W, const float* b, const double* x, int n_out, int n_in, double* y) {
    for (int o = 0; o < n_out; ++o) {
        double acc = b ? (double)b[o] : 0.0;
        const float* row = W + (size_t)o * n_in;
        for (int k = 0; k < n_in; ++k) acc += (double)row[k] * x[k];
        y[o] = acc;
    }
}

static double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }

/* nearest bf16 value (ties to even) of x: fp32 first, then the upper 16 bits of its pattern */
double oracle_bf16_round(double x) {
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, sizeof(u));
    if ((u & 0x7F800000u) == 0x7F800000u) return (double)f;   /* infinities and NaN pass */
    u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    memcpy(&f, &u, sizeof(f));
    return (double)f;
}

/*
 * One LSTM stack update for one token.  h, c: [L, P] fp64, updated in place.
 * Layer l: gates = W_ih x + b_ih + W_hh h + b_hh, split as (i, f, g, o);
 * c <- sigma(f)*c + sigma(i)*tanh(g); h <- sigma(o)*tanh(c); x of layer l+1 is
 * the new h of layer l.
 */
void oracle_lstm_step(const oracle_model_t* m, int32_t tok, double* h, double* c) {
    const int P = m->P;
    double* x = (double*)malloc(sizeof(double) * (size_t)(m->E > P ? m->E : P));
    double* ga = (double*)malloc(sizeof(double) * 4 * (size_t)P);
    double* gb = (double*)malloc(sizeof(double) * 4 * (size_t)P);
    for (int k = 0; k < m->E; ++k) x[k] = (double)m->emb[(size_t)tok * m->E + k];
    int n_in = m->E;
    for (int l = 0; l < m->L; ++l) {
        double* hl = h + (size_t)l * P;
        double* cl = c + (size_t)l * P;
        oracle_linear(m->w_ih[l], m->b_ih[l], x, 4 * P, n_in, ga);
        oracle_linear(m->w_hh[l], m->b_hh[l], hl, 4 * P, P, gb);
        for (int j = 0; j < P; ++j) {
            double gi = sigmoid(ga[j] + gb[j]);
            double gf = sigmoid(ga[P + j] + gb[P + j]);
            double gg = tanh(ga[2 * P + j] + gb[2 * P + j]);
            double go = sigmoid(ga[3 * P + j] + gb[3 * P + j]);
            cl[j] = gf * cl[j] + gi * gg;
            hl[j] = go * tanh(cl[j]);
            if (m->round_bf16) hl[j] = oracle_bf16_round(hl[j]);
        }
        for (int j = 0; j < P; ++j) x[j] = hl[j];
        n_in = P;
    }
    free(x); free(ga); free(gb);
}

/* pred_proj = W_pred h_top + b_pred */
void oracle_pred_proj(const oracle_model_t* m, const double* h, double* g) {
    oracle_linear(m->w_pred, m->b_pred, h + (size_t)(m->L - 1) * m->P, m->H, m->P, g);
}

/* enc_proj[t,:] = W_enc enc[t,:] + b_enc for t < T */
void oracle_enc_proj(const oracle_model_t* m, const float* enc, int T, double* out) {
    double* x = (double*)malloc(sizeof(double) * (size_t)m->D);
    for (int t = 0; t < T; ++t) {
        for (int k = 0; k < m->D; ++k) x[k] = (double)enc[(size_t)t * m->D + k];
        oracle_linear(m->w_enc, m->b_enc, x, m->H, m->D, out + (size_t)t * m->H);
        if (m->round_bf16)
            for (int k = 0; k < m->H; ++k) out[(size_t)t * m->H + k] = oracle_bf16_round(out[(size_t)t * m->H + k]);
    }
    free(x);
}

/* logits = W_out act(encp + g) + b_out ; z is scratch [H] */
void oracle_joint_logits(const oracle_model_t* m, const double* encp, const double* g, double* z, double* logits) {
    for (int k = 0; k < m->H; ++k) {
        double s = encp[k] + g[k];
        z[k] = (m->act == 0) ? (s > 0.0 ? s : 0.0) : tanh(s);
        if (m->round_bf16) z[k] = oracle_bf16_round(z[k]);
    }
    oracle_linear(m->w_out, m->b_out, z, m->V + 1, m->H, logits);
}

/* lowest index on ties; also returns the top-2 margin */
static int argmax_margin(const double* v, int n, double* margin) {
    int best = 0;
    for (int i = 1; i < n; ++i)
        if (v[i] > v[best]) best = i;
    double second = -INFINITY;
    for (int i = 0; i < n; ++i)
        if (i != best && v[i] > second) second = v[i];
    if (margin) *margin = v[best] - second;
    return best;
}

typedef struct {
    double *h, *c, *g, *z, *logits, *encp;
} scratch_t;

static void scratch_alloc(const oracle_model_t* m, int T, scratch_t* s) {
    s->h = (double*)calloc((size_t)m->L * m->P, sizeof(double));
    s->c = (double*)calloc((size_t)m->L * m->P, sizeof(double));
    s->g = (double*)malloc(sizeof(double) * (size_t)m->H);
    s->z = (double*)malloc(sizeof(double) * (size_t)m->H);
    s->logits = (double*)malloc(sizeof(double) * (size_t)(m->V + 1) * 64);
    s->encp = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1) * m->H);
}
static void scratch_free(scratch_t* s) {
    free(s->h); free(s->c); free(s->g); free(s->z); free(s->logits); free(s->encp);
}

/* start of sequence: zero state, feed the blank id once */
static void decoder_start(const oracle_model_t* m, scratch_t* s) {
    memset(s->h, 0, sizeof(double) * (size_t)m->L * m->P);
    memset(s->c, 0, sizeof(double) * (size_t)m->L * m->P);
    oracle_lstm_step(m, m->blank_id, s->h, s->c);
    oracle_pred_proj(m, s->h, s->g);
}
static void decoder_feed(const oracle_model_t* m, scratch_t* s, int32_t tok) {
    oracle_lstm_step(m, tok, s->h, s->c);
    oracle_pred_proj(m, s->h, s->g);
}

/*
 * Algorithm 1: one frame, one decision per iteration.
 * Returns the number of tokens (may exceed max_out; only the first max_out are stored).
 */
int32_t oracle_decode_seq(const oracle_model_t* m, const float* enc, int32_t T, int32_t S, double margin_thr,
                          int32_t* out_tokens, int32_t* out_frames, int32_t max_out, oracle_stats_t* st) {
    scratch_t s;
    scratch_alloc(m, T, &s);
    oracle_enc_proj(m, enc, T, s.encp);
    decoder_start(m, &s);
    int32_t n_out = 0, t = 0, count = 0, last_emit_frame = -1;
    while (t < T) {
        oracle_joint_logits(m, s.encp + (size_t)t * m->H, s.g, s.z, s.logits);
        double margin;
        int label = argmax_margin(s.logits, m->V + 1, &margin);
        if (st) {
            st->steps++; st->joint_rows++; st->decisions++;
            if (margin < margin_thr) st->low_margin++;
        }
        if (label != m->blank_id) {
            if (n_out < max_out) { out_tokens[n_out] = label; out_frames[n_out] = t; }
            n_out++;
            if (st) { st->pred_updates++; if (t != last_emit_frame) st->emit_frames++; }
            last_emit_frame = t;
            decoder_feed(m, &s, label);
            count++;
            if (count == S) { t += 1; count = 0; if (st) st->forced++; }
        } else {
            t += 1;
            count = 0;
        }
    }
    scratch_free(&s);
    return n_out;
}

/*
 * Algorithm 2: n = min(W, T - t) frames share the current decoder state.
 * All blank: t += n.  Otherwise i = first non-blank row, emit labels[i] at
 * frame t+i and set t += i (the next window starts ON the emitting frame).
 */
int32_t oracle_decode_wind(const oracle_model_t* m, const float* enc, int32_t T, int32_t W, int32_t S,
                           double margin_thr, int32_t* out_tokens, int32_t* out_frames, int32_t max_out,
                           oracle_stats_t* st) {
    if (W < 1 || W > 64) return -1;
    scratch_t s;
    scratch_alloc(m, T, &s);
    oracle_enc_proj(m, enc, T, s.encp);
    decoder_start(m, &s);
    const int NV = m->V + 1;
    int32_t n_out = 0, t = 0, count = 0, last_emit_frame = -1;
    int labels[64];
    double margins[64];
    while (t < T) {
        int n = (W < T - t) ? W : (T - t);
        for (int w = 0; w < n; ++w) {
            oracle_joint_logits(m, s.encp + (size_t)(t + w) * m->H, s.g, s.z, s.logits + (size_t)w * NV);
            labels[w] = argmax_margin(s.logits + (size_t)w * NV, NV, &margins[w]);
        }
        if (st) { st->steps++; st->joint_rows += n; }
        int i = -1;
        for (int w = 0; w < n; ++w)
            if (labels[w] != m->blank_id) { i = w; break; }
        if (i < 0) {
            if (st) {
                st->jump_hist[n]++;
                st->decisions += n;
                for (int w = 0; w < n; ++w) if (margins[w] < margin_thr) st->low_margin++;
            }
            t += n;
            count = 0;
            continue;
        }
        if (st) {
            st->jump_hist[i]++;
            st->decisions += i + 1;
            for (int w = 0; w <= i; ++w) if (margins[w] < margin_thr) st->low_margin++;
        }
        if (i > 0) count = 0;
        t += i;
        if (n_out < max_out) { out_tokens[n_out] = labels[i]; out_frames[n_out] = t; }
        n_out++;
        if (st) { st->pred_updates++; if (t != last_emit_frame) st->emit_frames++; }
        last_emit_frame = t;
        decoder_feed(m, &s, labels[i]);
        count++;
        if (count == S) { t += 1; count = 0; if (st) st->forced++; }
    }
    scratch_free(&s);
    return n_out;
}

/*
 * Batched front end: utterances are independent, so this is a plain loop over
 * them (OpenMP across utterances only).  W == 0 selects Algorithm 1.
 * enc [B, T, D]; out_tokens/out_frames [B, max_out]; out_len [B]; stats summed.
 */
void oracle_decode_batch(const oracle_model_t* m, const float* enc, const int32_t* enc_len, int32_t B, int32_t T,
                         int32_t W, int32_t S, double margin_thr, int32_t* out_tokens, int32_t* out_frames,
                         int32_t* out_len, int32_t max_out, oracle_stats_t* st_total) {
    oracle_stats_t* sts = (oracle_stats_t*)calloc((size_t)B, sizeof(oracle_stats_t));
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const float* e = enc + (size_t)b * T * m->D;
        int32_t* ot = out_tokens + (size_t)b * max_out;
        int32_t* of = out_frames + (size_t)b * max_out;
        if (W == 0)
            out_len[b] = oracle_decode_seq(m, e, enc_len[b], S, margin_thr, ot, of, max_out, &sts[b]);
        else
            out_len[b] = oracle_decode_wind(m, e, enc_len[b], W, S, margin_thr, ot, of, max_out, &sts[b]);
    }
    if (st_total) {
        memset(st_total, 0, sizeof(*st_total));
        for (int b = 0; b < B; ++b) {
            st_total->steps += sts[b].steps;
            st_total->joint_rows += sts[b].joint_rows;
            st_total->pred_updates += sts[b].pred_updates;
            st_total->forced += sts[b].forced;
            st_total->low_margin += sts[b].low_margin;
            st_total->decisions += sts[b].decisions;
            st_total->emit_frames += sts[b].emit_frames;
            for (int k = 0; k < 65; ++k) st_total->jump_hist[k] += sts[b].jump_hist[k];
        }
    }
    free(sts);
}

/* forward declaration: defined at the end of the file */
int32_t oracle_decode_window_greedy(const oracle_model_t* m, const float* enc, int32_t T, int32_t W, int32_t S,
                                    double margin_thr, int32_t* out_tokens, int32_t* out_frames, int32_t max_out,
                                    oracle_stats_t* st);

/* Window-based greedy decoding of a batch: the same plain loop over utterances. */
void oracle_decode_window_greedy_batch(const oracle_model_t* m, const float* enc, const int32_t* enc_len, int32_t B,
                                       int32_t T, int32_t W, int32_t S, double margin_thr, int32_t* out_tokens,
                                       int32_t* out_frames, int32_t* out_len, int32_t max_out, oracle_stats_t* st_total) {
    oracle_stats_t* sts = (oracle_stats_t*)calloc((size_t)B, sizeof(oracle_stats_t));
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        out_len[b] = oracle_decode_window_greedy(m, enc + (size_t)b * T * m->D, enc_len[b], W, S, margin_thr,
                                                 out_tokens + (size_t)b * max_out, out_frames + (size_t)b * max_out,
                                                 max_out, &sts[b]);
    if (st_total) {
        memset(st_total, 0, sizeof(*st_total));
        for (int b = 0; b < B; ++b) {
            st_total->steps += sts[b].steps;
            st_total->joint_rows += sts[b].joint_rows;
            st_total->pred_updates += sts[b].pred_updates;
            st_total->forced += sts[b].forced;
            st_total->low_margin += sts[b].low_margin;
            st_total->decisions += sts[b].decisions;
            for (int k = 0; k < 65; ++k) st_total->jump_hist[k] += sts[b].jump_hist[k];
        }
    }
    free(sts);
}

/*
 * Replay check of a (token, frame) sequence produced elsewhere against the
 * sequential definition.  Walk frames from 0; the sequence implies one choice
 * at every decision of Algorithm 1 (the listed token at its frame, blank at
 * every frame that is left without having hit the S cap).  Each implied choice
 * must be the oracle's argmax, or its oracle logit must lie within
 * `margin_thr` of the oracle's maximum (a low-margin decision: counted).
 * Returns 0 when consistent, else a positive code; *bad_pos gets the frame.
 *   1: implied choice loses by more than the margin
 *   2: frames not non-decreasing / out of range / more than S tokens on a frame
 *   3: token out of range or equal to blank
 */
int32_t oracle_replay_verify(const oracle_model_t* m, const float* enc, int32_t T, int32_t S, double margin_thr,
                             const int32_t* tokens, const int32_t* frames, int32_t n, int64_t* n_decisions,
                             int64_t* n_low_margin, int64_t* n_not_argmax, int32_t* bad_pos) {
    scratch_t s;
    scratch_alloc(m, T, &s);
    oracle_enc_proj(m, enc, T, s.encp);
    decoder_start(m, &s);
    int32_t rc = 0, t = 0, count = 0, idx = 0;
    int64_t dec = 0, low = 0, notmax = 0;
    for (int k = 0; k < n && !rc; ++k) {
        if (tokens[k] < 0 || tokens[k] > m->V || tokens[k] == m->blank_id) { rc = 3; *bad_pos = k; }
        if (frames[k] < 0 || frames[k] >= T || (k > 0 && frames[k] < frames[k - 1])) { rc = 2; *bad_pos = k; }
    }
    while (!rc && t < T) {
        oracle_joint_logits(m, s.encp + (size_t)t * m->H, s.g, s.z, s.logits);
        double margin;
        int best = argmax_margin(s.logits, m->V + 1, &margin);
        int choice = (idx < n && frames[idx] == t) ? tokens[idx] : m->blank_id;
        if (idx < n && frames[idx] < t) { rc = 2; *bad_pos = t; break; }
        dec++;
        if (margin < margin_thr) low++;
        if (choice != best) {
            notmax++;
            if (!(s.logits[choice] >= s.logits[best] - margin_thr)) { rc = 1; *bad_pos = t; break; }
        }
        if (choice != m->blank_id) {
            decoder_feed(m, &s, choice);
            idx++;
            count++;
            if (count == S) { t += 1; count = 0; }
        } else {
            t += 1;
            count = 0;
        }
    }
    if (!rc && idx != n) { rc = 2; *bad_pos = T; }
    if (n_decisions) *n_decisions = dec;
    if (n_low_margin) *n_low_margin = low;
    if (n_not_argmax) *n_not_argmax = notmax;
    scratch_free(&s);
    return rc;
}

/*
 * Teacher-forced window logits: feed `prefix` (after the start-of-sequence
 * blank) to the decoder, then evaluate the joint at frames t0 .. t0+n-1,
 * n = min(W, T - t0).  logits [W, V+1] fp64; rows >= n are left untouched.
 * Optionally returns pred_proj (g, [H]) and the top-layer state.
 */
int32_t oracle_eval_joint_window(const oracle_model_t* m, const float* enc, int32_t T, const int32_t* prefix,
                                 int32_t prefix_len, int32_t t0, int32_t W, double* logits, double* g_out,
                                 double* h_out, double* c_out) {
    scratch_t s;
    scratch_alloc(m, 0, &s);
    decoder_start(m, &s);
    for (int k = 0; k < prefix_len; ++k) decoder_feed(m, &s, prefix[k]);
    int n = (W < T - t0) ? W : (T - t0);
    if (n < 0) n = 0;
    double* ep = (double*)malloc(sizeof(double) * (size_t)m->H);
    for (int w = 0; w < n; ++w) {
        oracle_enc_proj(m, enc + (size_t)(t0 + w) * m->D, 1, ep);
        oracle_joint_logits(m, ep, s.g, s.z, logits + (size_t)w * (m->V + 1));
    }
    if (g_out) memcpy(g_out, s.g, sizeof(double) * (size_t)m->H);
    if (h_out) memcpy(h_out, s.h, sizeof(double) * (size_t)m->L * m->P);
    if (c_out) memcpy(c_out, s.c, sizeof(double) * (size_t)m->L * m->P);
    free(ep);
    scratch_free(&s);
    return n;
}

/*
 * Eq. (1): P'(v, t), the probability that v is the FIRST output in the window that starts at frame t0,
 * emitted at frame t0 + t, under the current decoder state:
 *   v != blank: P(v | t0 + t) * prod_{t' < t} P(blank | t0 + t')
 *   v == blank: 0 for t < n - 1, and prod_{t' <= n - 1} P(blank | t0 + t') for t = n - 1
 * with P(. | frame) = softmax of the joint's logits and n = min(W, T - t0) rows in the window (the paper writes
 * the window size w; at the end of an utterance the window is the truncated one of Algorithm 3, n = min(N, T - t)).
 * Output: natural-log probabilities, logp [n, V+1] (-INFINITY for the zero entries).  Returns n.
 * Plain steps: logits (teacher-forced prefix), log-softmax per row, running sum of the blank log-probabilities.
 */
int32_t oracle_first_output_logprobs(const oracle_model_t* m, const float* enc, int32_t T, const int32_t* prefix,
                                     int32_t prefix_len, int32_t t0, int32_t W, double* logp) {
    const int NV = m->V + 1;
    double* logits = (double*)malloc(sizeof(double) * (size_t)(W > 0 ? W : 1) * NV);
    const int n = oracle_eval_joint_window(m, enc, T, prefix, prefix_len, t0, W, logits, NULL, NULL, NULL);
    double blanks_before = 0.0; /* sum of log P(blank | t0 + t') for t' < t */
    for (int t = 0; t < n; ++t) {
        const double* row = logits + (size_t)t * NV;
        double mx = row[0];
        for (int v = 1; v < NV; ++v)
            if (row[v] > mx) mx = row[v];
        double se = 0.0;
        for (int v = 0; v < NV; ++v) se += exp(row[v] - mx);
        const double lse = mx + log(se);
        for (int v = 0; v < NV; ++v) {
            const double lp = row[v] - lse; /* log P(v | t0 + t) */
            if (v != m->blank_id)
                logp[(size_t)t * NV + v] = lp + blanks_before;
            else
                logp[(size_t)t * NV + v] = (t == n - 1) ? lp + blanks_before : -INFINITY;
        }
        blanks_before += row[m->blank_id] - lse;
    }
    free(logits);
    return n;
}

/*
 * Window-based greedy decoding: at every step the window's first-output distribution P'(v, t) of Eq. (1) is
 * evaluated under the current decoder state and the single most probable (label, offset) pair is taken
 * (the variant sketched beside Algorithm 2: "find the best prediction based on the whole window").
 *   pair (v != blank, j): emit v at frame t + j, then t += j (the next window starts ON the emitting frame);
 *   blank (only at the window's last row, i.e. the window is all blank): t += n.
 * Candidates are compared in the order j ascending, label ascending, the all-blank candidate last; the first
 * strict maximum wins.  The safeguard against staying on one frame is the one of the greedy decoders above.
 * Unlike Algorithm 2 the result depends on W (W = 1 is Algorithm 1).
 *
 * window_scores(): log P' restricted to what the decision needs, from the logits of the n rows:
 *   best[j]   = log P'(v_j, j) for the best non-blank label v_j of row j,
 *   *all_blank = log P'(blank, n - 1).
 */
static void window_scores(const oracle_model_t* m, const double* logits, int n, double* best, int* best_label,
                          double* all_blank) {
    const int NV = m->V + 1;
    double blanks_before = 0.0;
    for (int j = 0; j < n; ++j) {
        const double* row = logits + (size_t)j * NV;
        double mx = row[0];
        for (int v = 1; v < NV; ++v)
            if (row[v] > mx) mx = row[v];
        double se = 0.0;
        for (int v = 0; v < NV; ++v) se += exp(row[v] - mx);
        const double lse = mx + log(se);
        int bl = -1;
        for (int v = 0; v < NV; ++v)
            if (v != m->blank_id && (bl < 0 || row[v] > row[bl])) bl = v;
        best_label[j] = bl;
        best[j] = blanks_before + row[bl] - lse;
        blanks_before += row[m->blank_id] - lse;
    }
    *all_blank = blanks_before;
}

int32_t oracle_decode_window_greedy(const oracle_model_t* m, const float* enc, int32_t T, int32_t W, int32_t S,
                                    double margin_thr, int32_t* out_tokens, int32_t* out_frames, int32_t max_out,
                                    oracle_stats_t* st) {
    if (W < 1 || W > 64) return -1;
    scratch_t s;
    scratch_alloc(m, T, &s);
    oracle_enc_proj(m, enc, T, s.encp);
    decoder_start(m, &s);
    const int NV = m->V + 1;
    double* logits = (double*)malloc(sizeof(double) * (size_t)W * NV);
    int32_t n_out = 0, t = 0, count = 0;
    while (t < T) {
        const int n = (W < T - t) ? W : (T - t);
        for (int w = 0; w < n; ++w)
            oracle_joint_logits(m, s.encp + (size_t)(t + w) * m->H, s.g, s.z, logits + (size_t)w * NV);
        double best[64], all_blank;
        int best_label[64];
        window_scores(m, logits, n, best, best_label, &all_blank);
        int pick = -1; /* row of the chosen pair, -1 = all blank */
        double top = -INFINITY, second = -INFINITY;
        for (int j = 0; j <= n; ++j) {
            const double sc = j < n ? best[j] : all_blank;
            if (sc > top) { second = top; top = sc; pick = j < n ? j : -1; }
            else if (sc > second) second = sc;
        }
        if (st) {
            st->steps++;
            st->joint_rows += n;
            st->decisions++;
            if (top - second < margin_thr) st->low_margin++;
            st->jump_hist[pick < 0 ? n : pick]++;
        }
        if (pick < 0) { t += n; count = 0; continue; }
        if (pick > 0) count = 0;
        t += pick;
        if (n_out < max_out) { out_tokens[n_out] = best_label[pick]; out_frames[n_out] = t; }
        n_out++;
        if (st) st->pred_updates++;
        decoder_feed(m, &s, best_label[pick]);
        count++;
        if (count == S) { t += 1; count = 0; if (st) st->forced++; }
    }
    free(logits);
    scratch_free(&s);
    return n_out;
}

/*
 * Replay check of a (token, frame) sequence produced elsewhere against window-based greedy decoding with the
 * same W and S.  At every step the sequence implies one candidate: the next listed token if its frame lies
 * inside the current window, else "all blank".  The implied candidate's log P' must be the maximum over the
 * window's candidates, or lie within margin_thr of it (counted in *n_not_argmax when it is not the oracle's pick).
 * The label of a pair must be the row's best non-blank label or within margin_thr of it in that row's logits.
 * Return codes as in oracle_replay_verify.
 */
int32_t oracle_replay_verify_window(const oracle_model_t* m, const float* enc, int32_t T, int32_t W, int32_t S,
                                    double margin_thr, const int32_t* tokens, const int32_t* frames, int32_t n_tok,
                                    int64_t* n_decisions, int64_t* n_low_margin, int64_t* n_not_argmax,
                                    int32_t* bad_pos) {
    if (W < 1 || W > 64) return -1;
    scratch_t s;
    scratch_alloc(m, T, &s);
    oracle_enc_proj(m, enc, T, s.encp);
    decoder_start(m, &s);
    const int NV = m->V + 1;
    double* logits = (double*)malloc(sizeof(double) * (size_t)W * NV);
    int32_t rc = 0, t = 0, count = 0, idx = 0;
    int64_t dec = 0, low = 0, notmax = 0;
    for (int k = 0; k < n_tok && !rc; ++k) {
        if (tokens[k] < 0 || tokens[k] > m->V || tokens[k] == m->blank_id) { rc = 3; *bad_pos = k; }
        if (frames[k] < 0 || frames[k] >= T || (k > 0 && frames[k] < frames[k - 1])) { rc = 2; *bad_pos = k; }
    }
    while (!rc && t < T) {
        const int n = (W < T - t) ? W : (T - t);
        for (int w = 0; w < n; ++w)
            oracle_joint_logits(m, s.encp + (size_t)(t + w) * m->H, s.g, s.z, logits + (size_t)w * NV);
        double best[64], all_blank;
        int best_label[64];
        window_scores(m, logits, n, best, best_label, &all_blank);
        double top = all_blank, second = -INFINITY;
        int pick = -1;
        for (int j = 0; j < n; ++j) {
            if (best[j] > top) { second = top; top = best[j]; pick = j; }
            else if (best[j] > second) second = best[j];
        }
        if (idx < n_tok && frames[idx] < t) { rc = 2; *bad_pos = t; break; }
        const int j = (idx < n_tok && frames[idx] < t + n) ? frames[idx] - t : -1;
        dec++;
        if (top - second < margin_thr) low++;
        if (j < 0) {
            if (pick >= 0) {
                notmax++;
                if (!(all_blank >= top - margin_thr)) { rc = 1; *bad_pos = t; break; }
            }
            t += n;
            count = 0;
            continue;
        }
        const int v = tokens[idx];
        const double* row = logits + (size_t)j * NV;
        const double sc = best[j] + (row[v] - row[best_label[j]]); /* log P'(v, j) */
        if (j != pick || v != best_label[j]) {
            notmax++;
            if (!(sc >= top - margin_thr)) { rc = 1; *bad_pos = t; break; }
        }
        if (j > 0) count = 0;
        t += j;
        decoder_feed(m, &s, v);
        idx++;
        count++;
        if (count == S) { t += 1; count = 0; }
    }
    if (!rc && idx != n_tok) { rc = 2; *bad_pos = T; }
    if (n_decisions) *n_decisions = dec;
    if (n_low_margin) *n_low_margin = low;
    if (n_not_argmax) *n_not_argmax = notmax;
    free(logits);
    scratch_free(&s);
    return rc;
}

/*
 * Algorithm 3, "WIND Beam-search Algorithm", for one utterance.
 *
 * A hypothesis is (tokens, score) plus what this code needs to continue it: the frame of every token, the decoder
 * state after its tokens, and the count of consecutive emissions on its current frame.  t2hyps maps a frame t to the
 * hypotheses that have been decoded up to t.  Every iteration takes the smallest t, recombines and prunes its
 * hypotheses to the beam K, evaluates the joint over the window of n = min(W, T - t) frames for each of them, forms
 * P'(v, t) of Eq. (1) and expands each hypothesis by its K most probable entries:
 *   (v != blank, jump): tokens + [v], score + log P'(v, jump), goes to t + jump;
 *   blank (row n - 1):  same tokens, score + log P'(blank, n - 1), goes to t + n.
 * The best hypothesis of t2hyps[T] is the result.
 *
 * recombine_prune, as far as the paper states it without the cited prefix-search paper: (1) hypotheses with the
 * same tokens become one, their probabilities summed (the frames of the more probable one are kept; the decoder
 * states are equal).  Two hypotheses with the same tokens but different counts of emissions on the current frame
 * are NOT the same under the safeguard (they may continue differently), so they stay apart: with this reading a beam
 * that never prunes gives every token sequence its total probability over all alignments, for every window;
 * (3) the K most probable stay.  Step (2), moving the mass of a hypothesis A into a longer B that A is a prefix
 * of, is optional (prefix_search != 0): see beam_prefix_step.
 * Order conventions: entries of P' are ranked by log-probability, then offset, then label; new hypotheses are
 * appended in the order (hypothesis, rank); duplicates merge into their first occurrence; pruning is a stable sort.
 * Safeguard against staying on one frame (the paper omits its details): the rule of the greedy decoders above;
 * a hypothesis whose emission is the S-th in a row on its frame moves to the next frame without a blank factor.
 * With K = 1 this is window-based greedy decoding.
 *
 * min_gap: the smallest difference in log-probability that decided anything (K-th against (K+1)-th entry of a
 * hypothesis' P', K-th against (K+1)-th hypothesis at pruning, the two scores of a merged pair, best against second
 * final hypothesis).  A comparison against results computed in lower precision is only meaningful above it.
 */
typedef struct {
    int32_t* tok;
    int32_t* frm;
    int32_t len, count;
    double score;
    double *h, *c, *g;
} beam_hyp_t;

typedef struct { beam_hyp_t** v; int n, cap; } beam_list_t;
typedef struct { double lp; int32_t j, v; } beam_cand_t;

static void beam_push(beam_list_t* l, beam_hyp_t* h) {
    if (l->n == l->cap) { l->cap = l->cap ? 2 * l->cap : 8; l->v = (beam_hyp_t**)realloc(l->v, sizeof(beam_hyp_t*) * (size_t)l->cap); }
    l->v[l->n++] = h;
}
static void beam_free(beam_hyp_t* h) { free(h->tok); free(h->frm); free(h->h); free(h->c); free(h->g); free(h); }
static beam_hyp_t* beam_clone(const oracle_model_t* m, const beam_hyp_t* a, int extra) {
    beam_hyp_t* b = (beam_hyp_t*)malloc(sizeof(beam_hyp_t));
    *b = *a;
    b->tok = (int32_t*)malloc(sizeof(int32_t) * (size_t)(a->len + extra + 1));
    b->frm = (int32_t*)malloc(sizeof(int32_t) * (size_t)(a->len + extra + 1));
    memcpy(b->tok, a->tok, sizeof(int32_t) * (size_t)a->len);
    memcpy(b->frm, a->frm, sizeof(int32_t) * (size_t)a->len);
    const size_t ns = (size_t)m->L * m->P;
    b->h = (double*)malloc(sizeof(double) * ns); memcpy(b->h, a->h, sizeof(double) * ns);
    b->c = (double*)malloc(sizeof(double) * ns); memcpy(b->c, a->c, sizeof(double) * ns);
    b->g = (double*)malloc(sizeof(double) * (size_t)m->H); memcpy(b->g, a->g, sizeof(double) * (size_t)m->H);
    return b;
}
static int beam_cand_cmp(const void* pa, const void* pb) {
    const beam_cand_t* a = (const beam_cand_t*)pa; const beam_cand_t* b = (const beam_cand_t*)pb;
    if (a->lp != b->lp) return a->lp > b->lp ? -1 : 1;
    if (a->j != b->j) return a->j < b->j ? -1 : 1;
    return a->v < b->v ? -1 : (a->v > b->v ? 1 : 0);
}
static double log_add(double a, double b) {
    if (a == -INFINITY) return b;
    if (b == -INFINITY) return a;
    return a > b ? a + log1p(exp(b - a)) : b + log1p(exp(a - b));
}
static void note_gap(double* min_gap, double g) { if (g >= 0 && g < *min_gap) *min_gap = g; }

/* duplicates -> one (probabilities summed), then the K most probable, stable; freed hypotheses are released */
static void beam_prefix_step(const oracle_model_t* m, const double* encp_t, beam_list_t* l);

/* prefix_ctx_m == NULL: steps (1) and (3) only */
static void beam_recombine_prune(beam_list_t* l, int K, double* min_gap, const oracle_model_t* prefix_ctx_m,
                                 const double* encp_t) {
    for (int a = 0; a < l->n; ++a) {
        for (int b = a + 1; b < l->n;) {
            beam_hyp_t *x = l->v[a], *y = l->v[b];
            if (x->len == y->len && x->count == y->count && memcmp(x->tok, y->tok, sizeof(int32_t) * (size_t)x->len) == 0) {
                note_gap(min_gap, fabs(x->score - y->score));
                const double sum = log_add(x->score, y->score);
                if (y->score > x->score) { l->v[a] = y; beam_free(x); x = y; } else beam_free(y);
                x->score = sum;
                for (int k = b; k + 1 < l->n; ++k) l->v[k] = l->v[k + 1];
                l->n--;
            } else {
                ++b;
            }
        }
    }
    if (prefix_ctx_m) beam_prefix_step(prefix_ctx_m, encp_t, l);
    for (int a = 1; a < l->n; ++a) {   /* stable insertion sort, most probable first */
        beam_hyp_t* x = l->v[a];
        int k = a;
        while (k > 0 && l->v[k - 1]->score < x->score) { l->v[k] = l->v[k - 1]; --k; }
        l->v[k] = x;
    }
    if (l->n > K) {
        note_gap(min_gap, l->v[K - 1]->score - l->v[K]->score);
        for (int a = K; a < l->n; ++a) beam_free(l->v[a]);
        l->n = K;
    }
}

/*
 * Step (2) of recombine_prune as the paper states it: for all pairs (A, B) of the list where A's tokens are a proper
 * prefix of B's, the probability of completing A into B by emitting B's extra tokens at the current frame t,
 *     P(A) * prod_i P(b_i | frame t, decoder state after A + b_<i),
 * is added to B; then every such A is removed.  Every completion uses the probabilities the hypotheses had when the
 * step began, so the result does not depend on the order of the pairs.  (The details are in a cited paper that is
 * not at hand; this is the sentence of the paper, taken literally.)
 */
static void beam_prefix_step(const oracle_model_t* m, const double* encp_t, beam_list_t* l) {
    const int n = l->n, NV = m->V + 1;
    if (n < 2) return;
    double* add = (double*)malloc(sizeof(double) * (size_t)n);
    int* gone = (int*)calloc((size_t)n, sizeof(int));
    const size_t ns = (size_t)m->L * m->P;
    double* h = (double*)malloc(sizeof(double) * ns);
    double* c = (double*)malloc(sizeof(double) * ns);
    double* g = (double*)malloc(sizeof(double) * (size_t)m->H);
    double* z = (double*)malloc(sizeof(double) * (size_t)m->H);
    double* row = (double*)malloc(sizeof(double) * (size_t)NV);
    for (int b = 0; b < n; ++b) add[b] = -INFINITY;
    for (int a = 0; a < n; ++a)
        for (int b = 0; b < n; ++b) {
            const beam_hyp_t *A = l->v[a], *B = l->v[b];
            if (a == b || A->len >= B->len || memcmp(A->tok, B->tok, sizeof(int32_t) * (size_t)A->len) != 0) continue;
            memcpy(h, A->h, sizeof(double) * ns); memcpy(c, A->c, sizeof(double) * ns);
            memcpy(g, A->g, sizeof(double) * (size_t)m->H);
            double acc = A->score;
            for (int i = A->len; i < B->len; ++i) {
                oracle_joint_logits(m, encp_t, g, z, row);
                double mx = row[0];
                for (int v = 1; v < NV; ++v) if (row[v] > mx) mx = row[v];
                double se = 0.0;
                for (int v = 0; v < NV; ++v) se += exp(row[v] - mx);
                acc += row[B->tok[i]] - (mx + log(se));
                if (i + 1 < B->len) { oracle_lstm_step(m, B->tok[i], h, c); oracle_pred_proj(m, h, g); }
            }
            add[b] = log_add(add[b], acc);
            gone[a] = 1;
        }
    for (int b = 0; b < n; ++b) l->v[b]->score = log_add(l->v[b]->score, add[b]);
    int k = 0;
    for (int a = 0; a < n; ++a) {
        if (gone[a]) beam_free(l->v[a]); else l->v[k++] = l->v[a];
    }
    l->n = k;
    free(row); free(z); free(g); free(c); free(h); free(gone); free(add);
}

int32_t oracle_beam_search(const oracle_model_t* m, const float* enc, int32_t T, int32_t W, int32_t K, int32_t S,
                           int32_t prefix_search, int32_t max_hyps_out, int32_t max_out, int32_t* out_tokens,
                           int32_t* out_frames, int32_t* out_len, double* out_score, double* min_gap_out,
                           int64_t* n_steps_out) {
    if (W < 1 || W > 64 || K < 1 || S < 1 || T < 0) return -1;
    const int NV = m->V + 1;
    double* encp = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1) * m->H);
    oracle_enc_proj(m, enc, T, encp);
    double* logits = (double*)malloc(sizeof(double) * (size_t)W * NV);
    double* z = (double*)malloc(sizeof(double) * (size_t)m->H);
    beam_cand_t* cand = (beam_cand_t*)malloc(sizeof(beam_cand_t) * (size_t)W * NV);
    beam_list_t* t2hyps = (beam_list_t*)calloc((size_t)T + 1, sizeof(beam_list_t));
    double min_gap = INFINITY;
    int64_t steps = 0;
    {   /* t2hyps = {0: [Hyp(tokens = [], score = 0)]} */
        beam_hyp_t* h0 = (beam_hyp_t*)calloc(1, sizeof(beam_hyp_t));
        h0->tok = (int32_t*)malloc(sizeof(int32_t)); h0->frm = (int32_t*)malloc(sizeof(int32_t));
        h0->h = (double*)calloc((size_t)m->L * m->P, sizeof(double));
        h0->c = (double*)calloc((size_t)m->L * m->P, sizeof(double));
        h0->g = (double*)malloc(sizeof(double) * (size_t)m->H);
        oracle_lstm_step(m, m->blank_id, h0->h, h0->c);
        oracle_pred_proj(m, h0->h, h0->g);
        beam_push(&t2hyps[0], h0);
    }
    for (int t = 0; t < T; ++t) {
        beam_list_t* cur = &t2hyps[t];
        while (cur->n > 0) {   /* a frame is taken again when an expansion stays on it (jump 0) */
            beam_list_t hyps = *cur;
            cur->v = NULL; cur->n = 0; cur->cap = 0;
            beam_recombine_prune(&hyps, K, &min_gap, prefix_search ? m : NULL, encp + (size_t)t * m->H);
            const int n = (W < T - t) ? W : (T - t);
            steps++;
            for (int b = 0; b < hyps.n; ++b) {
                beam_hyp_t* hy = hyps.v[b];
                /* log P'(v, j) of Eq. (1) for this hypothesis' decoder state */
                double blanks_before = 0.0;
                int nc = 0;
                for (int j = 0; j < n; ++j) {
                    double* row = logits + (size_t)j * NV;
                    oracle_joint_logits(m, encp + (size_t)(t + j) * m->H, hy->g, z, row);
                    double mx = row[0];
                    for (int v = 1; v < NV; ++v) if (row[v] > mx) mx = row[v];
                    double se = 0.0;
                    for (int v = 0; v < NV; ++v) se += exp(row[v] - mx);
                    const double lse = mx + log(se);
                    for (int v = 0; v < NV; ++v) {
                        if (v == m->blank_id && j < n - 1) continue;
                        cand[nc].lp = row[v] - lse + blanks_before; cand[nc].j = j; cand[nc].v = v; nc++;
                    }
                    blanks_before += row[m->blank_id] - lse;
                }
                qsort(cand, (size_t)nc, sizeof(beam_cand_t), beam_cand_cmp);
                const int take = K < nc ? K : nc;
                if (take < nc) note_gap(&min_gap, cand[take - 1].lp - cand[take].lp);
                for (int k = 0; k < take; ++k) {
                    if (cand[k].v != m->blank_id) {
                        beam_hyp_t* nh = beam_clone(m, hy, 1);
                        int tt = t + cand[k].j;
                        nh->tok[nh->len] = cand[k].v; nh->frm[nh->len] = tt; nh->len++;
                        nh->score += cand[k].lp;
                        nh->count = cand[k].j == 0 ? hy->count + 1 : 1;
                        oracle_lstm_step(m, cand[k].v, nh->h, nh->c);
                        oracle_pred_proj(m, nh->h, nh->g);
                        if (nh->count == S) { tt += 1; nh->count = 0; }
                        beam_push(&t2hyps[tt], nh);
                    } else {
                        beam_hyp_t* nh = beam_clone(m, hy, 0);
                        nh->score += cand[k].lp;
                        nh->count = 0;
                        beam_push(&t2hyps[t + n], nh);
                    }
                }
            }
            for (int b = 0; b < hyps.n; ++b) beam_free(hyps.v[b]);
            free(hyps.v);
        }
        free(cur->v); cur->v = NULL;
    }
    /* best_hyp_in(t2hyps[T]): duplicates merged, most probable first */
    beam_list_t* fin = &t2hyps[T];
    beam_recombine_prune(fin, fin->n > 0 ? fin->n : 1, &min_gap, NULL, NULL);
    if (fin->n > 1) note_gap(&min_gap, fin->v[0]->score - fin->v[1]->score);
    int n_out = 0;
    for (int a = 0; a < fin->n; ++a) {
        if (a < max_hyps_out) {
            const beam_hyp_t* h = fin->v[a];
            out_len[a] = h->len; out_score[a] = h->score;
            for (int k = 0; k < h->len && k < max_out; ++k) {
                out_tokens[(size_t)a * max_out + k] = h->tok[k];
                out_frames[(size_t)a * max_out + k] = h->frm[k];
            }
            n_out++;
        }
        beam_free(fin->v[a]);
    }
    free(fin->v);
    free(t2hyps); free(cand); free(z); free(logits); free(encp);
    if (min_gap_out) *min_gap_out = min_gap;
    if (n_steps_out) *n_steps_out = steps;
    return n_out;
}

/*
 * Test access to step (2) alone: n hypotheses given by their tokens (row-major [n, max_len], lengths) and
 * log-probabilities at one encoder frame (enc_t [D]).  scores are updated in place, gone[i] = 1 for removed ones.
 */
void oracle_beam_prefix_step(const oracle_model_t* m, const float* enc_t, int32_t n, int32_t max_len, const int32_t* tokens,
                             const int32_t* lens, double* scores, int32_t* gone) {
    double* encp = (double*)malloc(sizeof(double) * (size_t)m->H);
    oracle_enc_proj(m, enc_t, 1, encp);
    beam_list_t l = {NULL, 0, 0};
    const size_t ns = (size_t)m->L * m->P;
    beam_hyp_t** all = (beam_hyp_t**)malloc(sizeof(beam_hyp_t*) * (size_t)(n > 0 ? n : 1));
    for (int i = 0; i < n; ++i) {
        beam_hyp_t* h = (beam_hyp_t*)calloc(1, sizeof(beam_hyp_t));
        h->len = lens[i];
        h->tok = (int32_t*)malloc(sizeof(int32_t) * (size_t)(lens[i] + 1));
        h->frm = (int32_t*)calloc((size_t)(lens[i] + 1), sizeof(int32_t));
        memcpy(h->tok, tokens + (size_t)i * max_len, sizeof(int32_t) * (size_t)lens[i]);
        h->h = (double*)calloc(ns, sizeof(double)); h->c = (double*)calloc(ns, sizeof(double));
        h->g = (double*)malloc(sizeof(double) * (size_t)m->H);
        oracle_lstm_step(m, m->blank_id, h->h, h->c);
        for (int k = 0; k < lens[i]; ++k) oracle_lstm_step(m, h->tok[k], h->h, h->c);
        oracle_pred_proj(m, h->h, h->g);
        h->score = scores[i];
        h->count = i;   /* tag: the position in the input, to find the survivors again */
        beam_push(&l, h);
        all[i] = h;
    }
    beam_prefix_step(m, encp, &l);
    for (int i = 0; i < n; ++i) gone[i] = 1;
    for (int k = 0; k < l.n; ++k) { gone[l.v[k]->count] = 0; scores[l.v[k]->count] = l.v[k]->score; beam_free(l.v[k]); }
    free(l.v); free(all); free(encp);
}
