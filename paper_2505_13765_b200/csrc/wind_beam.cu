// Algorithm 3 (WIND beam search) for one utterance.
//
// The hypothesis map, recombination and pruning are sequential bookkeeping over a handful of hypotheses and run on
// the host; everything that touches the model runs in kernels on the caller's stream: the encoder projection once,
// and per iteration (one frame t taken from the map) the decoder update of the hypotheses that survived pruning
// (batched over the beam), the windowed joint for every hypothesis, Eq. (1) and its K best entries per hypothesis.
// Only K x K (label, offset, log-probability) triples cross to the host per iteration.
//
// Decoder states live in a pool of slots in the workspace.  A hypothesis created by a label is evaluated lazily: it
// carries (parent slot, label) until it survives the pruning of its frame, so at most K decoder updates are made per
// iteration although K x K hypotheses are created.  Slots are reference-counted (a hypothesis created by the blank
// entry shares its parent's slot).
#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

#include "wind_internal.cuh"

namespace wind {

namespace {

// pool slot -> batch row (both parities of h are not needed: the update reads parity 0, writes parity 1)
__global__ void beam_gather_kernel(const float* __restrict__ h_pool, const float* __restrict__ c_pool, const int32_t* __restrict__ src,
                                   const int32_t* __restrict__ tok, float* __restrict__ h_in, float* __restrict__ c_state,
                                   int32_t* __restrict__ emit_tok, int B, int L, int P) {
    const int b = blockIdx.x;
    const int s = src[b];
    if (threadIdx.x == 0) emit_tok[b] = s >= 0 ? tok[b] : -1;
    if (s < 0) return;
    for (int e = threadIdx.x; e < L * P; e += blockDim.x) {
        const int l = e / P, k = e - l * P;
        h_in[((size_t)l * B + b) * P + k] = h_pool[(size_t)s * L * P + e];
        c_state[((size_t)l * B + b) * P + k] = c_pool[(size_t)s * L * P + e];
    }
}

// batch row -> pool slot: new state and its pred_proj
__global__ void beam_scatter_kernel(const float* __restrict__ h_out, const float* __restrict__ c_state, const float* __restrict__ pred_proj,
                                    const int32_t* __restrict__ dst, float* __restrict__ h_pool, float* __restrict__ c_pool,
                                    float* __restrict__ g_pool, int B, int L, int P, int H) {
    const int b = blockIdx.x;
    const int s = dst[b];
    if (s < 0) return;
    for (int e = threadIdx.x; e < L * P; e += blockDim.x) {
        const int l = e / P, k = e - l * P;
        h_pool[(size_t)s * L * P + e] = h_out[((size_t)l * B + b) * P + k];
        c_pool[(size_t)s * L * P + e] = c_state[((size_t)l * B + b) * P + k];
    }
    for (int k = threadIdx.x; k < H; k += blockDim.x) g_pool[(size_t)s * H + k] = pred_proj[(size_t)b * H + k];
}

// pred_proj of the hypotheses to expand, and their frame (rows without a hypothesis sit at the utterance's end)
__global__ void beam_gather_g_kernel(const float* __restrict__ g_pool, const int32_t* __restrict__ slot, float* __restrict__ pred_proj,
                                     int32_t* __restrict__ t_cur, int t, int T, int H) {
    const int b = blockIdx.x;
    const int s = slot[b];
    if (threadIdx.x == 0) t_cur[b] = s >= 0 ? t : T;
    if (s < 0) return;
    for (int k = threadIdx.x; k < H; k += blockDim.x) pred_proj[(size_t)b * H + k] = g_pool[(size_t)s * H + k];
}

// log-probability of one label per row, from a [B][NV] table of log-softmax values (rows without a label: untouched)
__global__ void beam_pick_kernel(const float* __restrict__ logp, const int32_t* __restrict__ label, float* __restrict__ out, int B, int NV) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B && label[b] >= 0) out[b] = logp[(size_t)b * NV + label[b]];
}

__global__ void beam_fill_kernel(int32_t* a, int n, int v) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) a[i] = v;
}

// Token histories are shared: a hypothesis points at the node of its last token, a node at the node before it.
struct Node {
    int32_t parent, tok, frm, len;
    uint64_t hash;          // of the token sequence up to here
};

struct Hyp {
    int32_t node = -1;      // -1: no tokens
    double score = 0.0;
    int count = 0;
    int slot = -1;          // decoder state after tok (-1: not evaluated yet)
    int parent = -1;        // slot of the state before the last token, while slot == -1
};

double log_add(double a, double b) {
    if (a == -INFINITY) return b;
    if (b == -INFINITY) return a;
    return a > b ? a + log1p(exp(b - a)) : b + log1p(exp(a - b));
}

}  // namespace

BeamLayout make_beam_layout(const wind_model_t& m, int T, int W, int K, int S, size_t base) {
    (void)T;
    BeamLayout L{};
    size_t off = base;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    const int s_eff = S < 32 ? S : 32;
    L.slots = K * (W + 2) * (s_eff + 2) + 2 * K + 2;
    L.h_pool = take(sizeof(float) * (size_t)L.slots * m.L * m.P);
    L.c_pool = take(sizeof(float) * (size_t)L.slots * m.L * m.P);
    L.g_pool = take(sizeof(float) * (size_t)L.slots * m.H);
    L.ints = take(sizeof(int32_t) * 8 * (size_t)K);
    L.logits = take(sizeof(float) * (size_t)K * W * (m.V + 1));
    L.top_label = take(sizeof(int32_t) * 3 * (size_t)K * K);   // labels, offsets, log-probabilities: one block, one copy
    L.top_jump = L.top_label + sizeof(int32_t) * (size_t)K * K;
    L.top_logp = L.top_jump + sizeof(int32_t) * (size_t)K * K;
    L.total = off;
    return L;
}

// cb: a call bundle with B = K rows (the beam), T, W, S of the utterance, enc = the utterance's frames [T, D];
// its enc_len / out_len pointers are set here.  Outputs are HOST arrays.
wind_status_t beam_search_run(Call& cb, const BeamLayout& bl, int K, int prefix_search, int max_hyps, int max_out, int32_t* out_tokens,
                              int32_t* out_frames, int32_t* out_len, double* out_score, int32_t* n_hyps, int64_t* n_steps,
                              cudaError_t* cuda_err) {
    const wind_model_t& m = cb.m;
    const int T = cb.T, W = cb.W, S = cb.S, NV = m.V + 1, LP = m.L * m.P;
    cudaStream_t st = cb.stream;
    uint8_t* ws = cb.ws;
    float* h_pool = reinterpret_cast<float*>(ws + bl.h_pool);
    float* c_pool = reinterpret_cast<float*>(ws + bl.c_pool);
    float* g_pool = reinterpret_cast<float*>(ws + bl.g_pool);
    int32_t* ints = reinterpret_cast<int32_t*>(ws + bl.ints);   // [0] src slots, [1] tokens, [2] dst slots, [3] expand slots, [4] lengths, [5] scratch, [6] frames
    int32_t *d_src = ints, *d_tok = ints + K, *d_dst = ints + 2 * K, *d_exp = ints + 3 * K, *d_len = ints + 4 * K,
            *d_scratch = ints + 5 * K, *d_t = ints + 6 * K;
    float* logits = reinterpret_cast<float*>(ws + bl.logits);
    int32_t* d_top_label = reinterpret_cast<int32_t*>(ws + bl.top_label);
    int32_t* d_top_jump = reinterpret_cast<int32_t*>(ws + bl.top_jump);
    float* d_top_logp = reinterpret_cast<float*>(ws + bl.top_logp);
#define BEAM_CUDA(expr) do { cudaError_t e__ = (expr); if (e__ != cudaSuccess) { *cuda_err = e__; return WIND_ERR_CUDA; } } while (0)

    // ---- setup: lengths, control block, encoder projection of the one utterance, an all-zero state in slot 0 ----
    beam_fill_kernel<<<1, 256, 0, st>>>(d_len, K, T);
    cb.enc_len = d_len;
    cb.out_len = d_scratch;
    BEAM_CUDA(launch_init(cb, WIND_KERNELS_SIMT, 0, 0));
    {
        Call c1 = cb;
        c1.B = 1;
        BEAM_CUDA(simt_enc_proj(c1));
    }
    BEAM_CUDA(cudaMemsetAsync(h_pool, 0, sizeof(float) * LP, st));
    BEAM_CUDA(cudaMemsetAsync(c_pool, 0, sizeof(float) * LP, st));

    std::vector<int> refs(bl.slots, 0), free_slots;
    for (int s = bl.slots - 1; s >= 1; --s) free_slots.push_back(s);
    refs[0] = 1;   // the zero state stays
    auto release = [&](int s) { if (s > 0 && --refs[s] == 0) free_slots.push_back(s); };

    std::vector<std::vector<Hyp>> t2hyps((size_t)T + 1);
    {
        Hyp h0;            // tokens = [], score = 0: its state is "zero state fed the blank id once"
        h0.parent = 0;
        refs[0]++;
        t2hyps[0].push_back(std::move(h0));
    }
    std::vector<int32_t> host_ints(4 * (size_t)K), top(3 * (size_t)K * K);
    const int32_t* top_label = top.data();
    const int32_t* top_jump = top.data() + (size_t)K * K;
    const float* top_logp = reinterpret_cast<const float*>(top.data() + 2 * (size_t)K * K);
    int64_t steps = 0;

    std::vector<Node> nodes;
    auto node_len = [&](int32_t n) { return n < 0 ? 0 : nodes[(size_t)n].len; };
    auto node_hash = [&](int32_t n) { return n < 0 ? 0x9E3779B97F4A7C15ull : nodes[(size_t)n].hash; };
    auto same_tokens = [&](int32_t x, int32_t y) {
        if (node_len(x) != node_len(y) || node_hash(x) != node_hash(y)) return false;
        while (x != y) {   // equal lengths: the chains end together, or meet at a shared node
            if (nodes[(size_t)x].tok != nodes[(size_t)y].tok) return false;
            x = nodes[(size_t)x].parent;
            y = nodes[(size_t)y].parent;
        }
        return true;
    };
    int32_t *d_pick = ints + 7 * K;
    // decoder update of up to K (parent slot, token) pairs into fresh slots; the parents' references are released
    auto run_update = [&](int nu) -> cudaError_t {   // host_ints [0..K) src, [K..2K) tokens, [2K..3K) dst are filled
        cudaError_t e = cudaMemcpyAsync(ints, host_ints.data(), sizeof(int32_t) * 3 * K, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return e;
        beam_gather_kernel<<<K, 128, 0, st>>>(h_pool, c_pool, d_src, d_tok, cb.h(0), cb.c(), cb.emit_tok(), K, m.L, m.P);
        if ((e = simt_pred_step(cb, 0)) != cudaSuccess) return e;
        beam_scatter_kernel<<<K, 128, 0, st>>>(cb.h(1), cb.c(), cb.pred_proj(), d_dst, h_pool, c_pool, g_pool, K, m.L, m.P, m.H);
        for (int u = 0; u < nu; ++u) release(host_ints[u]);
        return cudaGetLastError();
    };
    auto take_slot = [&]() -> int {
        if (free_slots.empty()) return -1;
        const int s = free_slots.back();
        free_slots.pop_back();
        refs[s] = 1;
        return s;
    };
    // Step (2) of the recombination as the paper states it: for every pair (A, B) of the list with A's tokens a proper
    // prefix of B's, P(A) * prod_i P(b_i | frame t, decoder after A + b_<i) is added to B, then every such A is removed.
    // The per-label probabilities come from the same kernels as the expansion (one-row window at frame t), K pairs at a
    // time, one round per extra token; completions use the probabilities the hypotheses had when the step began.
    struct Pair { int a, b, cur; std::vector<int32_t> extra; double acc; };
    auto prefix_step = [&](std::vector<Hyp>& l, int t) -> wind_status_t {
        const int n = (int)l.size();
        if (n < 2) return WIND_OK;
        std::vector<Pair> pairs;
        for (int a = 0; a < n; ++a)
            for (int b = 0; b < n; ++b) {
                const int la = node_len(l[a].node), lb = node_len(l[b].node);
                if (a == b || la >= lb) continue;
                std::vector<int32_t> extra((size_t)(lb - la));
                int32_t x = l[b].node;
                for (int k = lb - la - 1; k >= 0; --k) { extra[(size_t)k] = nodes[(size_t)x].tok; x = nodes[(size_t)x].parent; }
                if (!same_tokens(l[a].node, x)) continue;
                pairs.push_back(Pair{a, b, -1, std::move(extra), l[a].score});
            }
        if (pairs.empty()) return WIND_OK;
        // the prefixes need their decoder state now
        std::vector<char> is_prefix((size_t)n, 0);
        for (const Pair& p : pairs) is_prefix[(size_t)p.a] = 1;
        for (int a0 = 0; a0 < n;) {
            int nu = 0;
            for (int b = 0; b < K; ++b) { host_ints[b] = -1; host_ints[K + b] = -1; host_ints[2 * K + b] = -1; }
            for (; a0 < n && nu < K; ++a0) {
                Hyp& h = l[(size_t)a0];
                if (!is_prefix[(size_t)a0] || h.slot >= 0) continue;
                const int s = take_slot();
                if (s < 0) return WIND_ERR_WORKSPACE;
                host_ints[nu] = h.parent;
                host_ints[K + nu] = h.node < 0 ? m.blank_id : nodes[(size_t)h.node].tok;
                host_ints[2 * K + nu] = s;
                h.slot = s;
                ++nu;
            }
            if (nu > 0) BEAM_CUDA(run_update(nu));
        }
        for (Pair& p : pairs) { p.cur = l[(size_t)p.a].slot; refs[p.cur]++; }
        std::vector<float> picked((size_t)K);
        size_t depth = 0;
        for (bool more = true; more; ++depth) {
            more = false;
            std::vector<size_t> act;
            for (size_t i = 0; i < pairs.size(); ++i)
                if (pairs[i].extra.size() > depth) act.push_back(i);
            for (size_t c0 = 0; c0 < act.size(); c0 += (size_t)K) {
                const int nr = (int)std::min((size_t)K, act.size() - c0);
                // log-softmax at frame t under each pair's current state, and the extra token's entry
                for (int b = 0; b < K; ++b) { host_ints[3 * K + b] = -1; host_ints[b] = -1; host_ints[K + b] = -1; host_ints[2 * K + b] = -1; }
                std::vector<int32_t> labels((size_t)K, -1);
                for (int r = 0; r < nr; ++r) {
                    Pair& p = pairs[act[c0 + (size_t)r]];
                    host_ints[3 * K + r] = p.cur;
                    labels[(size_t)r] = p.extra[depth];
                }
                BEAM_CUDA(cudaMemcpyAsync(d_exp, host_ints.data() + 3 * K, sizeof(int32_t) * K, cudaMemcpyHostToDevice, st));
                BEAM_CUDA(cudaMemcpyAsync(d_pick, labels.data(), sizeof(int32_t) * K, cudaMemcpyHostToDevice, st));
                beam_gather_g_kernel<<<K, 128, 0, st>>>(g_pool, d_exp, cb.pred_proj(), d_t, t, T, m.H);
                BEAM_CUDA(launch_set_t(cb, d_t));
                Call one = cb;
                one.W = 1;
                BEAM_CUDA(simt_joint_shared(one, logits));
                BEAM_CUDA(launch_first_output(logits, d_len, d_t, K, 1, NV, m.blank_id, 0, nullptr, nullptr, nullptr, st));
                beam_pick_kernel<<<1, 32, 0, st>>>(logits, d_pick, d_top_logp, K, NV);
                BEAM_CUDA(cudaMemcpyAsync(picked.data(), d_top_logp, sizeof(float) * K, cudaMemcpyDeviceToHost, st));
                BEAM_CUDA(cudaStreamSynchronize(st));
                // one more decoder update for the pairs that have a further token
                int nu = 0;
                for (int r = 0; r < nr; ++r) {
                    Pair& p = pairs[act[c0 + (size_t)r]];
                    p.acc += (double)picked[(size_t)r];
                    if (p.extra.size() > depth + 1) {
                        const int s = take_slot();
                        if (s < 0) return WIND_ERR_WORKSPACE;
                        host_ints[nu] = p.cur;               // released by run_update
                        host_ints[K + nu] = p.extra[depth];
                        host_ints[2 * K + nu] = s;
                        p.cur = s;
                        ++nu;
                        more = true;
                    } else {
                        release(p.cur);
                        p.cur = -1;
                    }
                }
                if (nu > 0) BEAM_CUDA(run_update(nu));
            }
        }
        std::vector<double> add((size_t)n, -INFINITY);
        for (const Pair& p : pairs) add[(size_t)p.b] = log_add(add[(size_t)p.b], p.acc);
        std::vector<Hyp> kept;
        for (int a = 0; a < n; ++a) {
            if (is_prefix[(size_t)a]) {
                release(l[(size_t)a].slot >= 0 ? l[(size_t)a].slot : l[(size_t)a].parent);
            } else {
                l[(size_t)a].score = log_add(l[(size_t)a].score, add[(size_t)a]);
                kept.push_back(l[(size_t)a]);
            }
        }
        l.swap(kept);
        return WIND_OK;
    };
    auto merge_duplicates = [&](std::vector<Hyp>& l) {
        for (size_t a = 0; a < l.size(); ++a)
            for (size_t b = a + 1; b < l.size();) {
                if (l[a].count == l[b].count && same_tokens(l[a].node, l[b].node)) {
                    const double sum = log_add(l[a].score, l[b].score);
                    if (l[b].score > l[a].score) std::swap(l[a], l[b]);
                    l[a].score = sum;
                    release(l[b].slot >= 0 ? l[b].slot : l[b].parent);
                    l.erase(l.begin() + (long)b);
                } else {
                    ++b;
                }
            }
    };
    auto prune = [&](std::vector<Hyp>& l, size_t keep) {
        std::stable_sort(l.begin(), l.end(), [](const Hyp& x, const Hyp& y) { return x.score > y.score; });
        while (l.size() > keep) {
            release(l.back().slot >= 0 ? l.back().slot : l.back().parent);
            l.pop_back();
        }
    };

    for (int t = 0; t < T; ++t) {
        while (!t2hyps[t].empty()) {
            std::vector<Hyp> hyps;
            hyps.swap(t2hyps[t]);
            merge_duplicates(hyps);
            if (prefix_search) {
                const wind_status_t ps = prefix_step(hyps, t);
                if (ps != WIND_OK) return ps;
            }
            prune(hyps, (size_t)K);
            const int nh = (int)hyps.size();
            const int n = W < T - t ? W : T - t;
            ++steps;
            // ---- decoder update of the survivors that have no state yet ----
            int nu = 0;
            for (int b = 0; b < K; ++b) { host_ints[b] = -1; host_ints[K + b] = -1; host_ints[2 * K + b] = -1; host_ints[3 * K + b] = -1; }
            for (int b = 0; b < nh; ++b) {
                Hyp& h = hyps[b];
                if (h.slot < 0) {
                    if (free_slots.empty()) return WIND_ERR_WORKSPACE;
                    const int s = free_slots.back();
                    free_slots.pop_back();
                    refs[s] = 1;
                    host_ints[nu] = h.parent;
                    host_ints[K + nu] = h.node < 0 ? m.blank_id : nodes[(size_t)h.node].tok;
                    host_ints[2 * K + nu] = s;
                    h.slot = s;
                    ++nu;
                }
            }
            for (int b = 0; b < nh; ++b) host_ints[3 * K + b] = hyps[b].slot;
            BEAM_CUDA(cudaMemcpyAsync(d_exp, host_ints.data() + 3 * K, sizeof(int32_t) * K, cudaMemcpyHostToDevice, st));
            beam_gather_g_kernel<<<K, 128, 0, st>>>(g_pool, d_exp, cb.pred_proj(), d_t, t, T, m.H);   // sets the frames first
            BEAM_CUDA(launch_set_t(cb, d_t));   // frames of the rows, and the control block's "active" word
            if (nu > 0) {
                BEAM_CUDA(run_update(nu));   // (the parents are no longer needed by these hypotheses)
                beam_gather_g_kernel<<<K, 128, 0, st>>>(g_pool, d_exp, cb.pred_proj(), d_t, t, T, m.H);
            }
            // ---- window logits of every hypothesis, Eq. (1), the K best entries each ----
            BEAM_CUDA(simt_joint_shared(cb, logits));
            BEAM_CUDA(launch_first_output(logits, d_len, d_t, K, W, NV, m.blank_id, K, d_top_label, d_top_jump, d_top_logp, st));
            BEAM_CUDA(cudaMemcpyAsync(top.data(), d_top_label, sizeof(int32_t) * 3 * K * K, cudaMemcpyDeviceToHost, st));
            BEAM_CUDA(cudaStreamSynchronize(st));
            // ---- expansions ----
            for (int b = 0; b < nh; ++b) {
                const Hyp& h = hyps[b];
                for (int k = 0; k < K; ++k) {
                    const int label = top_label[(size_t)b * K + k], jump = top_jump[(size_t)b * K + k];
                    const float lp = top_logp[(size_t)b * K + k];
                    if (label < 0 || !(lp > -INFINITY)) continue;    // fewer than K entries in a small window
                    Hyp nhyp;
                    nhyp.score = h.score + (double)lp;
                    if (label != m.blank_id) {
                        int tt = t + jump;
                        Node nd;
                        nd.parent = h.node; nd.tok = label; nd.frm = tt; nd.len = node_len(h.node) + 1;
                        nd.hash = (node_hash(h.node) ^ (uint64_t)(uint32_t)label) * 0x100000001B3ull + 0x9E3779B97F4A7C15ull;
                        nodes.push_back(nd);
                        nhyp.node = (int32_t)nodes.size() - 1;
                        nhyp.count = jump == 0 ? h.count + 1 : 1;
                        nhyp.parent = h.slot;
                        refs[h.slot]++;
                        if (nhyp.count == S) { tt += 1; nhyp.count = 0; }
                        t2hyps[tt].push_back(std::move(nhyp));
                    } else {
                        nhyp.node = h.node;
                        nhyp.count = 0;
                        nhyp.slot = h.slot;
                        refs[h.slot]++;
                        t2hyps[t + n].push_back(std::move(nhyp));
                    }
                }
            }
            for (int b = 0; b < nh; ++b) release(hyps[b].slot);
        }
    }
    std::vector<Hyp>& fin = t2hyps[T];
    merge_duplicates(fin);
    prune(fin, fin.size() > 0 ? fin.size() : 1);
    int n_out = 0;
    for (size_t a = 0; a < fin.size() && (int)a < max_hyps; ++a) {
        const Hyp& h = fin[a];
        const int len = node_len(h.node);
        out_len[a] = len;
        out_score[a] = h.score;
        int32_t nd = h.node;
        for (int k = len - 1; k >= 0; --k) {   // walk the history back from the last token
            if (k < max_out) {
                out_tokens[a * (size_t)max_out + k] = nodes[(size_t)nd].tok;
                out_frames[a * (size_t)max_out + k] = nodes[(size_t)nd].frm;
            }
            nd = nodes[(size_t)nd].parent;
        }
        ++n_out;
    }
    *n_hyps = n_out;
    if (n_steps) *n_steps = steps;
#undef BEAM_CUDA
    return WIND_OK;
}

}  // namespace wind
