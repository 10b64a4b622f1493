// C ABI entry points: argument checks, workspace carving, launch sequence, and the
// device-resident decoding loop (a CUDA-graph WHILE node whose body is two lock steps).
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "wind_internal.cuh"
#include "wind_loop.cuh"

namespace wind {

static thread_local char g_cuda_err[256] = "";
static int g_kernels = WIND_KERNELS_AUTO;
static int g_trace_step = -2;   // first lock step of the loop kernel's timeline window; -2 = off

static wind_status_t cuda_fail(cudaError_t e, const char* where) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", where, cudaGetErrorString(e));
    return WIND_ERR_CUDA;
}
#define WIND_CUDA(expr)                                              \
    do {                                                             \
        cudaError_t e__ = (expr);                                    \
        if (e__ != cudaSuccess) return cuda_fail(e__, #expr);        \
    } while (0)

static wind_status_t check_model(const wind_model_t* m) {
    if (!m) return WIND_ERR_INVALID_ARG;
    if (m->D < 1 || m->E < 1 || m->P < 1 || m->L < 1 || m->H < 1 || m->V < 1) return WIND_ERR_INVALID_ARG;
    if (m->blank_id < 0 || m->blank_id > m->V) return WIND_ERR_INVALID_ARG;
    if (m->act != WIND_ACT_RELU && m->act != WIND_ACT_TANH) return WIND_ERR_INVALID_ARG;
    if (m->dtype != WIND_DT_F32 && m->dtype != WIND_DT_BF16) return WIND_ERR_INVALID_ARG;
    if (m->L > kMaxLayers) return WIND_ERR_UNSUPPORTED;
    return WIND_OK;
}

static wind_status_t check_shape(const wind_model_t* m, int B, int T, int W) {
    if (B < 1 || T < 1 || W < 1) return WIND_ERR_INVALID_ARG;
    if (W > kMaxWindow) return WIND_ERR_UNSUPPORTED;
    if ((long long)B * T * m->H > 0x7fffffffLL || (long long)B * T * m->D > 0x7fffffffLL) return WIND_ERR_UNSUPPORTED;
    if ((long long)B * W > 0x7fffffffLL) return WIND_ERR_UNSUPPORTED;
    return WIND_OK;
}

static wind_status_t check_weights(const wind_model_t* m) {
    if (!m->emb || !m->w_ih || !m->w_hh || !m->b_ih || !m->b_hh || !m->w_enc || !m->b_enc || !m->w_pred || !m->b_pred ||
        !m->w_out || !m->b_out)
        return WIND_ERR_INVALID_ARG;
    for (int l = 0; l < m->L; ++l)
        if (!m->w_ih[l] || !m->w_hh[l] || !m->b_ih[l] || !m->b_hh[l]) return WIND_ERR_INVALID_ARG;
    return WIND_OK;
}

static void fill_call(Call& c, const wind_model_t* m, const void* enc, const int32_t* enc_len, int B, int T, int W, int S,
                      int32_t* out_tokens, int32_t* out_frames, int32_t* out_len, int max_out, void* ws, cudaStream_t stream) {
    memset(&c, 0, sizeof(c));
    c.m = *m;
    for (int l = 0; l < m->L; ++l) {
        c.w_ih[l] = m->w_ih[l];
        c.w_hh[l] = m->w_hh[l];
        c.b_ih[l] = m->b_ih[l];
        c.b_hh[l] = m->b_hh[l];
    }
    c.m.w_ih = nullptr; c.m.w_hh = nullptr; c.m.b_ih = nullptr; c.m.b_hh = nullptr;  // host arrays: not part of the key
    c.m.reserved = 0;
    c.enc = enc; c.enc_len = enc_len;
    c.B = B; c.T = T; c.W = W; c.S = S; c.max_out = max_out;
    c.out_tokens = out_tokens; c.out_frames = out_frames; c.out_len = out_len;
    c.ws = static_cast<uint8_t*>(ws);
    c.lay = make_layout(*m, B, T, W, max_out);
    c.stream = stream;
}

static bool use_tensor(const Call& c) {
    if (c.m.dtype != WIND_DT_BF16) return false;
    if (g_kernels == WIND_KERNELS_SIMT) return false;
    return tc_supported(c.m, c.B, c.T, c.W);
}

// ---------------------------------------------------------------------------
// Decoding loop as a CUDA graph: WHILE(active > 0) { step(parity 1->0); step(parity 0->1) }.
// A lock step is joint -> control -> decoder update; kernels of a step that starts with
// active == 0 return at once, so the second step of the last iteration is a no-op.
// Kernel arguments are baked into the graph, hence the cache keyed by the whole call.
// ---------------------------------------------------------------------------
struct LoopGraph {
    Call key;
    int tensor;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    unsigned long long last_use = 0;
};
static std::mutex g_mutex;
static std::vector<LoopGraph> g_graphs;
static unsigned long long g_use_counter = 0;
static cudaStream_t g_capture_stream = nullptr;
constexpr size_t kMaxGraphs = 12;

static cudaError_t enqueue_step(const Call& c, bool tensor, int parity_in, cudaGraphConditionalHandle handle, int use_handle) {
    (void)tensor;
    cudaError_t e = simt_joint(c, nullptr);
    if (e != cudaSuccess) return e;
    e = launch_control(c, handle, use_handle);
    if (e != cudaSuccess) return e;
    return simt_pred_step(c, parity_in);
}

static bool same_key(const Call& a, const Call& b) {
    Call x = a, y = b;
    x.stream = nullptr; y.stream = nullptr;
    x.tc = nullptr; y.tc = nullptr;
    return memcmp(&x, &y, sizeof(Call)) == 0;
}

static wind_status_t get_loop_graph(const Call& c, bool tensor, cudaGraphExec_t* exec_out) {
    std::lock_guard<std::mutex> lock(g_mutex);
    for (auto& g : g_graphs)
        if (g.tensor == (int)tensor && same_key(g.key, c)) {
            g.last_use = ++g_use_counter;
            *exec_out = g.exec;
            return WIND_OK;
        }
    if (!g_capture_stream) WIND_CUDA(cudaStreamCreateWithFlags(&g_capture_stream, cudaStreamNonBlocking));
    LoopGraph g;
    g.key = c;
    g.tensor = tensor;
    WIND_CUDA(cudaGraphCreate(&g.graph, 0));
    cudaGraphConditionalHandle handle;
    WIND_CUDA(cudaGraphConditionalHandleCreate(&handle, g.graph, 1, cudaGraphCondAssignDefault));
    cudaGraphNodeParams np = {cudaGraphNodeTypeConditional};
    np.conditional.handle = handle;
    np.conditional.type = cudaGraphCondTypeWhile;
    np.conditional.size = 1;
    cudaGraphNode_t node;
    WIND_CUDA(cudaGraphAddNode(&node, g.graph, nullptr, 0, &np));
    cudaGraph_t body = np.conditional.phGraph_out[0];
    Call cc = c;
    cc.stream = g_capture_stream;
    WIND_CUDA(cudaStreamBeginCaptureToGraph(g_capture_stream, body, nullptr, nullptr, 0, cudaStreamCaptureModeRelaxed));
    cudaError_t e1 = enqueue_step(cc, tensor, 1, handle, 1);
    cudaError_t e2 = e1 == cudaSuccess ? enqueue_step(cc, tensor, 0, handle, 1) : e1;
    cudaGraph_t ended = nullptr;
    cudaError_t e3 = cudaStreamEndCapture(g_capture_stream, &ended);
    if (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess) {
        cudaGraphDestroy(g.graph);
        return cuda_fail(e1 != cudaSuccess ? e1 : (e2 != cudaSuccess ? e2 : e3), "capture of the decoding loop");
    }
    cudaError_t e4 = cudaGraphInstantiate(&g.exec, g.graph, 0);
    if (e4 != cudaSuccess) {
        cudaGraphDestroy(g.graph);
        return cuda_fail(e4, "cudaGraphInstantiate");
    }
    if (g_graphs.size() >= kMaxGraphs) {
        size_t victim = 0;
        for (size_t i = 1; i < g_graphs.size(); ++i)
            if (g_graphs[i].last_use < g_graphs[victim].last_use) victim = i;
        cudaGraphExecDestroy(g_graphs[victim].exec);
        cudaGraphDestroy(g_graphs[victim].graph);
        g_graphs.erase(g_graphs.begin() + victim);
    }
    g.last_use = ++g_use_counter;
    g_graphs.push_back(g);
    *exec_out = g.exec;
    return WIND_OK;
}

// Enqueue the whole decode on c.stream (no synchronisation).
static wind_status_t enqueue_decode(Call& c) {
    const bool tensor = use_tensor(c);
    if (c.m.dtype == WIND_DT_BF16 && g_kernels == WIND_KERNELS_TENSOR && !tensor) return WIND_ERR_UNSUPPORTED;
    if (tensor) {
        // projection and gate table once, then the whole loop as one persistent kernel
        WIND_CUDA(tc_prepare(c));
        WIND_CUDA(launch_init(c, WIND_KERNELS_TENSOR, 0, tc_setup_launches(c)));
        WIND_CUDA(tc_enc_proj(c));
        WIND_CUDA(tc_gate_table(c));
        WIND_CUDA(tc_loop(c, nullptr, 0, nullptr, nullptr, g_trace_step));
        return WIND_OK;
    }
    const int per_step = 2 + simt_pred_launches(c);
    const int setup = 2 + simt_pred_launches(c);
    WIND_CUDA(launch_init(c, WIND_KERNELS_SIMT, per_step, setup));
    WIND_CUDA(simt_enc_proj(c));
    WIND_CUDA(simt_pred_step(c, 0));  // start of sequence: h[0] (zeros) -> h[1]
    cudaGraphExec_t exec = nullptr;
    wind_status_t s = get_loop_graph(c, false, &exec);
    if (s != WIND_OK) return s;
    WIND_CUDA(cudaGraphLaunch(exec, c.stream));
    return WIND_OK;
}

static wind_status_t read_status(const Call& c) {
    int32_t st = 0;
    WIND_CUDA(cudaMemcpyAsync(&st, &c.ctrl()->status, sizeof(int32_t), cudaMemcpyDeviceToHost, c.stream));
    WIND_CUDA(cudaStreamSynchronize(c.stream));
    return (wind_status_t)st;
}

static wind_status_t check_decode_args(const wind_model_t* m, const void* enc, const int32_t* enc_len, int B, int T, int W,
                                       int S, const int32_t* ot, const int32_t* of, const int32_t* ol, int max_out,
                                       const void* ws) {
    wind_status_t s = check_model(m);
    if (s != WIND_OK) return s;
    s = check_weights(m);
    if (s != WIND_OK) return s;
    s = check_shape(m, B, T, W);
    if (s != WIND_OK) return s;
    if (!enc || !enc_len || !ot || !of || !ol || !ws) return WIND_ERR_INVALID_ARG;
    if (S < 1 || max_out < 1) return WIND_ERR_INVALID_ARG;
    if ((long long)B * max_out > 0x7fffffffLL) return WIND_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(ws) % kAlign) return WIND_ERR_WORKSPACE;
    return WIND_OK;
}

}  // namespace wind

using namespace wind;

extern "C" {

wind_status_t wind_workspace_bytes(const wind_model_t* m, int32_t B, int32_t T, int32_t W, size_t* bytes) {
    wind_status_t s = check_model(m);
    if (s != WIND_OK) return s;
    s = check_shape(m, B, T, W);
    if (s != WIND_OK) return s;
    if (!bytes) return WIND_ERR_INVALID_ARG;
    *bytes = make_layout(*m, B, T, W, 1).total;
    return WIND_OK;
}

wind_status_t wind_host_staging_bytes(const wind_model_t* m, int32_t B, int32_t T, int32_t max_out, size_t* bytes) {
    wind_status_t s = check_model(m);
    if (s != WIND_OK) return s;
    s = check_shape(m, B, T, 1);
    if (s != WIND_OK) return s;
    if (!bytes || max_out < 1) return WIND_ERR_INVALID_ARG;
    *bytes = make_layout(*m, B, T, 1, max_out).st_total;
    return WIND_OK;
}

wind_status_t wind_decode_greedy(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B, int32_t T,
                                 int32_t W, int32_t max_symbols, int32_t* out_tokens, int32_t* out_frames, int32_t* out_len,
                                 int32_t max_out, void* workspace, size_t workspace_bytes, void* stream) {
    wind_status_t s = check_decode_args(m, enc, enc_len, B, T, W, max_symbols, out_tokens, out_frames, out_len, max_out, workspace);
    if (s != WIND_OK) return s;
    Call c;
    fill_call(c, m, enc, enc_len, B, T, W, max_symbols, out_tokens, out_frames, out_len, max_out, workspace, (cudaStream_t)stream);
    if (workspace_bytes < c.lay.total) return WIND_ERR_WORKSPACE;
    s = enqueue_decode(c);
    if (s != WIND_OK) return s;
    return read_status(c);
}

wind_status_t wind_decode_window_greedy(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B, int32_t T,
                                        int32_t W, int32_t max_symbols, int32_t* out_tokens, int32_t* out_frames,
                                        int32_t* out_len, int32_t max_out, void* workspace, size_t workspace_bytes,
                                        void* stream) {
    wind_status_t s = check_decode_args(m, enc, enc_len, B, T, W, max_symbols, out_tokens, out_frames, out_len, max_out, workspace);
    if (s != WIND_OK) return s;
    Call c;
    fill_call(c, m, enc, enc_len, B, T, W, max_symbols, out_tokens, out_frames, out_len, max_out, workspace, (cudaStream_t)stream);
    c.mode = WIND_MODE_WINDOW;
    if (workspace_bytes < c.lay.total) return WIND_ERR_WORKSPACE;
    s = enqueue_decode(c);
    if (s != WIND_OK) return s;
    return read_status(c);
}

wind_status_t wind_refill_workspace_bytes(const wind_model_t* m, int32_t N, int32_t T, int32_t B, int32_t W, size_t* bytes) {
    wind_status_t s = check_model(m);
    if (s != WIND_OK) return s;
    if (N < 1) return WIND_ERR_INVALID_ARG;
    s = check_shape(m, N > B ? N : B, T, W);
    if (s != WIND_OK) return s;
    if (!bytes) return WIND_ERR_INVALID_ARG;
    *bytes = make_layout(*m, B, T, W, 1, N).total;
    return WIND_OK;
}

wind_status_t wind_decode_greedy_refill(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t N, int32_t T,
                                        int32_t B, int32_t W, int32_t max_symbols, int32_t* out_tokens, int32_t* out_frames,
                                        int32_t* out_len, int32_t max_out, void* workspace, size_t workspace_bytes,
                                        void* stream) {
    if (N < 1) return WIND_ERR_INVALID_ARG;
    wind_status_t s = check_decode_args(m, enc, enc_len, B, T, W, max_symbols, out_tokens, out_frames, out_len, max_out, workspace);
    if (s != WIND_OK) return s;
    s = check_shape(m, N > B ? N : B, T, W);
    if (s != WIND_OK) return s;
    if ((long long)N * max_out > 0x7fffffffLL) return WIND_ERR_UNSUPPORTED;
    Call c;
    fill_call(c, m, enc, enc_len, B, T, W, max_symbols, out_tokens, out_frames, out_len, max_out, workspace, (cudaStream_t)stream);
    c.N = N;
    c.lay = make_layout(*m, B, T, W, max_out, N);
    if (workspace_bytes < c.lay.total) return WIND_ERR_WORKSPACE;
    // rows are refilled inside the persistent loop kernel of the tensor-core set only
    if (!use_tensor(c)) return WIND_ERR_UNSUPPORTED;
    WIND_CUDA(tc_prepare(c));
    WIND_CUDA(launch_init(c, WIND_KERNELS_TENSOR, 0, tc_setup_launches(c)));
    WIND_CUDA(tc_enc_proj(c));
    WIND_CUDA(tc_gate_table(c));
    WIND_CUDA(tc_loop(c, nullptr, 0, nullptr, nullptr, g_trace_step));
    return read_status(c);
}

wind_status_t wind_decode_greedy_host(const wind_model_t* m, const void* enc_host, const int32_t* enc_len_host, int32_t B,
                                      int32_t T, int32_t W, int32_t max_symbols, int32_t* out_tokens_host,
                                      int32_t* out_frames_host, int32_t* out_len_host, int32_t max_out, void* workspace,
                                      size_t workspace_bytes, void* stream) {
    wind_status_t s = check_decode_args(m, enc_host, enc_len_host, B, T, W, max_symbols, out_tokens_host, out_frames_host,
                                        out_len_host, max_out, workspace);
    if (s != WIND_OK) return s;
    Layout lay = make_layout(*m, B, T, W, max_out);
    if (workspace_bytes < lay.total + lay.st_total) return WIND_ERR_WORKSPACE;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    cudaStream_t st = (cudaStream_t)stream;
    const size_t es = m->dtype == WIND_DT_BF16 ? 2 : 4;
    void* d_enc = ws + lay.st_enc;
    int32_t* d_len = reinterpret_cast<int32_t*>(ws + lay.st_len);
    int32_t* d_tok = reinterpret_cast<int32_t*>(ws + lay.st_tok);
    int32_t* d_frm = reinterpret_cast<int32_t*>(ws + lay.st_frm);
    int32_t* d_olen = reinterpret_cast<int32_t*>(ws + lay.st_olen);
    for (int b = 0; b < B; ++b)
        if (enc_len_host[b] < 0 || enc_len_host[b] > T) return WIND_ERR_INVALID_ARG;   // before anything is enqueued
    // only the valid frames of every utterance cross the bus (padding frames are never read for a decision)
    for (int b = 0; b < B; ++b) {
        const int len = enc_len_host[b];
        if (len > 0)
            WIND_CUDA(cudaMemcpyAsync(static_cast<uint8_t*>(d_enc) + es * (size_t)b * T * m->D,
                                      static_cast<const uint8_t*>(enc_host) + es * (size_t)b * T * m->D, es * (size_t)len * m->D,
                                      cudaMemcpyHostToDevice, st));
    }
    WIND_CUDA(cudaMemcpyAsync(d_len, enc_len_host, sizeof(int32_t) * B, cudaMemcpyHostToDevice, st));
    Call c;
    fill_call(c, m, d_enc, d_len, B, T, W, max_symbols, d_tok, d_frm, d_olen, max_out, workspace, st);
    s = enqueue_decode(c);
    if (s != WIND_OK) return s;
    // lengths first, then the columns of the two output arrays that hold tokens (up to the longest transcript)
    WIND_CUDA(cudaMemcpyAsync(out_len_host, d_olen, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, st));
    const wind_status_t status = read_status(c);   // synchronises the stream
    if (status != WIND_OK && status != WIND_ERR_OUTPUT_OVERFLOW) return status;
    int longest = 0;
    for (int b = 0; b < B; ++b) longest = out_len_host[b] > longest ? out_len_host[b] : longest;
    if (longest > max_out) longest = max_out;
    if (longest > 0) {
        const size_t pitch = sizeof(int32_t) * (size_t)max_out, width = sizeof(int32_t) * (size_t)longest;
        WIND_CUDA(cudaMemcpy2DAsync(out_tokens_host, pitch, d_tok, pitch, width, (size_t)B, cudaMemcpyDeviceToHost, st));
        WIND_CUDA(cudaMemcpy2DAsync(out_frames_host, pitch, d_frm, pitch, width, (size_t)B, cudaMemcpyDeviceToHost, st));
        WIND_CUDA(cudaStreamSynchronize(st));
    }
    return status;
}

// Teacher-forced window logits, enqueued on the stream (no synchronisation); c receives the call's bundle.
static wind_status_t enqueue_eval_joint_window(Call& c, const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B,
                                               int32_t T, int32_t W, const int32_t* prefix, int32_t U, const int32_t* prefix_len,
                                               const int32_t* t0, float* logits, void* workspace, size_t workspace_bytes,
                                               void* stream) {
    wind_status_t s = check_model(m);
    if (s != WIND_OK) return s;
    s = check_weights(m);
    if (s != WIND_OK) return s;
    s = check_shape(m, B, T, W);
    if (s != WIND_OK) return s;
    if (!enc || !enc_len || !prefix_len || !t0 || !logits || !workspace || U < 0 || (U > 0 && !prefix)) return WIND_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return WIND_ERR_WORKSPACE;
    // the control arrays double as scratch outputs here: out_len is reset by the init kernel
    fill_call(c, m, enc, enc_len, B, T, W, 1, nullptr, nullptr, nullptr, 1, workspace, (cudaStream_t)stream);
    if (workspace_bytes < c.lay.total) return WIND_ERR_WORKSPACE;
    c.out_len = c.count();  // any int32 [B] scratch: init writes zeros to it
    const bool tensor = use_tensor(c);
    if (c.m.dtype == WIND_DT_BF16 && g_kernels == WIND_KERNELS_TENSOR && !tensor) return WIND_ERR_UNSUPPORTED;
    if (tensor) {
        WIND_CUDA(tc_prepare(c));
        WIND_CUDA(launch_init(c, WIND_KERNELS_TENSOR, 0, 0));
        WIND_CUDA(tc_enc_proj(c));
        WIND_CUDA(tc_gate_table(c));
        WIND_CUDA(launch_set_t(c, t0));
        WIND_CUDA(tc_loop(c, prefix, U, prefix_len, logits, -2));
        return WIND_OK;
    }
    WIND_CUDA(launch_init(c, WIND_KERNELS_SIMT, 0, 0));
    WIND_CUDA(simt_enc_proj(c));
    WIND_CUDA(launch_set_t(c, t0));  // also sets active = B, so the decoder updates run even if every length is 0
    int parity = 0;
    WIND_CUDA(simt_pred_step(c, parity));  // start of sequence
    parity ^= 1;
    for (int u = 0; u < U; ++u) {
        WIND_CUDA(launch_force_tokens(c, prefix, U, prefix_len, u));
        WIND_CUDA(simt_pred_step(c, parity));
        parity ^= 1;
    }
    WIND_CUDA(launch_set_t(c, t0));
    WIND_CUDA(simt_joint(c, logits));
    return WIND_OK;
}

wind_status_t wind_eval_joint_window(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B, int32_t T,
                                     int32_t W, const int32_t* prefix, int32_t U, const int32_t* prefix_len, const int32_t* t0,
                                     float* logits, void* workspace, size_t workspace_bytes, void* stream) {
    Call c;
    wind_status_t s = enqueue_eval_joint_window(c, m, enc, enc_len, B, T, W, prefix, U, prefix_len, t0, logits, workspace,
                                                workspace_bytes, stream);
    if (s != WIND_OK) return s;
    return read_status(c);
}

wind_status_t wind_window_first_output(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B, int32_t T,
                                       int32_t W, const int32_t* prefix, int32_t U, const int32_t* prefix_len, const int32_t* t0,
                                       float* logp, int32_t K, int32_t* top_label, int32_t* top_jump, float* top_logp,
                                       void* workspace, size_t workspace_bytes, void* stream) {
    if (K < 0 || (K > 0 && (!top_label || !top_jump || !top_logp))) return WIND_ERR_INVALID_ARG;
    Call c;
    wind_status_t s = enqueue_eval_joint_window(c, m, enc, enc_len, B, T, W, prefix, U, prefix_len, t0, logp, workspace,
                                                workspace_bytes, stream);
    if (s != WIND_OK) return s;
    WIND_CUDA(launch_first_output(logp, enc_len, t0, B, W, m->V + 1, m->blank_id, K, top_label, top_jump, top_logp, (cudaStream_t)stream));
    return read_status(c);
}

// Scratch of wind_eval_joint_window_static.  In host code `g_static_ws` is only a handle for
// the runtime's symbol lookup, never a device address: the address is resolved below.
static __device__ __align__(256) unsigned char g_static_ws[WIND_STATIC_WORKSPACE_BYTES];
constexpr int kMaxDevices = 64;
static void* g_static_ws_addr[kMaxDevices] = {};
static std::mutex g_static_mutex;

wind_status_t wind_eval_joint_window_static(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B,
                                            int32_t T, int32_t W, const int32_t* prefix, int32_t U,
                                            const int32_t* prefix_len, const int32_t* t0, float* logits, void* stream) {
    size_t need = 0;
    wind_status_t s = wind_workspace_bytes(m, B, T, W, &need);
    if (s != WIND_OK) return s;
    if (need > (size_t)WIND_STATIC_WORKSPACE_BYTES) return WIND_ERR_WORKSPACE;
    int dev = -1;
    WIND_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return WIND_ERR_UNSUPPORTED;
    void* ws = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ws_addr[dev]) {
            // once per device, with that device current: the array's address on this device
            void* addr = nullptr;
            WIND_CUDA(cudaGetSymbolAddress(&addr, g_static_ws));
            g_static_ws_addr[dev] = addr;
        }
        ws = g_static_ws_addr[dev];
    }
    return wind_eval_joint_window(m, enc, enc_len, B, T, W, prefix, U, prefix_len, t0, logits, ws,
                                  (size_t)WIND_STATIC_WORKSPACE_BYTES, stream);
}

wind_status_t wind_profile_decode(const wind_model_t* m, const void* enc, const int32_t* enc_len, int32_t B, int32_t T,
                                  int32_t W, int32_t max_symbols, int32_t* out_tokens, int32_t* out_frames, int32_t* out_len,
                                  int32_t max_out, void* workspace, size_t workspace_bytes, void* stream,
                                  wind_profile_t* host_out) {
    wind_status_t s = check_decode_args(m, enc, enc_len, B, T, W, max_symbols, out_tokens, out_frames, out_len, max_out, workspace);
    if (s != WIND_OK) return s;
    if (!host_out) return WIND_ERR_INVALID_ARG;
    Call c;
    fill_call(c, m, enc, enc_len, B, T, W, max_symbols, out_tokens, out_frames, out_len, max_out, workspace, (cudaStream_t)stream);
    if (workspace_bytes < c.lay.total) return WIND_ERR_WORKSPACE;
    const bool tensor = use_tensor(c);
    if (c.m.dtype == WIND_DT_BF16 && g_kernels == WIND_KERNELS_TENSOR && !tensor) return WIND_ERR_UNSUPPORTED;
    memset(host_out, 0, sizeof(*host_out));
    if (tensor) {
        // every kernel is bracketed by CUDA events on the stream; the loop is one kernel, so its phases are
        // split by the SM cycles CTA 0 counted in each of them
        cudaEvent_t ev[4];
        for (auto& e : ev) WIND_CUDA(cudaEventCreate(&e));
        WIND_CUDA(tc_prepare(c));
        WIND_CUDA(launch_init(c, WIND_KERNELS_TENSOR, 0, tc_setup_launches(c)));
        WIND_CUDA(cudaEventRecord(ev[0], c.stream));
        WIND_CUDA(tc_enc_proj(c));
        WIND_CUDA(cudaEventRecord(ev[1], c.stream));
        WIND_CUDA(tc_gate_table(c));
        WIND_CUDA(cudaEventRecord(ev[2], c.stream));
        WIND_CUDA(tc_loop(c, nullptr, 0, nullptr, nullptr, g_trace_step));
        WIND_CUDA(cudaEventRecord(ev[3], c.stream));
        Ctrl hc;
        WIND_CUDA(cudaMemcpyAsync(&hc, c.ctrl(), sizeof(Ctrl), cudaMemcpyDeviceToHost, c.stream));
        WIND_CUDA(cudaStreamSynchronize(c.stream));
        float ms_proj = 0.f, ms_table = 0.f, ms_loop = 0.f;
        cudaEventElapsedTime(&ms_proj, ev[0], ev[1]);
        cudaEventElapsedTime(&ms_table, ev[1], ev[2]);
        cudaEventElapsedTime(&ms_loop, ev[2], ev[3]);
        for (auto& e : ev) cudaEventDestroy(e);
        host_out->enc_proj_ms = ms_proj;
        host_out->enc_proj_launches = 1;
        host_out->gate_table_ms = ms_table;
        const double cyc = (double)(hc.phase_cycles[0] + hc.phase_cycles[1] + hc.phase_cycles[2]);
        const double ms_per_cycle = cyc > 0 ? (double)ms_loop / cyc : 0.0;
        host_out->joint_ms = hc.phase_cycles[0] * ms_per_cycle;
        host_out->pred_ms = (hc.phase_cycles[1] + hc.phase_cycles[2]) * ms_per_cycle;
        host_out->control_ms = 0.0;   // the control step runs inside the decoder-update phase
        host_out->joint_launches = hc.step;       // phases, not launches: one joint phase per lock step
        host_out->pred_launches = hc.step + 1;
        host_out->control_launches = 0;
        host_out->loop_ms = ms_loop;
        host_out->lstm_ms = hc.phase_cycles[1] * ms_per_cycle;
        host_out->proj_ms = hc.phase_cycles[2] * ms_per_cycle;
        return (wind_status_t)hc.status;
    }
    constexpr int kBurst = 32;              // steps per burst
    constexpr int kEvents = 3 * kBurst + 1; // joint | control | pred boundaries
    std::vector<cudaEvent_t> ev(kEvents);
    for (auto& e : ev) WIND_CUDA(cudaEventCreate(&e));
    auto destroy = [&]() { for (auto& e : ev) cudaEventDestroy(e); };
    const int pred_l = simt_pred_launches(c);
    WIND_CUDA(launch_init(c, WIND_KERNELS_SIMT, 2 + pred_l, 2 + pred_l));
    WIND_CUDA(cudaEventRecord(ev[0], c.stream));
    WIND_CUDA(simt_enc_proj(c));
    WIND_CUDA(cudaEventRecord(ev[1], c.stream));
    WIND_CUDA(simt_pred_step(c, 0));
    WIND_CUDA(cudaEventRecord(ev[2], c.stream));
    WIND_CUDA(cudaStreamSynchronize(c.stream));
    float ms = 0.f;
    cudaEventElapsedTime(&ms, ev[0], ev[1]); host_out->enc_proj_ms += ms; host_out->enc_proj_launches += 1;
    cudaEventElapsedTime(&ms, ev[1], ev[2]); host_out->pred_ms += ms; host_out->pred_launches += pred_l;
    cudaGraphConditionalHandle none{};
    int parity = 1;
    for (;;) {
        Ctrl before;
        WIND_CUDA(cudaMemcpyAsync(&before, c.ctrl(), sizeof(Ctrl), cudaMemcpyDeviceToHost, c.stream));
        WIND_CUDA(cudaStreamSynchronize(c.stream));
        if (before.active == 0) break;
        WIND_CUDA(cudaEventRecord(ev[0], c.stream));
        for (int k = 0; k < kBurst; ++k) {
            WIND_CUDA(simt_joint(c, nullptr));
            WIND_CUDA(cudaEventRecord(ev[3 * k + 1], c.stream));
            WIND_CUDA(launch_control(c, none, 0));
            WIND_CUDA(cudaEventRecord(ev[3 * k + 2], c.stream));
            WIND_CUDA(simt_pred_step(c, parity));
            WIND_CUDA(cudaEventRecord(ev[3 * k + 3], c.stream));
            parity ^= 1;
        }
        Ctrl after;
        WIND_CUDA(cudaMemcpyAsync(&after, c.ctrl(), sizeof(Ctrl), cudaMemcpyDeviceToHost, c.stream));
        WIND_CUDA(cudaStreamSynchronize(c.stream));
        const int live = after.step - before.step;  // steps of this burst that did real work
        for (int k = 0; k < live && k < kBurst; ++k) {
            cudaEventElapsedTime(&ms, ev[3 * k], ev[3 * k + 1]); host_out->joint_ms += ms;
            cudaEventElapsedTime(&ms, ev[3 * k + 1], ev[3 * k + 2]); host_out->control_ms += ms;
            cudaEventElapsedTime(&ms, ev[3 * k + 2], ev[3 * k + 3]); host_out->pred_ms += ms;
        }
        host_out->joint_launches += live;
        host_out->control_launches += live;
        host_out->pred_launches += (int64_t)live * pred_l;
    }
    destroy();
    return read_status(c);
}

static wind_status_t check_beam_args(const wind_model_t* m, int32_t T, int32_t W, int32_t K, int32_t S) {
    wind_status_t s = check_model(m);
    if (s != WIND_OK) return s;
    if (K < 1 || S < 1) return WIND_ERR_INVALID_ARG;
    if (K > 16) return WIND_ERR_UNSUPPORTED;
    return check_shape(m, K, T, W);
}

wind_status_t wind_beam_workspace_bytes(const wind_model_t* m, int32_t T, int32_t W, int32_t K, int32_t max_symbols,
                                        size_t* bytes) {
    wind_status_t s = check_beam_args(m, T, W, K, max_symbols);
    if (s != WIND_OK) return s;
    if (!bytes) return WIND_ERR_INVALID_ARG;
    *bytes = make_beam_layout(*m, T, W, K, max_symbols, make_layout(*m, K, T, W, 1).total).total;
    return WIND_OK;
}

wind_status_t wind_beam_search(const wind_model_t* m, const void* enc, int32_t T, int32_t W, int32_t K, int32_t max_symbols,
                               int32_t prefix_search, int32_t max_hyps, int32_t max_out, int32_t* out_tokens_host, int32_t* out_frames_host,
                               int32_t* out_len_host, double* out_score_host, int32_t* n_hyps_host, int64_t* n_steps_host,
                               void* workspace, size_t workspace_bytes, void* stream) {
    wind_status_t s = check_beam_args(m, T, W, K, max_symbols);
    if (s != WIND_OK) return s;
    s = check_weights(m);
    if (s != WIND_OK) return s;
    if (!enc || !out_tokens_host || !out_frames_host || !out_len_host || !out_score_host || !n_hyps_host || !workspace ||
        max_hyps < 1 || max_out < 1)
        return WIND_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return WIND_ERR_WORKSPACE;
    Call cb;
    fill_call(cb, m, enc, nullptr, K, T, W, max_symbols, nullptr, nullptr, nullptr, 1, workspace, (cudaStream_t)stream);
    const BeamLayout bl = make_beam_layout(*m, T, W, K, max_symbols, cb.lay.total);
    if (workspace_bytes < bl.total) return WIND_ERR_WORKSPACE;
    cudaError_t ce = cudaSuccess;
    s = beam_search_run(cb, bl, K, prefix_search != 0, max_hyps, max_out, out_tokens_host, out_frames_host, out_len_host, out_score_host,
                        n_hyps_host, n_steps_host, &ce);
    if (s == WIND_ERR_CUDA) return cuda_fail(ce, "beam search");
    return s;
}

wind_status_t wind_plan_batches(const int32_t* enc_len, int32_t N, int32_t B, int32_t* order, int32_t* batch_T,
                                int32_t* n_batches) {
    if (!enc_len || !order || !n_batches || N < 0 || B < 1) return WIND_ERR_INVALID_ARG;
    for (int32_t i = 0; i < N; ++i)
        if (enc_len[i] < 0) return WIND_ERR_INVALID_ARG;
    for (int32_t i = 0; i < N; ++i) order[i] = i;
    std::stable_sort(order, order + N, [&](int32_t a, int32_t b) { return enc_len[a] > enc_len[b]; });
    const int32_t nb = (N + B - 1) / B;
    if (batch_T)
        for (int32_t k = 0; k < nb; ++k) batch_T[k] = enc_len[order[(size_t)k * B]];   // sorted: the batch's first is its longest
    *n_batches = nb;
    return WIND_OK;
}

wind_status_t wind_read_stats(const void* workspace, void* stream, wind_stats_t* host_out) {
    if (!workspace || !host_out) return WIND_ERR_INVALID_ARG;
    Ctrl hc;
    WIND_CUDA(cudaMemcpyAsync(&hc, workspace, sizeof(Ctrl), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    WIND_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    memset(host_out, 0, sizeof(*host_out));
    host_out->steps = hc.step;
    host_out->joint_rows = hc.joint_rows;
    host_out->tokens = hc.tokens;
    host_out->forced = hc.forced;
    host_out->frames = hc.frames;
    for (int k = 0; k < 65; ++k) host_out->jump_hist[k] = hc.jump_hist[k];
    host_out->status = hc.status;
    host_out->launches_per_step = hc.launches_per_step;
    host_out->launches_setup = hc.launches_setup;
    host_out->kernels = hc.kernels;
    host_out->timeout_site = hc.timeout_site;
    host_out->timeout_cta = hc.timeout_cta;
    return WIND_OK;
}

wind_status_t wind_bench_joint(const wind_model_t* m, int32_t B, int32_t W, int32_t iters, void* workspace, size_t workspace_bytes,
                               void* stream, wind_joint_bench_t* host_out) {
    wind_status_t s = check_model(m);
    if (s != WIND_OK) return s;
    s = check_shape(m, B, 1, W);
    if (s != WIND_OK) return s;
    if (!m->w_out || !m->b_out || !workspace || !host_out || iters < 1) return WIND_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return WIND_ERR_WORKSPACE;
    memset(host_out, 0, sizeof(*host_out));
    Call c;
    memset(&c, 0, sizeof(c));
    c.m = *m;
    c.m.w_ih = nullptr; c.m.w_hh = nullptr; c.m.b_ih = nullptr; c.m.b_hh = nullptr;
    for (int l = 0; l < m->L; ++l) {    // the tensor maps of the decoder's weights are built with the plan; nothing reads them here
        c.w_ih[l] = m->w_ih ? m->w_ih[l] : nullptr; c.w_hh[l] = m->w_hh ? m->w_hh[l] : nullptr;
        c.b_ih[l] = m->b_ih ? m->b_ih[l] : nullptr; c.b_hh[l] = m->b_hh ? m->b_hh[l] : nullptr;
    }
    c.B = B; c.T = 1; c.W = W; c.S = 1; c.max_out = 1;
    c.ws = static_cast<uint8_t*>(workspace);
    c.lay = make_layout(*m, B, 1, W, 1);
    c.stream = (cudaStream_t)stream;
    c.joint_iters = iters;
    if (workspace_bytes < c.lay.total) return WIND_ERR_WORKSPACE;
    if (!(m->dtype == WIND_DT_BF16 && tc_supported(c.m, B, 1, W)) || !m->w_pred || !c.w_hh[0]) return WIND_ERR_UNSUPPORTED;
    // the kernel whose joint phase reads z from the workspace: grid barriers (resident weights) or streamed weights
    const LoopOptions saved = loop_get_options();
    LoopOptions o = saved;
    o.dataflow = 0;
    loop_set_options(o);
    cudaError_t pe = loop_prepare(c);
    LoopPlan pl;
    cudaError_t pe2 = pe == cudaSuccess ? loop_plan(c, &pl) : pe;
    loop_set_options(saved);
    if (pe2 != cudaSuccess) return cuda_fail(pe2, "plan of the joint phase");
    WIND_CUDA(cudaMemsetAsync(c.ctrl(), 0, sizeof(Ctrl), c.stream));
    WIND_CUDA(cudaMemsetAsync(c.keys(), 0, sizeof(unsigned long long) * 3 * (size_t)c.lay.rows_pad, c.stream));
    WIND_CUDA(launch_fill_z(c));
    cudaEvent_t ev[2];
    for (auto& e : ev) WIND_CUDA(cudaEventCreate(&e));
    // one short launch first (first-use costs), then the timed one
    c.joint_iters = iters < 8 ? iters : 8;
    WIND_CUDA(tc_loop(c, nullptr, 0, nullptr, nullptr, -2));
    c.joint_iters = iters;
    WIND_CUDA(cudaEventRecord(ev[0], c.stream));
    WIND_CUDA(tc_loop(c, nullptr, 0, nullptr, nullptr, -2));
    WIND_CUDA(cudaEventRecord(ev[1], c.stream));
    const wind_status_t st = read_status(c);
    float ms = 0.f;
    cudaEventElapsedTime(&ms, ev[0], ev[1]);
    for (auto& e : ev) cudaEventDestroy(e);
    host_out->ms = ms;
    host_out->iters = iters;
    host_out->resident = pl.resident;
    host_out->rows = (int64_t)B * W;
    host_out->rows_issued = (int64_t)pl.rg_count * pl.nj;
    host_out->labels_issued = (int64_t)pl.vt_count * 128;
    host_out->ctas = pl.resident ? (pl.vt_count * (pl.rg_count < pl.rg_stride ? pl.rg_count : pl.rg_stride)) : (pl.j_items < pl.grid ? pl.j_items : pl.grid);
    return st;
}

int32_t wind_debug_stall_barrier(int32_t extra_arrivals) { return loop_set_extra_arrivals(extra_arrivals); }

void wind_set_loop_options(int32_t resident, int32_t joint_placement, int32_t max_joint_waves, int32_t dataflow) {
    LoopOptions o;
    o.resident = resident != 0;
    o.joint_placement = joint_placement >= 0 && joint_placement <= 2 ? joint_placement : -1;
    o.max_joint_waves = max_joint_waves >= 1 && max_joint_waves <= 4 ? max_joint_waves : 4;
    o.dataflow = dataflow < 0 ? -1 : (dataflow != 0);
    loop_set_options(o);
}

wind_status_t wind_debug_plan(const wind_model_t* m, int32_t B, int32_t W, int32_t sms, int32_t smem_optin, wind_plan_t* out) {
    wind_status_t s = check_model(m);
    if (s != WIND_OK) return s;
    if (!out || B < 1 || W < 1 || W > kMaxWindow || sms < 1 || smem_optin < 1) return WIND_ERR_INVALID_ARG;
    memset(out, 0, sizeof(*out));
    if (!(m->dtype == WIND_DT_BF16 && m->D % 64 == 0 && m->E % 64 == 0 && m->P % 64 == 0 && m->H % 64 == 0 && m->V + 1 >= 128))
        return WIND_ERR_UNSUPPORTED;
    LoopPlan pl;
    if (loop_plan_for(*m, B, W, sms, smem_optin, &pl) != cudaSuccess) return WIND_ERR_UNSUPPORTED;
    out->grid = pl.grid; out->resident = pl.resident; out->dataflow = pl.resident ? pl.dataflow : 0; out->smem_bytes = (int32_t)pl.smem_bytes;
    out->nj = pl.nj; out->vt_count = pl.vt_count; out->rg_count = pl.rg_count; out->rg_stride = pl.rg_stride; out->j_mode = pl.j_mode;
    out->tm_j = pl.tm_j; out->tm_l = pl.tm_l; out->tm_p = pl.tm_p;
    out->nl = pl.nl; out->np = pl.np; out->ut_count = pl.ut_count; out->ht_count = pl.ht_count; out->ql_count = pl.ql_count;
    out->qp_count = pl.qp_count; out->l_items = pl.l_items; out->p_items = pl.p_items; out->w_first = pl.w_first; out->w_count = pl.w_count;
    out->tile_bytes = (int32_t)pl.stat_bytes; out->buf_off = (int32_t)pl.buf_off; out->z_off = (int32_t)pl.z_off;
    out->z_off_p = (int32_t)pl.z_off_p; out->stage_off = (int32_t)pl.stage_off;
    out->slots = pl.slots; out->ul = pl.ul; out->ug_count = pl.ug_count; out->mt_count = pl.mt_count; out->hg_count = pl.hg_count;
    out->stages_lp = pl.stages_lp; out->stages_j = pl.stages_j; out->stage_lp = (int32_t)pl.stage_lp; out->stage_j = (int32_t)pl.stage_j;
    out->l_sets = pl.resident ? (m->L == 2 ? 3 : 1) : 0;
    return WIND_OK;
}

int32_t wind_set_trace(int32_t first_step) {
    int32_t prev = g_trace_step;
    g_trace_step = first_step < -1 ? -2 : first_step;
    return prev;
}

wind_status_t wind_read_trace(const wind_model_t* m, int32_t B, int32_t T, int32_t W, const void* workspace, void* stream,
                              wind_trace_event_t* host_out, int32_t capacity, int32_t* n_out) {
    wind_status_t s = check_model(m);
    if (s != WIND_OK) return s;
    s = check_shape(m, B, T, W);
    if (s != WIND_OK) return s;
    if (!workspace || !host_out || !n_out || capacity < 0) return WIND_ERR_INVALID_ARG;
    *n_out = 0;
    if (m->dtype != WIND_DT_BF16) return WIND_OK;
    Layout lay = make_layout(*m, B, T, W, 1);
    std::vector<TraceEvent> ev((size_t)kTraceRoles * kTraceEvents);
    WIND_CUDA(cudaMemcpyAsync(ev.data(), static_cast<const uint8_t*>(workspace) + lay.trace, ev.size() * sizeof(TraceEvent),
                              cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    WIND_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    int n = 0;
    for (int r = 0; r < kTraceRoles; ++r)
        for (int k = 0; k < kTraceEvents; ++k) {
            const TraceEvent& t = ev[(size_t)r * kTraceEvents + k];
            if (t.clock == 0 || n >= capacity) continue;
            host_out[n].role = r;
            host_out[n].phase = (int32_t)(t.tag / 16);
            host_out[n].event = (int32_t)(t.tag % 16);
            host_out[n].step = t.step;
            host_out[n].clock = t.clock;
            ++n;
        }
    *n_out = n;
    return WIND_OK;
}

int32_t wind_set_kernels(int32_t kernels) {
    int32_t prev = g_kernels;
    if (kernels >= WIND_KERNELS_AUTO && kernels <= WIND_KERNELS_TENSOR) g_kernels = kernels;
    return prev;
}

const char* wind_status_string(wind_status_t s) {
    switch (s) {
        case WIND_OK: return "WIND_OK";
        case WIND_ERR_INVALID_ARG: return "WIND_ERR_INVALID_ARG";
        case WIND_ERR_UNSUPPORTED: return "WIND_ERR_UNSUPPORTED";
        case WIND_ERR_CUDA: return "WIND_ERR_CUDA";
        case WIND_ERR_OUTPUT_OVERFLOW: return "WIND_ERR_OUTPUT_OVERFLOW";
        case WIND_ERR_TIMEOUT: return "WIND_ERR_TIMEOUT";
        case WIND_ERR_INTERNAL: return "WIND_ERR_INTERNAL";
        case WIND_ERR_WORKSPACE: return "WIND_ERR_WORKSPACE";
    }
    return "WIND_ERR_UNKNOWN";
}

const char* wind_last_cuda_error(void) { return g_cuda_err; }

}  // extern "C"
