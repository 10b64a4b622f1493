// Tensor-core kernels for the bf16 path (sm_100a): tcgen05.mma with fp32 accumulators in
// tensor memory, operands staged in shared memory by TMA (or computed by warps, for the
// joint's activation tile), mbarrier pipelines, one elected MMA-issuing thread per CTA.
//
//   gemm kernel, three epilogues:
//     ENC_PROJ  enc_proj[r, :] = enc[r, :] . W_enc^T + b_enc           (rows = frames, bf16 store)
//     LSTM      gates^T = [W_ih | W_hh] . [x | h]^T, then the cell update  (rows = gate units, columns = utterances)
//     PRED_PROJ pred_proj^T = W_pred . h_top^T + b_pred                  (rows = joint units, columns = utterances)
//   joint kernel: A = act(enc_proj window rows + pred_proj) built in shared memory by
//     producer warps, B = W_out tile by TMA, epilogue = per-row argmax key (or logits store).
//
// Every wait on an mbarrier is bounded: after about two seconds the CTA flags
// WIND_ERR_TIMEOUT in the control block, stops waiting, frees its tensor memory and returns.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <mutex>

#include "wind_internal.cuh"

namespace wind {

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

// Bounded wait.  Returns false when the CTA has given up (this wait or an earlier one ran out).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (*abort_flag) return false;
            unsigned long long now = globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* tmap, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_u32(smem_dst)),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, one CTA.
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 lanes x 16 consecutive columns: thread `lane` of the warp gets its row's 16 fp32 values.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor: K-major tile, rows of 64 bf16 (128 bytes), 128-byte swizzle,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);  // start address
    d |= (uint64_t)1 << 16;                         // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                         // 128-byte swizzle
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__host__ __device__ constexpr uint32_t idesc_bf16(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

constexpr int BK = 64;              // K elements per pipeline stage (one 128-byte swizzle row)
constexpr int BM = 128;             // MMA M
constexpr int A_STAGE_BYTES = BM * BK * 2;

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float tanh_fast(float x) {
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float sigmoid_f(float x) { return 1.f / (1.f + __expf(-x)); }

// ---------------------------------------------------------------------------
// Tensor maps (host)
// ---------------------------------------------------------------------------
struct TcMaps {
    CUtensorMap enc, w_enc, w_pred, w_out;
    CUtensorMap w_ih[kMaxLayers], w_hh[kMaxLayers];
    CUtensorMap hb[2][kMaxLayers];
    int joint_bn;   // N tile of the joint kernel
    int batch_n;    // N tile (utterances) of the decoder kernels
};

static PFN_cuTensorMapEncodeTiled g_encode = nullptr;
static std::mutex g_tc_mutex;

static cudaError_t get_encode() {
    std::lock_guard<std::mutex> lock(g_tc_mutex);
    if (g_encode) return cudaSuccess;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess) return e;
    if (q != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(fn);
    return cudaSuccess;
}

// bf16 matrix [rows, cols] row-major, box = box_rows x 64 columns, 128-byte swizzle, zero fill outside.
static cudaError_t make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

bool tc_supported(const wind_model_t& m, int B, int T, int W) {
    (void)B; (void)T; (void)W;
    return m.dtype == WIND_DT_BF16 && m.D % 64 == 0 && m.E % 64 == 0 && m.P % 64 == 0 && m.H % 64 == 0;
}

static int pick_joint_bn(int rows, int nv) {
    // one wave on 148 SMs if possible; cost model: activation tile production ~ one unit,
    // MMA + epilogue ~ BN / 128 units, per wave
    const int m_tiles = (rows + BM - 1) / BM;
    int best = 128;
    double best_cost = 1e30;
    for (int bn : {32, 64, 128, 256}) {
        int n_tiles = (nv + bn - 1) / bn;
        long long ctas = (long long)m_tiles * n_tiles;
        long long waves = (ctas + 147) / 148;
        double cost = (double)waves * (1.0 + bn / 128.0);
        if (cost < best_cost - 1e-9) { best_cost = cost; best = bn; }
    }
    return best;
}

static thread_local TcMaps t_maps;
cudaError_t tc_set_attributes(int joint_bn, int batch_n);

cudaError_t tc_prepare(Call& c) {
    cudaError_t e = get_encode();
    if (e != cudaSuccess) return e;
    TcMaps& M = t_maps;
    const wind_model_t& m = c.m;
    M.joint_bn = pick_joint_bn(c.B * c.W, m.V + 1);
    M.batch_n = c.lay.Bpad <= 256 ? c.lay.Bpad : 256;
#define WIND_MAP(call_) do { e = (call_); if (e != cudaSuccess) return e; } while (0)
    WIND_MAP(make_map(&M.enc, c.enc, (uint64_t)c.B * c.T, m.D, BM));
    WIND_MAP(make_map(&M.w_enc, m.w_enc, m.H, m.D, 128));
    WIND_MAP(make_map(&M.w_pred, m.w_pred, m.H, m.P, BM));
    WIND_MAP(make_map(&M.w_out, m.w_out, (uint64_t)m.V + 1, m.H, M.joint_bn));
    for (int l = 0; l < m.L; ++l) {
        WIND_MAP(make_map(&M.w_ih[l], c.w_ih[l], 4ull * m.P, l == 0 ? m.E : m.P, 32));
        WIND_MAP(make_map(&M.w_hh[l], c.w_hh[l], 4ull * m.P, m.P, 32));
        for (int p = 0; p < 2; ++p) WIND_MAP(make_map(&M.hb[p][l], c.hb(p, l), c.lay.Bpad, m.P, M.batch_n));
    }
#undef WIND_MAP
    c.tc = &M;
    return tc_set_attributes(M.joint_bn, M.batch_n);
}

// ---------------------------------------------------------------------------
// GEMM kernel with TMA-fed operands
// ---------------------------------------------------------------------------
enum GemmMode { MODE_ENC_PROJ = 0, MODE_LSTM = 1, MODE_PRED_PROJ = 2 };

struct GemmParams {
    Ctrl* ctrl;
    int k_blocks_a0;          // K blocks taken from the first A/B map pair (LSTM: the x part), rest from the second
    int k_blocks;             // total K blocks
    int n_tile;               // MMA N (multiple of 16, <= 256)
    int tmem_cols;            // power of two >= max(32, n_tile)
    // ENC_PROJ
    const int32_t* enc_len; int T; long long rows; int H;
    __nv_bfloat16* enc_proj; const float* b_enc;
    // LSTM / PRED_PROJ
    int B, P;
    const int32_t* emit_tok;
    const __nv_bfloat16* emb; int E; int gather_x;    // layer 0: x rows gathered from the embedding table
    const float* b_ih; const float* b_hh;
    float* c_state;                                      // [B, P] of this layer
    const __nv_bfloat16* hb_in; __nv_bfloat16* hb_out;  // [Bpad, P] of this layer (in / out parity)
    const float* b_pred; float* pred_proj;
};

constexpr int GEMM_THREADS = 192;  // warp 0: TMA, warp 1: MMA + tensor memory, warps 2..5: epilogue (and x gather)
constexpr int GEMM_STAGES = 4;

template <int MODE>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
            const __grid_constant__ CUtensorMap map_b0, const __grid_constant__ CUtensorMap map_b1, const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[GEMM_STAGES], empty_bar[GEMM_STAGES], accum_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    if (MODE != MODE_ENC_PROJ && p.ctrl->active == 0) return;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tile = p.n_tile;
    const uint32_t b_stage_bytes = (uint32_t)n_tile * BK * 2;
    const uint32_t stage_bytes = A_STAGE_BYTES + b_stage_bytes;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

    // tile coordinates
    // ENC_PROJ: 1-D grid, H tile fastest so that the CTAs sharing a frame tile run together;
    // LSTM: x = block of 32 hidden units, y = utterance tile; PRED_PROJ: x = H tile, y = utterance tile
    const int h_tiles = MODE == MODE_ENC_PROJ ? (p.H + 127) / 128 : 1;
    const int m_tile = MODE == MODE_ENC_PROJ ? (int)(blockIdx.x % h_tiles) : (int)blockIdx.x;
    const int n_blk = MODE == MODE_ENC_PROJ ? (int)(blockIdx.x / h_tiles) : (int)blockIdx.y;
    if (MODE == MODE_ENC_PROJ) {
        // skip row tiles without a valid frame (block-uniform)
        long long r0 = (long long)n_blk * BM, rl = r0 + BM - 1;
        if (rl >= p.rows) rl = p.rows - 1;
        int b0 = (int)(r0 / p.T), b1 = (int)(rl / p.T);
        bool any = false;
        for (int b = b0; b <= b1; ++b) {
            long long first = (long long)b * p.T > r0 ? (long long)b * p.T : r0;
            if (first <= rl && first - (long long)b * p.T < p.enc_len[b]) any = true;
        }
        if (!any) return;
    }

    const bool gather = (MODE == MODE_LSTM) && p.gather_x;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < GEMM_STAGES; ++s) {
            mbar_init(&full_bar[s], gather ? 5 : 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&accum_bar, 1);
        fence_barrier_init();
        prefetch_tmap(&map_a0); prefetch_tmap(&map_a1); prefetch_tmap(&map_b0); prefetch_tmap(&map_b1);
    }
    if (warp == 1) tmem_alloc(&tmem_slot, (uint32_t)p.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            for (int kb = 0; kb < p.k_blocks; ++kb) {
                const int s = kb % GEMM_STAGES;
                const uint32_t par = ((kb / GEMM_STAGES) & 1) ^ 1;
                if (!mbar_wait(&empty_bar[s], par, &abort_flag)) break;
                uint8_t* a_dst = smem + (size_t)s * stage_bytes;
                uint8_t* b_dst = a_dst + A_STAGE_BYTES;
                const bool first = kb < p.k_blocks_a0;
                const int kx = (first ? kb : kb - p.k_blocks_a0) * BK;
                const CUtensorMap* ma = first ? &map_a0 : &map_a1;
                const CUtensorMap* mb = first ? &map_b0 : &map_b1;
                if (MODE == MODE_ENC_PROJ) {
                    // A = 128 frames of enc, B = 128 rows of W_enc
                    mbar_expect_tx(&full_bar[s], A_STAGE_BYTES + b_stage_bytes);
                    tma_load_2d(a_dst, ma, kx, n_blk * BM, &full_bar[s]);
                    tma_load_2d(b_dst, mb, kx, m_tile * 128, &full_bar[s]);
                } else if (MODE == MODE_LSTM) {
                    // A = 4 gate blocks x 32 hidden units of [W_ih | W_hh], B = utterance rows of [x | h]
                    const bool b_by_tma = !(gather && first);
                    mbar_expect_tx(&full_bar[s], A_STAGE_BYTES + (b_by_tma ? b_stage_bytes : 0));
                    for (int g = 0; g < 4; ++g)
                        tma_load_2d(a_dst + g * 32 * BK * 2, ma, kx, g * p.P + m_tile * 32, &full_bar[s]);
                    if (b_by_tma) tma_load_2d(b_dst, mb, kx, n_blk * n_tile, &full_bar[s]);
                } else {
                    // A = 128 rows of W_pred, B = utterance rows of h_top
                    mbar_expect_tx(&full_bar[s], A_STAGE_BYTES + b_stage_bytes);
                    tma_load_2d(a_dst, ma, kx, m_tile * BM, &full_bar[s]);
                    tma_load_2d(b_dst, mb, kx, n_blk * n_tile, &full_bar[s]);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16(BM, n_tile);
            bool ok = true;
            for (int kb = 0; kb < p.k_blocks && ok; ++kb) {
                const int s = kb % GEMM_STAGES;
                const uint32_t par = (kb / GEMM_STAGES) & 1;
                ok = mbar_wait(&full_bar[s], par, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
                const uint64_t adesc = smem_desc_sw128(a_addr);
                const uint64_t bdesc = smem_desc_sw128(a_addr + A_STAGE_BYTES);
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)
                    tc_mma_bf16(tmem_base, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kb | k) != 0);
                tc_commit(&empty_bar[s]);
            }
            if (ok) tc_commit(&accum_bar);
        }
    } else {
        // ---------------- epilogue warps (and x gather for LSTM layer 0) ----------------
        const int q = warp & 3;            // tensor-memory lane quadrant this warp may read
        const int et = threadIdx.x - 64;   // 0..127
        if (gather) {
            for (int kb = 0; kb < p.k_blocks; ++kb) {
                const int s = kb % GEMM_STAGES;
                const uint32_t par = ((kb / GEMM_STAGES) & 1) ^ 1;
                if (!mbar_wait(&empty_bar[s], par, &abort_flag)) break;
                if (kb < p.k_blocks_a0) {
                    uint8_t* b_dst = smem + (size_t)s * stage_bytes + A_STAGE_BYTES;
                    for (int ch = et; ch < n_tile * 8; ch += 128) {
                        const int row = ch >> 3, kc = ch & 7;
                        const int b = n_blk * n_tile + row;
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (b < p.B) {
                            const int tok = p.emit_tok[b];
                            const int col = kb * BK + kc * 8;
                            if (tok >= 0 && col < p.E) v = *reinterpret_cast<const uint4*>(p.emb + (size_t)tok * p.E + col);
                        }
                        *reinterpret_cast<uint4*>(b_dst + row * 128 + ((kc ^ (row & 7)) << 4)) = v;
                    }
                    fence_proxy_async();
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&full_bar[s]);
            }
        }
        const bool ready = __all_sync(0xffffffffu, mbar_wait(&accum_bar, 0, &abort_flag));
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
        if (MODE == MODE_LSTM) {
            // stage 1: gate pre-activations to shared memory (the drained pipeline buffers), [gate][utterance][unit]
            float* gsm = reinterpret_cast<float*>(smem);
            if (ready) {
                for (int c0 = 0; c0 < n_tile; c0 += 16) {
                    float v[16];
                    tmem_ld16(taddr + c0, v);
#pragma unroll
                    for (int i = 0; i < 16; ++i) gsm[((size_t)q * n_tile + c0 + i) * 32 + lane] = v[i];
                }
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");   // all four epilogue warps, whatever `ready` says
            if (ready && !abort_flag) {
                // stage 2: cell update; lane = unit, warp q takes utterances q, q+4, ...
                const int j = m_tile * 32 + lane;
                const float bi = p.b_ih[j] + p.b_hh[j], bf = p.b_ih[p.P + j] + p.b_hh[p.P + j];
                const float bg = p.b_ih[2 * p.P + j] + p.b_hh[2 * p.P + j], bo = p.b_ih[3 * p.P + j] + p.b_hh[3 * p.P + j];
                for (int col = q; col < n_tile; col += 4) {
                    const int b = n_blk * n_tile + col;
                    if (b >= p.B) break;
                    const size_t idx = (size_t)b * p.P + j;
                    if (p.emit_tok[b] < 0) {
                        p.hb_out[idx] = p.hb_in[idx];
                        continue;
                    }
                    const float gi = sigmoid_f(gsm[((size_t)0 * n_tile + col) * 32 + lane] + bi);
                    const float gf = sigmoid_f(gsm[((size_t)1 * n_tile + col) * 32 + lane] + bf);
                    const float gg = tanhf(gsm[((size_t)2 * n_tile + col) * 32 + lane] + bg);
                    const float go = sigmoid_f(gsm[((size_t)3 * n_tile + col) * 32 + lane] + bo);
                    const float cc = gf * p.c_state[idx] + gi * gg;
                    p.c_state[idx] = cc;
                    p.hb_out[idx] = __float2bfloat16_rn(go * tanhf(cc));
                }
            }
        } else if (ready) {
            if (MODE == MODE_ENC_PROJ) {
                const long long r = (long long)n_blk * BM + q * 32 + lane;
                bool valid = false;
                if (r < p.rows) {
                    const int b = (int)(r / p.T);
                    valid = (int)(r - (long long)b * p.T) < p.enc_len[b];
                }
                for (int c0 = 0; c0 < n_tile; c0 += 16) {
                    float v[16];
                    tmem_ld16(taddr + c0, v);
                    const int h0 = m_tile * 128 + c0;
                    if (valid && h0 < p.H) {   // H is a multiple of 64, so 16-column groups are all-in or all-out
                        uint32_t w[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) w[i] = pack_bf16x2(v[2 * i] + p.b_enc[h0 + 2 * i], v[2 * i + 1] + p.b_enc[h0 + 2 * i + 1]);
                        uint4* dst = reinterpret_cast<uint4*>(p.enc_proj + r * p.H + h0);
                        dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                        dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
                    }
                }
            } else {
                const int o = m_tile * BM + q * 32 + lane;
                const float bias = o < p.H ? p.b_pred[o] : 0.f;
                for (int c0 = 0; c0 < n_tile; c0 += 16) {
                    float v[16];
                    tmem_ld16(taddr + c0, v);
                    if (o < p.H) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const int b = n_blk * n_tile + c0 + i;
                            if (b < p.B) p.pred_proj[(size_t)b * p.H + o] = v[i] + bias;
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
    if (threadIdx.x == 0 && abort_flag) set_status(p.ctrl, WIND_ERR_TIMEOUT);
}

static int tmem_cols_for(int n) {
    int c = 32;
    while (c < n) c <<= 1;
    return c;
}

static size_t gemm_smem_bytes(int n_tile) { return (size_t)GEMM_STAGES * (A_STAGE_BYTES + (size_t)n_tile * BK * 2) + 1024; }

template <int MODE>
static cudaError_t ensure_gemm_smem(size_t smem) {
    static size_t attr_set = 0;
    if (smem > attr_set) {
        cudaError_t e = cudaFuncSetAttribute(gemm_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_set = smem;
    }
    return cudaSuccess;
}

template <int MODE>
static cudaError_t launch_gemm(const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& b0, const CUtensorMap& b1,
                               const GemmParams& p, dim3 grid, cudaStream_t stream) {
    gemm_kernel<MODE><<<grid, GEMM_THREADS, gemm_smem_bytes(p.n_tile), stream>>>(a0, a1, b0, b1, p);
    return cudaGetLastError();
}

cudaError_t tc_enc_proj(const Call& c) {
    const TcMaps& M = *static_cast<const TcMaps*>(c.tc);
    GemmParams p{};
    p.ctrl = c.ctrl();
    p.k_blocks = c.m.D / BK;
    p.k_blocks_a0 = p.k_blocks;
    p.n_tile = 128;
    p.tmem_cols = 128;
    p.enc_len = c.enc_len; p.T = c.T; p.rows = (long long)c.B * c.T; p.H = c.m.H;
    p.enc_proj = (__nv_bfloat16*)c.enc_proj(); p.b_enc = c.m.b_enc;
    dim3 grid((unsigned)(((c.m.H + 127) / 128) * ((p.rows + BM - 1) / BM)));
    return launch_gemm<MODE_ENC_PROJ>(M.enc, M.enc, M.w_enc, M.w_enc, p, grid, c.stream);
}

int tc_pred_launches(const Call& c) { return c.m.L + 1; }

cudaError_t tc_pred_step(const Call& c, int parity_in) {
    const TcMaps& M = *static_cast<const TcMaps*>(c.tc);
    const int po = 1 - parity_in;
    const int n_tile = M.batch_n;
    const unsigned n_blocks = (unsigned)((c.lay.Bpad + n_tile - 1) / n_tile);
    for (int l = 0; l < c.m.L; ++l) {
        GemmParams p{};
        p.ctrl = c.ctrl();
        const int n_in = l == 0 ? c.m.E : c.m.P;
        p.k_blocks_a0 = n_in / BK;
        p.k_blocks = p.k_blocks_a0 + c.m.P / BK;
        p.n_tile = n_tile;
        p.tmem_cols = tmem_cols_for(n_tile);
        p.B = c.B; p.P = c.m.P; p.emit_tok = c.emit_tok();
        p.emb = (const __nv_bfloat16*)c.m.emb; p.E = c.m.E; p.gather_x = (l == 0);
        p.b_ih = c.b_ih[l]; p.b_hh = c.b_hh[l];
        p.c_state = c.c() + (size_t)l * c.B * c.m.P;
        p.hb_in = c.hb(parity_in, l); p.hb_out = c.hb(po, l);
        // x of layer l > 0 is the new h of the layer below (output parity)
        const CUtensorMap& bx = l == 0 ? M.hb[parity_in][0] : M.hb[po][l - 1];
        dim3 grid(c.m.P / 32, n_blocks);
        cudaError_t e = launch_gemm<MODE_LSTM>(M.w_ih[l], M.w_hh[l], bx, M.hb[parity_in][l], p, grid, c.stream);
        if (e != cudaSuccess) return e;
    }
    GemmParams p{};
    p.ctrl = c.ctrl();
    p.k_blocks = c.m.P / BK;
    p.k_blocks_a0 = p.k_blocks;
    p.n_tile = n_tile;
    p.tmem_cols = tmem_cols_for(n_tile);
    p.B = c.B; p.P = c.m.P; p.H = c.m.H;
    p.b_pred = c.m.b_pred; p.pred_proj = c.pred_proj();
    dim3 grid((c.m.H + BM - 1) / BM, n_blocks);
    const CUtensorMap& hb = M.hb[po][c.m.L - 1];
    return launch_gemm<MODE_PRED_PROJ>(M.w_pred, M.w_pred, hb, hb, p, grid, c.stream);
}

// ---------------------------------------------------------------------------
// Fused windowed joint
// ---------------------------------------------------------------------------
struct JointParams {
    Ctrl* ctrl;
    const int32_t* t_cur; const int32_t* enc_len;
    const __nv_bfloat16* enc_proj; const float* pred_proj; const float* b_out;
    unsigned long long* keys; float* logits_out;
    int B, T, W, H, NV, act;
    int k_blocks;
};

constexpr int JOINT_A_WARPS = 8;
constexpr int JOINT_THREADS = 64 + JOINT_A_WARPS * 32;  // warp 0: TMA (W_out), warp 1: MMA, warps 2..9: A producers + epilogue
constexpr int JOINT_STAGES = 4;

template <int BN>
__global__ void __launch_bounds__(JOINT_THREADS, 1)
joint_kernel(const __grid_constant__ CUtensorMap map_wout, const JointParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[JOINT_STAGES], empty_bar[JOINT_STAGES], accum_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    constexpr uint32_t B_STAGE = BN * BK * 2;
    constexpr uint32_t STAGE = A_STAGE_BYTES + B_STAGE;
    constexpr uint32_t TMEM_COLS = BN < 32 ? 32 : BN;

    if (p.ctrl->active == 0) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN;          // first vocabulary column of this tile
    const int row0 = blockIdx.y * BM;        // first window row (b * W + w) of this tile
    const int total_rows = p.B * p.W;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

    // block-uniform early exit: no utterance of this row tile is still decoding
    {
        const int b_first = row0 / p.W;
        int b_last = (min(row0 + BM, total_rows) - 1) / p.W;
        bool any = false;
        for (int b = b_first; b <= b_last; ++b) any |= p.t_cur[b] < p.enc_len[b];
        if (!any) return;
    }

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < JOINT_STAGES; ++s) {
            mbar_init(&full_bar[s], 1 + JOINT_A_WARPS);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&accum_bar, 1);
        fence_barrier_init();
        prefetch_tmap(&map_wout);
    }
    if (warp == 1) tmem_alloc(&tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < p.k_blocks; ++kb) {
                const int s = kb % JOINT_STAGES;
                if (!mbar_wait(&empty_bar[s], ((kb / JOINT_STAGES) & 1) ^ 1, &abort_flag)) break;
                mbar_expect_tx(&full_bar[s], B_STAGE);
                tma_load_2d(smem + (size_t)s * STAGE + A_STAGE_BYTES, &map_wout, kb * BK, n0, &full_bar[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(BM, BN);
            bool ok = true;
            for (int kb = 0; kb < p.k_blocks; ++kb) {
                const int s = kb % JOINT_STAGES;
                ok = mbar_wait(&full_bar[s], (kb / JOINT_STAGES) & 1, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = smem_u32(smem + (size_t)s * STAGE);
                const uint64_t adesc = smem_desc_sw128(a_addr);
                const uint64_t bdesc = smem_desc_sw128(a_addr + A_STAGE_BYTES);
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)
                    tc_mma_bf16(tmem_base, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kb | k) != 0);
                tc_commit(&empty_bar[s]);
            }
            if (ok) tc_commit(&accum_bar);
        }
    } else {
        // ---------------- activation-tile producers ----------------
        // thread -> 16-byte chunk kc of rows rr, rr + 32, rr + 64, rr + 96 of the tile, for every K block
        const int pt = threadIdx.x - 64;        // 0..255
        const int kc = pt & 7;
        const int rr = pt >> 3;                 // 0..31
        const __nv_bfloat16* e_ptr[4];
        const float* g_ptr[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = row0 + rr + 32 * i;
            e_ptr[i] = nullptr;
            g_ptr[i] = nullptr;
            if (r < total_rows) {
                const int b = r / p.W, w = r - b * p.W;
                const int t = p.t_cur[b] + w;
                if (t < p.enc_len[b]) {
                    e_ptr[i] = p.enc_proj + ((size_t)b * p.T + t) * p.H + kc * 8;
                    g_ptr[i] = p.pred_proj + (size_t)b * p.H + kc * 8;
                }
            }
        }
        for (int kb = 0; kb < p.k_blocks; ++kb) {
            const int s = kb % JOINT_STAGES;
            // issue the global loads before waiting for the stage to drain
            uint4 ev[4];
            float4 g0[4], g1[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (e_ptr[i]) {
                    ev[i] = *reinterpret_cast<const uint4*>(e_ptr[i] + kb * BK);
                    g0[i] = *reinterpret_cast<const float4*>(g_ptr[i] + kb * BK);
                    g1[i] = *reinterpret_cast<const float4*>(g_ptr[i] + kb * BK + 4);
                }
            }
            if (!mbar_wait(&empty_bar[s], ((kb / JOINT_STAGES) & 1) ^ 1, &abort_flag)) break;
            uint8_t* a_dst = smem + (size_t)s * STAGE;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 out = make_uint4(0, 0, 0, 0);
                if (e_ptr[i]) {
                    const __nv_bfloat162* eb = reinterpret_cast<const __nv_bfloat162*>(&ev[i]);
                    float z[8];
                    const float gg[8] = {g0[i].x, g0[i].y, g0[i].z, g0[i].w, g1[i].x, g1[i].y, g1[i].z, g1[i].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float2 e2 = __bfloat1622float2(eb[j]);
                        z[2 * j] = e2.x + gg[2 * j];
                        z[2 * j + 1] = e2.y + gg[2 * j + 1];
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) z[j] = p.act == WIND_ACT_RELU ? fmaxf(z[j], 0.f) : tanh_fast(z[j]);
                    out = make_uint4(pack_bf16x2(z[0], z[1]), pack_bf16x2(z[2], z[3]), pack_bf16x2(z[4], z[5]), pack_bf16x2(z[6], z[7]));
                }
                const int row = rr + 32 * i;
                *reinterpret_cast<uint4*>(a_dst + row * 128 + ((kc ^ (row & 7)) << 4)) = out;
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&full_bar[s]);
        }
        // ---------------- epilogue: per-row argmax over this tile's columns ----------------
        const bool ready = __all_sync(0xffffffffu, mbar_wait(&accum_bar, 0, &abort_flag));
        tc_fence_after();
        if (ready) {
            const int q = warp & 3;
            const int half = (warp - 2) >> 2;        // warps 2..5 take the first half of the columns, 6..9 the second
            const int r = row0 + q * 32 + lane;
            bool valid = false;
            if (r < total_rows) {
                const int b = r / p.W, w = r - b * p.W;
                valid = p.t_cur[b] + w < p.enc_len[b];
            }
            constexpr int COLS_PER_HALF = BN / 2;     // multiple of 16 for BN >= 32
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(half * COLS_PER_HALF);
            float best = -INFINITY;
            int best_v = -1;
            for (int c0 = 0; c0 < COLS_PER_HALF; c0 += 16) {
                float v[16];
                tmem_ld16(taddr + c0, v);
                const int vbase = n0 + half * COLS_PER_HALF + c0;
                if (valid) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int vv = vbase + i;
                        if (vv < p.NV) {
                            const float s = v[i] + p.b_out[vv];
                            if (p.logits_out) p.logits_out[(size_t)r * p.NV + vv] = s;
                            if (s > best || best_v < 0) { best = s; best_v = vv; }
                        }
                    }
                }
            }
            if (valid && best_v >= 0) atomicMax(&p.keys[r], pack_key(best, (uint32_t)best_v));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
    if (threadIdx.x == 0 && abort_flag) set_status(p.ctrl, WIND_ERR_TIMEOUT);
}

template <int BN>
constexpr size_t joint_smem_bytes() { return (size_t)JOINT_STAGES * (A_STAGE_BYTES + BN * BK * 2) + 1024; }

template <int BN>
static cudaError_t ensure_joint_smem() {
    static bool done = false;
    if (!done) {
        cudaError_t e = cudaFuncSetAttribute(joint_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)joint_smem_bytes<BN>());
        if (e != cudaSuccess) return e;
        done = true;
    }
    return cudaSuccess;
}

template <int BN>
static cudaError_t launch_joint(const CUtensorMap& map, const JointParams& p, cudaStream_t stream) {
    dim3 grid((p.NV + BN - 1) / BN, (p.B * p.W + BM - 1) / BM);
    joint_kernel<BN><<<grid, JOINT_THREADS, joint_smem_bytes<BN>(), stream>>>(map, p);
    return cudaGetLastError();
}

// Shared-memory opt-in of every kernel this call will launch (kept out of graph capture).
cudaError_t tc_set_attributes(int joint_bn, int batch_n) {
    cudaError_t e;
    if ((e = ensure_gemm_smem<MODE_ENC_PROJ>(gemm_smem_bytes(128))) != cudaSuccess) return e;
    if ((e = ensure_gemm_smem<MODE_LSTM>(gemm_smem_bytes(batch_n))) != cudaSuccess) return e;
    if ((e = ensure_gemm_smem<MODE_PRED_PROJ>(gemm_smem_bytes(batch_n))) != cudaSuccess) return e;
    switch (joint_bn) {
        case 32: return ensure_joint_smem<32>();
        case 64: return ensure_joint_smem<64>();
        case 128: return ensure_joint_smem<128>();
        default: return ensure_joint_smem<256>();
    }
}

cudaError_t tc_joint(const Call& c, float* logits_out) {
    const TcMaps& M = *static_cast<const TcMaps*>(c.tc);
    JointParams p{};
    p.ctrl = c.ctrl();
    p.t_cur = c.t(); p.enc_len = c.enc_len;
    p.enc_proj = (const __nv_bfloat16*)c.enc_proj(); p.pred_proj = c.pred_proj(); p.b_out = c.m.b_out;
    p.keys = c.keys(); p.logits_out = logits_out;
    p.B = c.B; p.T = c.T; p.W = c.W; p.H = c.m.H; p.NV = c.m.V + 1; p.act = c.m.act;
    p.k_blocks = c.m.H / BK;
    switch (M.joint_bn) {
        case 32: return launch_joint<32>(M.w_out, p, c.stream);
        case 64: return launch_joint<64>(M.w_out, p, c.stream);
        case 128: return launch_joint<128>(M.w_out, p, c.stream);
        default: return launch_joint<256>(M.w_out, p, c.stream);
    }
}

}  // namespace wind
