// One-shot tensor-core GEMMs of the bf16 path (sm_100a): tcgen05.mma with fp32 accumulators in
// tensor memory, both operands staged in shared memory by TMA, mbarrier pipeline, one elected
// MMA-issuing thread per CTA.  Two uses, both once per call, outside the decoding loop:
//
//     ENC_PROJ   enc_proj[r, :] = enc[r, :] . W_enc^T + b_enc      (rows = valid frames, bf16 store)
//     GATE_TABLE g0[tok, :] = emb[tok, :] . W_ih[0]^T + b_ih[0] + b_hh[0]   (rows = tokens, fp32 store)
//
// The gate table turns layer 0's input term of the LSTM into a row lookup inside the loop.
//
// Every wait on an mbarrier is bounded: after about two seconds the CTA flags
// WIND_ERR_TIMEOUT in the control block, stops waiting, frees its tensor memory and returns.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <mutex>

#include "wind_internal.cuh"
#include "wind_ptx.cuh"
#include "wind_loop.cuh"

namespace wind {

// ---------------------------------------------------------------------------
// Tensor maps (host)
// ---------------------------------------------------------------------------
struct TcMaps {
    CUtensorMap enc, w_enc, emb, w_ih0;
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
    (void)T;
    if (!(m.dtype == WIND_DT_BF16 && m.D % 64 == 0 && m.E % 64 == 0 && m.P % 64 == 0 && m.H % 64 == 0 && m.V + 1 >= 128)) return false;
    return loop_plan_ok(m, B, W);   // the loop kernels have a tile plan for these shapes on this device
}

static thread_local TcMaps t_maps;
static cudaError_t tc_set_attributes();

cudaError_t tc_prepare(Call& c) {
    cudaError_t e = get_encode();
    if (e != cudaSuccess) return e;
    TcMaps& M = t_maps;
    const wind_model_t& m = c.m;
#define WIND_MAP(call_) do { e = (call_); if (e != cudaSuccess) return e; } while (0)
    WIND_MAP(make_map(&M.enc, c.enc, (uint64_t)(c.N > 0 ? c.N : c.B) * c.T, m.D, BM));
    WIND_MAP(make_map(&M.w_enc, m.w_enc, m.H, m.D, 256));
    WIND_MAP(make_map(&M.emb, m.emb, (uint64_t)m.V + 1, m.E, BM));
    WIND_MAP(make_map(&M.w_ih0, c.w_ih[0], 4ull * m.P, m.E, 128));
#undef WIND_MAP
    c.tc = &M;
    if ((e = tc_set_attributes()) != cudaSuccess) return e;
    return loop_prepare(c);
}

// ---------------------------------------------------------------------------
// GEMM kernel with TMA-fed operands: out[r, n] = sum_k A[r, k] B[n, k] (+ bias)
// ---------------------------------------------------------------------------
enum GemmMode { MODE_ENC_PROJ = 0, MODE_GATE_TABLE = 1 };

struct GemmParams {
    Ctrl* ctrl;
    int k_blocks;             // K blocks of 64
    long long rows;           // rows of A (frames or tokens)
    int N;                    // columns of the output (H or 4P), multiple of 64
    // ENC_PROJ
    const int32_t* enc_len; int T;
    __nv_bfloat16* out_bf16; const float* bias0;
    // GATE_TABLE
    float* out_f32; const float* bias1;
};

constexpr int GEMM_THREADS = 192;  // warp 0: TMA, warp 1: MMA + tensor memory, warps 2..5: epilogue
// Two CTAs share an SM, so that one's epilogue overlaps the other's main loop.  The encoder projection uses 128 x 256
// tiles (the kernel is paced by its two issuing threads: half as many TMA and MMA instructions per flop as with 128 x
// 128) with two 48 KB stages; the gate table (fp32 output, staged through the same buffers) 128 x 128 with three.
template <int MODE> struct GemmShape { static constexpr int BN = MODE == 0 ? 256 : 128; static constexpr int STAGES = MODE == 0 ? 2 : 3; };

template <int MODE>
__global__ void __launch_bounds__(GEMM_THREADS, 2)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[GemmShape<MODE>::STAGES], empty_bar[GemmShape<MODE>::STAGES], accum_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float s_bias[GemmShape<MODE>::BN];
    __shared__ int s_valid[BM];

    constexpr int GEMM_BN = GemmShape<MODE>::BN, GEMM_STAGES = GemmShape<MODE>::STAGES;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t b_stage_bytes = GEMM_BN * BK * 2;
    constexpr uint32_t stage_bytes = A_STAGE_BYTES + b_stage_bytes;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

    // 1-D grid, column tile fastest so that the CTAs sharing a row tile run together
    const int n_tiles = (p.N + GEMM_BN - 1) / GEMM_BN;
    const int n_tile_idx = (int)(blockIdx.x % n_tiles);
    const int m_blk = (int)(blockIdx.x / n_tiles);
    if (MODE == MODE_ENC_PROJ) {
        // skip row tiles without a valid frame (block-uniform)
        long long r0 = (long long)m_blk * BM, rl = r0 + BM - 1;
        if (rl >= p.rows) rl = p.rows - 1;
        int b0 = (int)(r0 / p.T), b1 = (int)(rl / p.T);
        bool any = false;
        for (int b = b0; b <= b1; ++b) {
            long long first = (long long)b * p.T > r0 ? (long long)b * p.T : r0;
            if (first <= rl && first - (long long)b * p.T < p.enc_len[b]) any = true;
        }
        if (!any) return;
    }

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < GEMM_STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&accum_bar, 1);
        fence_barrier_init();
        prefetch_tmap(&map_a); prefetch_tmap(&map_b);
    }
    if (warp == 1) tmem_alloc(&tmem_slot, GEMM_BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < p.k_blocks; ++kb) {
                const int s = kb % GEMM_STAGES;
                const uint32_t par = ((kb / GEMM_STAGES) & 1) ^ 1;
                if (!mbar_wait(&empty_bar[s], par, &abort_flag)) break;
                uint8_t* a_dst = smem + (size_t)s * stage_bytes;
                mbar_expect_tx(&full_bar[s], stage_bytes);
                tma_load_2d(a_dst, &map_a, kb * BK, m_blk * BM, &full_bar[s]);
                tma_load_2d(a_dst + A_STAGE_BYTES, &map_b, kb * BK, n_tile_idx * GEMM_BN, &full_bar[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(BM, GEMM_BN);
            bool ok = true;
            for (int kb = 0; kb < p.k_blocks && ok; ++kb) {
                const int s = kb % GEMM_STAGES;
                ok = mbar_wait(&full_bar[s], (kb / GEMM_STAGES) & 1, &abort_flag);
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
        const int q = warp & 3;            // tensor-memory lane quadrant this warp may read
        const int et = threadIdx.x - 64;   // 0..127
        const int row = q * 32 + lane;     // accumulator row of this thread
        // before the accumulator is ready: this tile's bias values and which of its rows are valid frames
        {
            for (int k = et; k < GEMM_BN; k += 128) {
                const int n = n_tile_idx * GEMM_BN + k;
                float bsum = 0.f;
                if (n < p.N) bsum = p.bias0[n] + (MODE == MODE_GATE_TABLE ? p.bias1[n] : 0.f);
                s_bias[k] = bsum;
            }
            const long long r = (long long)m_blk * BM + row;
            bool valid = r < p.rows;
            if (MODE == MODE_ENC_PROJ && valid) {
                const int b = (int)(r / p.T);
                valid = (int)(r - (long long)b * p.T) < p.enc_len[b];
            }
            s_valid[row] = valid;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const bool ready = __all_sync(0xffffffffu, mbar_wait(&accum_bar, 0, &abort_flag));
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
        // The tile goes through shared memory (the pipeline's buffers: every MMA has completed), so that it leaves
        // as whole row segments: 16 (bf16) or 32 (fp32) neighbouring threads write one row's 256 or 512 bytes.
        constexpr int ELEM = MODE == MODE_ENC_PROJ ? 2 : 4;
        constexpr int ROW_BYTES = GEMM_BN * ELEM + 16;          // padded: consecutive rows start in different banks
        if (ready) {
            uint8_t* my = smem + (size_t)row * ROW_BYTES;
            for (int c0 = 0; c0 < GEMM_BN; c0 += 16) {
                float v[16];
                tmem_ld16(taddr + c0, v);
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] += s_bias[c0 + i];
                if (MODE == MODE_ENC_PROJ) {
                    uint4* dst = reinterpret_cast<uint4*>(my + c0 * 2);
                    dst[0] = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
                    dst[1] = make_uint4(pack_bf16x2(v[8], v[9]), pack_bf16x2(v[10], v[11]), pack_bf16x2(v[12], v[13]), pack_bf16x2(v[14], v[15]));
                } else {
                    float4* dst = reinterpret_cast<float4*>(my + c0 * 4);
#pragma unroll
                    for (int i = 0; i < 4; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                }
            }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (ready) {
            constexpr int CHUNKS = GEMM_BN * ELEM / 16;           // 16-byte chunks per row
            const int n_cols = min(GEMM_BN, p.N - n_tile_idx * GEMM_BN);
            uint8_t* out = MODE == MODE_ENC_PROJ ? reinterpret_cast<uint8_t*>(p.out_bf16) : reinterpret_cast<uint8_t*>(p.out_f32);
            for (int ch = et; ch < BM * CHUNKS; ch += 128) {
                const int rr = ch / CHUNKS, cc = ch - rr * CHUNKS;
                if (s_valid[rr] && cc * 16 < n_cols * ELEM) {
                    const uint4 x = *reinterpret_cast<const uint4*>(smem + (size_t)rr * ROW_BYTES + cc * 16);
                    const long long r = (long long)m_blk * BM + rr;
                    *reinterpret_cast<uint4*>(out + ((size_t)r * p.N + (size_t)n_tile_idx * GEMM_BN) * ELEM + cc * 16) = x;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, GEMM_BN);
    }
    if (threadIdx.x == 0 && abort_flag) set_status(p.ctrl, WIND_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------
// Encoder projection, persistent form: one CTA per SM walks a static list of 128 x 256 output tiles.
//
// Row tiles are cut per utterance (rows b T + 128 j, j < ceil(len_b / 128)), so a tile never holds two utterances and
// the tiles of padding are never enumerated: tile k of the list is found from the prefix sums of the utterances' tile
// counts, which every CTA builds once in shared memory.  Column tile fastest, so that the CTAs working on one row tile
// at the same time fetch it from DRAM once.  Four TMA stages of 48 KB feed one MMA-issuing thread; the accumulator is
// double-buffered in tensor memory (2 x 256 columns), so that the epilogue of a tile (tensor memory -> registers ->
// + bias -> bf16 -> 64 contiguous bytes per thread and store) runs under the next tile's MMAs.  Rows past the
// utterance's end inside a tile are computed and not stored (rows of a GEMM are independent).
// ---------------------------------------------------------------------------
constexpr int EP_STAGES = 4;
constexpr int EP_BN = 256;
constexpr uint32_t EP_STAGE_BYTES = A_STAGE_BYTES + EP_BN * BK * 2;
constexpr int EP_MAX_UTTS = 2048;     // prefix sums in shared memory; larger sets use the one-tile-per-CTA kernel
constexpr int EP_MAX_H = 2048;        // bias values in shared memory

// 256-bit store: one full 32-byte sector per thread (16-byte stores from 32 threads to 32 different rows would touch 32
// sectors half-filled each, twice the traffic between the SM and L2)
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t* w) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]),
                 "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}

struct EncProjParams {
    Ctrl* ctrl;
    int k_blocks, H, T, n_utts;
    const int32_t* enc_len;
    __nv_bfloat16* out;
    const float* bias;
};

__global__ void __launch_bounds__(GEMM_THREADS, 1)
enc_proj_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const EncProjParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[EP_STAGES], empty_bar[EP_STAGES], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int s_prefix[EP_MAX_UTTS + 1];     // s_prefix[b] = row tiles of utterances before b
    __shared__ float s_bias[EP_MAX_H];
    __shared__ int s_scan[GEMM_THREADS / 32];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    if (p.ctrl->bad_input) return;   // a length outside [0, T]: nothing is read through it

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < EP_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 4); }
        fence_barrier_init();
        prefetch_tmap(&map_a); prefetch_tmap(&map_b);
    }
    if (warp == 1) tmem_alloc(&tmem_slot, 512);
    for (int i = threadIdx.x; i < p.H; i += GEMM_THREADS) s_bias[i] = p.bias[i];
    // exclusive prefix sums of the utterances' row-tile counts (block-wide scan, GEMM_THREADS utterances per round)
    {
        int carry = 0;
        for (int b0 = 0; b0 < p.n_utts; b0 += GEMM_THREADS) {
            const int b = b0 + (int)threadIdx.x;
            const int cnt = b < p.n_utts ? (p.enc_len[b] + BM - 1) / BM : 0;
            int incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            if (lane == 31) s_scan[warp] = incl;
            __syncthreads();
            int before = carry;
            for (int w = 0; w < warp; ++w) before += s_scan[w];
            if (b < p.n_utts) s_prefix[b] = before + incl - cnt;
            int total = 0;
            for (int w = 0; w < GEMM_THREADS / 32; ++w) total += s_scan[w];
            carry += total;
            __syncthreads();
        }
        if (threadIdx.x == 0) s_prefix[p.n_utts] = carry;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;

    const int n_col_tiles = (p.H + EP_BN - 1) / EP_BN;
    const int n_tiles = s_prefix[p.n_utts] * n_col_tiles;
    // tile k -> (utterance, row tile inside it, column tile)
    auto locate = [&](int k, int& b, int& j, int& nt) {
        const int mt = k / n_col_tiles;
        nt = k - mt * n_col_tiles;
        int lo = 0, hi = p.n_utts;            // the last b with s_prefix[b] <= mt (utterances without frames have no tile)
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_prefix[mid] <= mt) lo = mid; else hi = mid;
        }
        b = lo;
        j = mt - s_prefix[lo];
    };

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int k = blockIdx.x; k < n_tiles && ok; k += gridDim.x) {
                int b, j, nt;
                locate(k, b, j, nt);
                const int row0 = b * p.T + j * BM;
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % EP_STAGES;
                    if (!mbar_wait(&empty_bar[s], ((it / EP_STAGES) & 1) ^ 1, &abort_flag)) { ok = false; break; }
                    uint8_t* a_dst = smem + (size_t)s * EP_STAGE_BYTES;
                    mbar_expect_tx(&full_bar[s], EP_STAGE_BYTES);
                    tma_load_2d(a_dst, &map_a, kb * BK, row0, &full_bar[s]);
                    tma_load_2d(a_dst + A_STAGE_BYTES, &map_b, kb * BK, nt * EP_BN, &full_bar[s]);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t it = 0, n_acc = 0;
            bool ok = true;
            for (int k = blockIdx.x; k < n_tiles && ok; k += gridDim.x, ++n_acc) {
                const int nt = k % n_col_tiles;
                const int n_cols = min(EP_BN, p.H - nt * EP_BN);            // a multiple of 64
                const uint32_t idesc = idesc_bf16(BM, n_cols);
                const uint32_t a = n_acc & 1u;
                if (!mbar_wait(&acc_empty[a], ((n_acc >> 1) & 1u) ^ 1u, &abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tm_d = tmem_base + a * EP_BN;
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % EP_STAGES;
                    if (!mbar_wait(&full_bar[s], (it / EP_STAGES) & 1, &abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(smem + (size_t)s * EP_STAGE_BYTES);
                    const uint64_t adesc = smem_desc_sw128(a_addr);
                    const uint64_t bdesc = smem_desc_sw128(a_addr + A_STAGE_BYTES);
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk)
                        tc_mma_bf16(tm_d, adesc + (uint64_t)(kk * 2), bdesc + (uint64_t)(kk * 2), idesc, (kb | kk) != 0);
                    tc_commit(&empty_bar[s]);
                }
                if (ok) tc_commit(&acc_full[a]);
            }
        }
    } else {
        const int q = warp & 3;            // tensor-memory lane quadrant this warp may read
        const int row = q * 32 + lane;     // accumulator row of this thread
        uint32_t n_acc = 0;
        for (int k = blockIdx.x; k < n_tiles; k += gridDim.x, ++n_acc) {
            int b, j, nt;
            locate(k, b, j, nt);
            const int n_cols = min(EP_BN, p.H - nt * EP_BN);
            const bool valid = j * BM + row < p.enc_len[b];
            __nv_bfloat16* dst = p.out + ((size_t)b * p.T + (size_t)j * BM + row) * p.H + (size_t)nt * EP_BN;
            const float* bias = s_bias + nt * EP_BN;
            const uint32_t a = n_acc & 1u;
            const bool ready = __all_sync(0xffffffffu, mbar_wait(&acc_full[a], (n_acc >> 1) & 1u, &abort_flag));
            if (!ready) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + a * EP_BN + ((uint32_t)(q * 32) << 16);
            for (int c0 = 0; c0 < n_cols; c0 += 32) {
                float v[32];
                tmem_ld16(taddr + c0, v);
                tmem_ld16(taddr + c0 + 16, v + 16);
                if (valid) {
                    uint32_t w[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) w[i] = pack_bf16x2(v[2 * i] + bias[c0 + 2 * i], v[2 * i + 1] + bias[c0 + 2 * i + 1]);
                    // whole 32-byte sectors per store (a row's segment is 32-byte aligned: H is a multiple of 64)
                    st_global_v8(dst + c0, w);
                    st_global_v8(dst + c0 + 16, w + 8);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[a]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && abort_flag) set_status(p.ctrl, WIND_ERR_TIMEOUT);
}

constexpr size_t enc_proj_smem_bytes() { return (size_t)EP_STAGES * EP_STAGE_BYTES + 1024; }

template <int MODE>
constexpr size_t gemm_smem_bytes() { return (size_t)GemmShape<MODE>::STAGES * (A_STAGE_BYTES + (size_t)GemmShape<MODE>::BN * BK * 2) + 1024; }

// Shared-memory opt-in of the kernels of this file.
static cudaError_t tc_set_attributes() {
    static bool done_on[64] = {};   // the attribute belongs to the (function, device) pair
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_tc_mutex);
    bool& done = done_on[dev];
    if (done) return cudaSuccess;
    if ((e = cudaFuncSetAttribute(gemm_kernel<MODE_ENC_PROJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem_bytes<MODE_ENC_PROJ>())) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(gemm_kernel<MODE_GATE_TABLE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem_bytes<MODE_GATE_TABLE>())) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(enc_proj_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)enc_proj_smem_bytes())) != cudaSuccess) return e;
    done = true;
    return cudaSuccess;
}

cudaError_t tc_enc_proj(const Call& c) {
    const TcMaps& M = *static_cast<const TcMaps*>(c.tc);
    const int n_utts = c.N > 0 ? c.N : c.B;
    if (n_utts <= EP_MAX_UTTS && c.m.H <= EP_MAX_H) {
        EncProjParams q{};
        q.ctrl = c.ctrl();
        q.k_blocks = c.m.D / BK; q.H = c.m.H; q.T = c.T; q.n_utts = n_utts;
        q.enc_len = c.enc_len; q.out = (__nv_bfloat16*)c.enc_proj(); q.bias = c.m.b_enc;
        int sms = 0;
        cudaError_t e = loop_sm_count(&sms);
        if (e != cudaSuccess) return e;
        const long long most = ((long long)n_utts * ((c.T + BM - 1) / BM)) * ((c.m.H + EP_BN - 1) / EP_BN);
        const int grid = (int)(most < sms ? (most < 1 ? 1 : most) : sms);
        enc_proj_kernel<<<grid, GEMM_THREADS, enc_proj_smem_bytes(), c.stream>>>(M.enc, M.w_enc, q);
        return cudaGetLastError();
    }
    GemmParams p{};
    p.ctrl = c.ctrl();
    p.k_blocks = c.m.D / BK;
    p.rows = (long long)(c.N > 0 ? c.N : c.B) * c.T;
    p.N = c.m.H;
    p.enc_len = c.enc_len; p.T = c.T;
    p.out_bf16 = (__nv_bfloat16*)c.enc_proj(); p.bias0 = c.m.b_enc;
    constexpr int BN = GemmShape<MODE_ENC_PROJ>::BN;
    dim3 grid((unsigned)(((c.m.H + BN - 1) / BN) * ((p.rows + BM - 1) / BM)));
    gemm_kernel<MODE_ENC_PROJ><<<grid, GEMM_THREADS, gemm_smem_bytes<MODE_ENC_PROJ>(), c.stream>>>(M.enc, M.w_enc, p);
    return cudaGetLastError();
}

cudaError_t tc_gate_table(const Call& c) {
    const TcMaps& M = *static_cast<const TcMaps*>(c.tc);
    GemmParams p{};
    p.ctrl = c.ctrl();
    p.k_blocks = c.m.E / BK;
    p.rows = (long long)c.m.V + 1;
    p.N = 4 * c.m.P;
    p.out_f32 = c.g0(); p.bias0 = c.b_ih[0]; p.bias1 = c.b_hh[0];
    constexpr int BN = GemmShape<MODE_GATE_TABLE>::BN;
    dim3 grid((unsigned)(((p.N + BN - 1) / BN) * ((p.rows + BM - 1) / BM)));
    gemm_kernel<MODE_GATE_TABLE><<<grid, GEMM_THREADS, gemm_smem_bytes<MODE_GATE_TABLE>(), c.stream>>>(M.emb, M.w_ih0, p);
    return cudaGetLastError();
}

int tc_setup_launches(const Call& c) { (void)c; return 4; }  // init, projection, gate table, loop

}  // namespace wind
