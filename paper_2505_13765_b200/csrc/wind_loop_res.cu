// The decoding loop of the bf16 path, resident-weights mode (sm_100a): ONE persistent cooperative kernel in which
// every weight matrix stays on chip for the whole decode and the CTAs hand results to one another through
// per-group arrival counters and stamped data instead of grid-wide barriers.
//
// One CTA per SM.  A lock step of the batch (Algorithm 2 applied to every utterance at once) is three slots,
// each a tensor-core GEMM with the weights as the stationary operand (M axis) and utterances / window rows on N:
//
//   J  joint      logits^T [128 vocabulary entries, nj window rows] = W_out tile . z^T.  The W_out tile lives in
//                 TENSOR MEMORY (the A operand of tcgen05.mma) for the whole decode.  The CTA builds its own operand
//                 z = act(enc_proj[b, t_b + w, :] + pred_proj[b, :]) in shared memory: the enc_proj rows of the row
//                 group's utterances are copied in (cp.async, 128-byte swizzled K-major layout) as soon as the
//                 control step has published the next frame, pred_proj arrives as stamped (value, stamp) pairs that
//                 the CTA polls, the sum is activated in place.  Epilogue: per-row argmax over the tile's 128
//                 entries by warp shuffles; the winner of every (window row, vocabulary tile) goes, stamped with
//                 the lock step, into its own key slot by a plain store; the logits never leave the chip.
//   L  decoder    gates [4 gates x 16 units, nl utterances] = W_hh tile . h^T, tile resident in shared memory.  The
//                 GEMM needs only the state, so it is issued a slot ahead and its result waits in tensor memory; the
//                 slot itself is: poll the key slots of the CTA's utterances (four lanes per utterance read a
//                 row's slots and take the maximum over the vocabulary tiles themselves), control
//                 step (Algorithm 2's branch: first non-blank row of the window, jump, emission, max-symbols rule),
//                 gate-table rows of the chosen tokens, LSTM cell update, new h (bf16) and c (fp32), one arrival on
//                 the utterance group's counter.  CTAs without a weight tile record the steps (outputs, counters,
//                 next frame, published at once as a stamped word per utterance).  With two layers, layer 1's input
//                 GEMM runs on CTAs holding a W_ih[1] tile after layer 0's arrivals, its recurrent term a slot ahead
//                 on CTAs holding a W_hh[1] tile.
//   P  projection pred_proj [64 H rows, np utterances] = W_pred tile . h_top^T + b_pred after the state counters of
//                 its utterances have filled; written as (bf16 pair, stamp) 8-byte words, which is what the joint
//                 CTAs poll: data and "ready" arrive in one load.
//
// No CTA waits for the whole grid: utterances are independent (Algorithm 2 has no cross-utterance term), so a joint
// CTA waits only for the pred_proj of its row group's utterances, a decoder CTA for the vocabulary tiles of its own
// utterances' rows, a projection CTA for the unit tiles of its own utterance group.  Every wait is bounded (about two
// seconds): a CTA that gives up flags WIND_ERR_TIMEOUT, raises the global abort word, and every CTA leaves at its next
// wait and frees its tensor memory.  Roles per CTA: warp 0 issues TMA, warps 0 and 1 issue tcgen05.mma (half of the K
// blocks each, into separate accumulators that the epilogue adds), warps 2..9 run the epilogues and build the operand.
//
// FULL: teacher forcing with the logits store (wind_eval_joint_window), window-based decoding (which keeps two grid
// barriers around its decision phase) and the timeline records; a plain decode launches the smaller variant.
#include <cuda.h>

#include <mutex>

#include "wind_loop_dev.cuh"

namespace wind {

constexpr int kGroupUtts = 96;   // utterances one joint row group can touch (at most 96 rows, window >= 1)
constexpr int kPrepItems = 3;    // (utterance, 16-byte chunk) items a thread finishes per round of the operand build

// relaxed (L2-coherent) loads: many may be in flight at once, which an acquire load does not allow
__device__ __forceinline__ void ld_relaxed_v2_u64(const unsigned long long* p, unsigned long long& a, unsigned long long& b) {
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "l"(p) : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_v2_u64(unsigned long long* p, unsigned long long a, unsigned long long b) {
    asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(a), "l"(b) : "memory");
}
// two neighbouring pred_proj values as bf16, with the stamp of the slot that wrote them
__device__ __forceinline__ unsigned long long stamped(float lo, float hi, uint32_t stamp) {
    return ((unsigned long long)stamp << 32) | (unsigned long long)pack_bf16x2(lo, hi);
}
template <bool FULL>
__global__ void __launch_bounds__(LOOP_THREADS_RES, 1) loop_res_kernel(const __grid_constant__ LoopMaps M, const LoopParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[2], empty_bar[2], stat_bar;   // [0]: the state box, [1]: the joint's operand
    __shared__ uint64_t acc_full[3], acc_empty[3];             // accumulators: joint, decoder, projection
    __shared__ uint32_t tmem_slot;
    __shared__ int s_abort;      // this CTA has given up (1: a wait of its own ran out, 2: it saw the global abort word)
    __shared__ int s_active;     // utterances still decoding (set in the projection slot)
    __shared__ float win_lpb[FULL ? kMaxWindow : 1], win_sc[FULL ? kMaxWindow : 1];
    __shared__ unsigned long long win_key[FULL ? kMaxWindow : 1];
    __shared__ int s_jt[kGroupUtts], s_jrem[kGroupUtts];       // operand build: frame and frames left of the group's utterances

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    // a length outside [0, T] (found by the init kernel, which ran before this launch): the status is set, no CTA starts
    if (p.ctrl->bad_input) return;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* stat = smem;                       // this CTA's resident weight tile: kb_p blocks of 64 rows x 64 columns
    uint8_t* buf0 = smem + p.buf_off;           // the per-step state box
    float* stage_f = reinterpret_cast<float*>(smem + p.stage_off);   // epilogue staging
    volatile int* vabort = &s_abort;

    if (threadIdx.x == 0) {
        s_abort = 0;
        s_active = 1;
        for (int s = 0; s < 2; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 2);      // two threads issue the MMAs of a GEMM, both commit
        }
        mbar_init(&stat_bar, 1);
        for (int k = 0; k < 3; ++k) {
            mbar_init(&acc_full[k], 2);
            mbar_init(&acc_empty[k], 8);      // one arrival per epilogue warp
        }
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(&tmem_slot, LOOP_TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t tm_j = tmem_base + (uint32_t)p.tm_j, tm_l = tmem_base + (uint32_t)p.tm_l, tm_p = tmem_base + (uint32_t)p.tm_p;

    const int e = threadIdx.x - 64;            // epilogue thread: 0..255 (warps 2..9)
    const int sub = (warp - 2) >> 2;           // which of the two warps of a tensor-memory lane quadrant
    const int q = warp & 3;                    // tensor-memory lane quadrant of this warp
    const int row_in_tile = q * 32 + lane;     // the tensor-memory lane (accumulator row) of this thread
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const bool forced = FULL && p.forced;

    // ----- roles -----
    // joint: the CTA keeps ONE vocabulary tile (cta % vt_count) and takes the row groups j_first, j_first + rg_stride, ...
    // (one per wave); CTAs beyond vt_count * rg_stride have none
    const int j_first = cta < p.vt_count * p.rg_stride ? cta / p.vt_count : p.rg_count;
    const bool has_j = j_first < p.rg_count;
    const int my_vt = cta % p.vt_count;
    // CTAs [0, l_items) keep a W_hh tile (4 gates x 16 units) of layer 0; with two layers the next two sets keep a
    // W_ih[1] tile ("x1") and a W_hh[1] tile ("h1"); the last p_items CTAs keep a W_pred tile (64 rows); CTAs
    // [w_first, w_first + w_count) record the steps
    const int r_role = cta / p.l_items;
    const int r_idx = cta - r_role * p.l_items;
    const bool res_l = cta < p.l_items;
    const bool res_x1 = p.L == 2 && r_role == 1;
    const bool res_h1 = p.L == 2 && r_role == 2;
    const bool res_p = !res_l && !res_x1 && !res_h1 && G - 1 - cta < p.p_items;
    const bool res_w = cta >= p.w_first && cta < p.w_first + p.w_count;
    const int r_ut = r_idx % p.ut_count, r_ql = r_idx / p.ut_count;                  // unit tile / utterance group of an L CTA
    const int r_ht = (G - 1 - cta) % p.ht_count, r_qp = (G - 1 - cta) / p.ht_count;  // H tile / utterance group of a P CTA
    constexpr uint32_t RES_A_BYTES = 64 * BK * 2;
    uint8_t* zbuf = smem + (res_p ? p.z_off_p : p.z_off);     // the joint's operand: kb_h blocks of nj rows x 64 columns
    const bool z_sh = zbuf == buf0 && (res_l || res_x1 || res_h1 || res_p);   // it shares the state box's memory

    if (threadIdx.x == 0 && (res_l || res_x1 || res_h1 || res_p)) {
        mbar_expect_tx(&stat_bar, (uint32_t)p.kb_p * RES_A_BYTES);
        for (int kb = 0; kb < p.kb_p; ++kb) {
            uint8_t* dst = stat + (size_t)kb * RES_A_BYTES;
            if (!res_p) {
                const CUtensorMap* wm = res_l ? &M.w_hh_r : (res_x1 ? &M.w_ih1_r : &M.w_hh1_r);
                for (int g = 0; g < 4; ++g) tma_load_2d(dst + g * 16 * 128, wm, kb * BK, g * p.P + r_ut * 16, &stat_bar);
            } else {
                tma_load_2d(dst, &M.w_pred_r, kb * BK, r_ht * 64, &stat_bar);
            }
        }
    }
    if (warp >= 2 && has_j) {
        // tensor memory, lane = vocabulary entry, 32-bit column j = W_out[v, 2j], W_out[v, 2j + 1]
        const int v = my_vt * 128 + row_in_tile;
        const uint4* src = reinterpret_cast<const uint4*>(p.w_out + (size_t)(v < p.NV ? v : 0) * p.H);
        for (int c0 = 0; c0 < p.H / 2; c0 += 16) {
            uint32_t r[16];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 x = v < p.NV ? src[c0 / 4 + j] : make_uint4(0, 0, 0, 0);
                r[4 * j] = x.x; r[4 * j + 1] = x.y; r[4 * j + 2] = x.z; r[4 * j + 3] = x.w;
            }
            tmem_st16(tmem_base + lane_off + (uint32_t)c0, r);
        }
        tmem_st_wait();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    // ----- arrival counters (global, zeroed per call) -----
    uint32_t* f_keys = p.flags;                  // [rg_count]  vocabulary tiles that have left their keys for a row group
    uint32_t* f_h0 = f_keys + p.rg_count;        // [ql_count]  layer-0 state of an utterance group written (+ its steps recorded)
    uint32_t* f_h1 = f_h0 + p.ql_count;          // [ql_count]  layer-1 state written (two layers)
    uint32_t* f_dh = f_h1 + p.ql_count;          // [ql_count]  layer 1's recurrent term written (two layers)
    // arrivals per decoder-update slot on group ql's layer-0 counter: its unit tiles, plus (when separate CTAs record
    // the steps) one per recording CTA (64 utterances) that overlaps the group.  Under teacher forcing nothing is recorded
    // and the recording CTAs stay out: a counter that sums arrivals over slots is only sound while no participant
    // can run ahead of the others, and a CTA with nothing to wait for could.
    auto arr_h0 = [&](int ql) -> uint32_t {
        uint32_t a = (uint32_t)p.ut_count;
        const int lo = ql * p.nl, hi = min(lo + p.nl, p.B);
        if (p.w_count > 0 && !forced && hi > lo) a += (uint32_t)((hi - 1) / 64 - lo / 64 + 1);
        return a;
    };
    // a wait of this CTA ran out: note which one (the first in the grid stays), flag the CTA and everybody else
    auto give_up = [&](int site) {
        if (atomicCAS(&p.ctrl->timeout_site, 0, site) == 0) p.ctrl->timeout_cta = cta;
        *vabort = 1;
        atomicExch(&p.ctrl->abort, 1);
    };
    // bounded mbarrier wait that notes its site when it is the one that runs out
    auto mwait = [&](uint64_t* bar, uint32_t parity, int site) -> bool {
        const int before = *vabort;
        const bool ok = mbar_wait(bar, parity, vabort);
        if (!ok && before == 0 && *vabort == 1) give_up(site);
        return ok;
    };
    // one thread waits until a counter has reached its target; false when the kernel is being abandoned
    auto flag_wait = [&](const uint32_t* ptr, uint32_t target, int site) -> bool {
        unsigned long long t0 = 0;
        for (uint32_t it = 1;; ++it) {
            if ((int32_t)(ld_acquire_u32(ptr) - target) >= 0) return true;
            if ((it & 63u) == 0u) {
                if (*vabort) return false;
                if (ld_volatile_i32(&p.ctrl->abort)) { *vabort = 2; return false; }
                const unsigned long long now = globaltimer_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > kWaitLimitNs) { give_up(site); return false; }
            }
        }
    };
    // a whole warp waits for counters base[first .. first + count): lane i polls counter i (, i + 32, ...)
    auto warp_flag_wait = [&](const uint32_t* base, int first, int count, uint32_t target, int site) -> bool {
        bool ok = true;
        for (int i0 = 0; i0 < count && ok; i0 += 32) {
            const int i = i0 + lane;
            bool mine = i >= count;
            unsigned long long t0 = 0;
            for (uint32_t it = 1;; ++it) {
                if (!mine) mine = (int32_t)(ld_acquire_u32(base + first + i) - target) >= 0;
                if (__all_sync(0xffffffffu, mine)) break;
                if ((it & 63u) == 0u) {
                    bool quit = *vabort != 0;
                    if (!quit && ld_volatile_i32(&p.ctrl->abort)) { *vabort = 2; quit = true; }
                    const unsigned long long now = globaltimer_ns();
                    if (t0 == 0) t0 = now;
                    else if (!quit && now - t0 > kWaitLimitNs) { give_up(site); quit = true; }
                    if (__any_sync(0xffffffffu, quit)) { ok = false; break; }
                }
            }
        }
        __syncwarp();
        return ok;
    };

    // ----- per-thread pipeline state (every thread keeps the same counts) -----
    uint32_t acc_n[3] = {0u, 0u, 0u}; // uses of each accumulator so far (issuing threads and epilogue threads count alike)
    uint32_t use0 = 0, use1 = 0;      // uses of the state box and of the joint's operand buffer so far
    uint32_t n_l = 0, n_p = 0, n_j = 0;   // decoder-update / projection / joint slots completed
    int step = -1;                    // -1: start of sequence
    int pin = 0;                      // hb[pin] holds the current decoder state
    bool prepped = false;             // the copies of the next joint operand are already under way
    long long clk_last = 0, cyc[3] = {0, 0, 0};
    unsigned long long ns0 = 0;
    if (cta == 0 && e == 0) { clk_last = clock64(); ns0 = globaltimer_ns(); }
    int exit_status = 0;
    int tr_n = 0;                     // trace events written by this thread
    uint32_t epoch = 0;               // grid barrier target (window-based decoding only)

    auto mark = [&](int kind, int id) {
        if constexpr (FULL) trace_mark(p, step, kind, id);
    };
    // this thread has finished its CTA's part of a slot: CTA 0 attributes the time, the timeline notes every CTA
    auto slot_done = [&](int kind) {
        if (cta == 0) {
            const long long now = clock64();
            cyc[kind] += now - clk_last;
            clk_last = now;
        }
        if constexpr (FULL) trace_phase_done(p, step, kind);
    };

    // Grid barrier for all threads of all CTAs (window-based decoding: its decision phase needs every vocabulary
    // tile's statistics of every row); false when the kernel is being abandoned.
    auto grid_sync = [&]() -> bool {
        __syncthreads();
        if (threadIdx.x == 0) {
            epoch += (uint32_t)G;
            if (*vabort) {
                atomicExch(&p.ctrl->abort, 1);
            } else {
                __threadfence();
                atomicAdd(&p.ctrl->bar, 1u);
                flag_wait(&p.ctrl->bar, epoch, 1);
            }
        }
        __syncthreads();
        return *vabort == 0;
    };

    // ----- one issuing thread's share of a GEMM: K blocks [kb_lo, kb_hi) into the accumulator at tm_d -----
    // Two threads call this for every GEMM (warp 1 and warp 0), with disjoint K ranges and separate accumulator
    // copies that the epilogue adds; an empty range only takes part in the commits.  sidx / use: which operand
    // buffer, and how often it has been used before.
    auto mma_part = [&](int k_acc, uint32_t tm_d, int n_tile, int kb_lo, int kb_hi, bool a_tmem, int sidx, uint32_t use,
                        const uint8_t* b_smem) -> bool {
        const uint32_t idesc = idesc_bf16(a_tmem ? 128 : 64, n_tile);
        if (!a_tmem && !mwait(&stat_bar, 0, 10)) return false;
        if (!mwait(&acc_empty[k_acc], (acc_n[k_acc] & 1u) ^ 1u, 11 + k_acc)) return false;   // the epilogue has drained it
        tc_fence_after();
        if (!mwait(&full_bar[sidx], use & 1u, 14 + sidx)) return false;
        tc_fence_after();
        const uint32_t b_addr = smem_u32(b_smem);
        const uint32_t b_block = (uint32_t)n_tile * BK * 2;
        for (int kb = kb_lo; kb < kb_hi; ++kb) {
            const uint64_t bdesc = smem_desc_sw128(b_addr + (uint32_t)kb * b_block);
            if (a_tmem) {
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)
                    tc_mma_bf16_ts(tm_d, tmem_base + (uint32_t)(kb * (BK / 2) + k * 8), bdesc + (uint64_t)(k * 2), idesc,
                                   kb != kb_lo || k != 0);
            } else {
                const uint64_t adesc = smem_desc_sw128(smem_u32(stat + (size_t)kb * RES_A_BYTES));
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)
                    tc_mma_bf16(tm_d, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, kb != kb_lo || k != 0);
            }
        }
        tc_commit(&empty_bar[sidx]);
        tc_commit(&acc_full[k_acc]);
        ++acc_n[k_acc];
        return true;
    };
    // the state box of this step: ONE three-dimensional TMA box (64 columns, rows, all K blocks), once the MMAs
    // that read the buffer last have completed
    auto produce_box = [&](const CUtensorMap* map, int row0, uint32_t bytes) -> bool {
        if (use0 > 0 && !mwait(&empty_bar[0], (use0 - 1) & 1u, 16)) return false;
        if (z_sh && use1 > 0 && !mwait(&empty_bar[1], (use1 - 1) & 1u, 17)) return false;
        mbar_expect_tx(&full_bar[0], bytes);
        tma_load_3d(buf0, map, 0, row0, 0, &full_bar[0]);
        return true;
    };

    // =========================================================================================
    // decoder-update slot of an L CTA: units [r_ut*16, +16), utterances [r_ql*nl, +nl), 64 utterances per pass.
    // Warp (q, sub) of the epilogue owns gate q and the pass's utterances [32 sub, 32 sub + 32).  All global reads of a
    // pass are requested together: first everything the control step needs, then the gate-table rows of the chosen
    // tokens.  Lanes 16..31 hold no accumulator row (64-row tile); they take the second 16 utterances.
    // ctl_only: the CTA is one of the step-recording CTAs: it takes the control step of 64 utterances, records it
    // (outputs, counters, next frame) and has no cell update; the L CTAs then record nothing.
    // =========================================================================================
    constexpr unsigned long long kStampMask = 0xFFFull << 20;   // bits of a key slot that hold the joint slot's stamp
    const int vt_pad = (p.vt_count + 1) & ~1;   // key slots of a window row: one per vocabulary tile, padded to 16 bytes
    // The (logit, label) keys of window rows wr and wr + 1 of utterance b (rows < n only): per row the maximum over the
    // vocabulary tiles' slots, each of which must carry this step's stamp (the whole warp polls until all do).  Result
    // per row: high word = orderable logit (0: nothing there), low 20 bits = 0xFFFFF - label.
    auto fetch_keys2 = [&](int b, int wr, int n, bool live, unsigned long long& k0, unsigned long long& k1) -> bool {
        const uint32_t want = n_j & 0xFFFu;
        const bool in0 = live && wr < n, in1 = live && wr + 1 < n;
        const int r0 = b * p.W + wr, r1 = r0 + 1;
        const unsigned long long* s0 = p.kslot + (size_t)(in0 ? r0 : 0) * vt_pad;   // rows lie one after the other: (row group, row in it)
        const unsigned long long* s1 = p.kslot + (size_t)(in1 ? r1 : 0) * vt_pad;
        unsigned long long t0 = 0;
        for (uint32_t it = 1;; ++it) {
            bool ok = true;
            k0 = 0ull; k1 = 0ull;
            for (int v0 = 0; v0 < vt_pad; v0 += 10) {
                unsigned long long x[10], y[10];
#pragma unroll
                for (int j = 0; j < 5; ++j) {
                    x[2 * j] = x[2 * j + 1] = y[2 * j] = y[2 * j + 1] = 0ull;
                    if (in0 && v0 + 2 * j < vt_pad) ld_relaxed_v2_u64(s0 + v0 + 2 * j, x[2 * j], x[2 * j + 1]);
                    if (in1 && v0 + 2 * j < vt_pad) ld_relaxed_v2_u64(s1 + v0 + 2 * j, y[2 * j], y[2 * j + 1]);
                }
#pragma unroll
                for (int j = 0; j < 10; ++j) {
                    if (v0 + j < p.vt_count) {
                        if (in0) {
                            ok = ok && (uint32_t)((x[j] & kStampMask) >> 20) == want;
                            const unsigned long long key = x[j] & ~kStampMask;
                            k0 = key > k0 ? key : k0;
                        }
                        if (in1) {
                            ok = ok && (uint32_t)((y[j] & kStampMask) >> 20) == want;
                            const unsigned long long key = y[j] & ~kStampMask;
                            k1 = key > k1 ? key : k1;
                        }
                    }
                }
            }
            if (__all_sync(0xffffffffu, ok)) return true;
            if ((it & 15u) == 0u) {
                bool quit = *vabort != 0;
                if (!quit && ld_volatile_i32(&p.ctrl->abort)) { *vabort = 2; quit = true; }
                const unsigned long long now = globaltimer_ns();
                if (t0 == 0) t0 = now;
                else if (!quit && now - t0 > kWaitLimitNs) { give_up(43); quit = true; }
                if (__any_sync(0xffffffffu, quit)) return false;
            }
        }
    };
    auto epilogue_res_L = [&](const int layer, const bool ctl_only) -> bool {
        const int32_t* t_cur = p.t2 + (size_t)(step & 1) * p.B;
        int32_t* t_nxt = p.t2 + (size_t)((step + 1) & 1) * p.B;
        const unsigned long long* keys_cur = p.keys2 + (size_t)(step & 1) * p.rows_pad;
        unsigned long long* keys_nxt = p.keys2 + (size_t)((step + 1) & 1) * p.rows_pad;
        const int u16 = lane & 15, half = lane >> 4;
        const int unit = r_ut * 16 + u16;        // this thread's hidden unit; its gate is q
        // Control step: four neighbouring lanes per utterance (eight utterances per warp, 64 per pass over the eight
        // epilogue warps); lane kq of a group looks at window rows 2 kq and 2 kq + 1 (+ 8 per round), the group's first
        // lane decides and, where this CTA records the steps, records.  Without recording CTAs, one CTA per utterance
        // group (unit tile 0) records.
        const int kq = lane & 3;
        const int ju = 8 * (warp - 2) + (lane >> 2);     // the group's utterance of the pass
        const bool head = kq == 0;
        const bool writer = head && (ctl_only ? true : (p.w_count == 0 && layer == 0 && r_ut == 0));
        const bool mark_here = e == 0;
        const int n_here = ctl_only ? 64 : p.nl;
        const int base = ctl_only ? (cta - p.w_first) * 64 : r_ql * p.nl;
        const bool decode = step >= 0 && !forced && layer == 0;
        const bool from_slots = !(FULL && p.window);   // window-based decoding leaves its decision in the key arrays
        float* cst = p.c_state + (size_t)layer * p.B * p.P + unit;
        const __nv_bfloat16* hin = p.hb + ((size_t)(pin * p.L + layer) * p.Bpad) * p.P + unit;
        __nv_bfloat16* hout = p.hb + ((size_t)((pin ^ 1) * p.L + layer) * p.Bpad) * p.P + unit;
        const float bias1 = layer == 0 ? 0.f : p.b_ih[1][q * p.P + unit] + p.b_hh[1][q * p.P + unit];
        const float* g0u = p.g0 + (size_t)q * p.P + unit;
        const uint32_t g0_stride = 4u * (uint32_t)p.P;
        int* tok_s = reinterpret_cast<int*>(stage_f + 4 * 64 * 16);   // tokens of the pass's 64 utterances
        bool ready = true;
        // ---- what this slot waits for from other CTAs ----
        if (forced && p.L == 2 && layer == 0 && n_l >= 2u) {
            // Teacher forcing feeds tokens without waiting for keys, so nothing else holds layer 0 back: before this
            // slot overwrites the state buffer it wrote two slots ago, layer 1's CTAs must have read it (their arrivals
            // of the slot before last).  While decoding, the wait for the keys implies this.
            bool ok = true;
            if (lane == 0) ok = flag_wait(f_h1 + r_ql, (n_l - 1u) * (uint32_t)p.ut_count, 21);
            ready = __all_sync(0xffffffffu, ok);
        } else if (layer > 0) {
            // layer 1: the step's tokens (recorded with layer 0's arrivals) and the recurrent term computed a slot ahead
            bool ok = true;
            if (lane == 0) ok = flag_wait(f_h0 + r_ql, n_l * arr_h0(r_ql), 22) && flag_wait(f_dh + r_ql, n_l * (uint32_t)p.ut_count, 23);
            ready = __all_sync(0xffffffffu, ok);
        }
        for (int c0 = 0; c0 < n_here; c0 += 64) {
            const int b0 = base + c0;
            const int jl = 32 * sub + lane;      // the utterance of the pass whose token this lane hands to the gate-table reads
            // old cell state of the four (utterance, unit) pairs this thread finishes
            float cold[4];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int j = half + 2 * q + 8 * sub + 16 * jj;     // 0..63 over the CTA's 256 epilogue threads
                cold[jj] = (!ctl_only && c0 + j < p.nl && b0 + j < p.B) ? cst[(size_t)(b0 + j) * p.P] : 0.f;
            }
            {
                // ---- the token utterance b feeds to its decoder in this step (-1: none) ----
                const int b = b0 + ju;
                const bool in = c0 + ju < n_here && b < p.B;
                int tok = -1, t_out = 0;
                if (step < 0) {
                    tok = in ? p.blank : -1;
                } else if (forced) {
                    if (in) {
                        tok = step < p.prefix_len[b] ? p.prefix[(size_t)b * p.U + step] : -1;
                        if (tok >= p.NV || tok < -1) { tok = p.blank; set_status(p.ctrl, WIND_ERR_INVALID_ARG); }   // caller's mistake
                    }
                } else if (layer > 0) {
                    if (in) tok = __ldcg(p.emit_tok + b);     // decided by layer 0's CTAs one slot earlier
                } else {
                    int t = 0, len = 0, cnt = 0, pos = 0;
                    if (in) {
                        t = __ldcg(t_cur + b);
                        len = p.enc_len[b];
                        if (writer) { cnt = __ldcg(p.count + b); pos = __ldcg(p.out_len + b); }
                    }
                    if (c0 == 0 && from_slots) {
                        // A hint only (relaxed counters, no ordering; behind the loads above, so that their latency is
                        // hidden): every vocabulary tile of the row groups of this CTA's utterances has put out its
                        // keys.  The keys themselves are checked by their stamps.
                        const int b_hi = min(base + n_here, p.B);
                        if (b_hi > base) {
                            const int rg_lo = base * p.W / p.nj, rg_hi = (b_hi * p.W - 1) / p.nj;
                            ready = warp_flag_wait(f_keys, rg_lo, rg_hi - rg_lo + 1, n_j * (uint32_t)(p.vt_count * ((p.nj + 31) / 32)) + (uint32_t)p.extra_arrivals, 20);
                        }
                        if (mark_here) mark(TR_L, MK_L_KEYS);
                    }
                    const bool live = in && t < len;
                    const int n = live ? min(p.W, len - t) : 0;
                    // control step (Algorithm 2's branch): first non-blank row of the window, eight rows per round
                    int first = -1, label = p.blank;
                    bool bad = false;
                    const int n_max = __reduce_max_sync(0xffffffffu, n);
                    for (int w0 = 0; w0 < n_max; w0 += 8) {
                        const bool more = live && w0 < n && first < 0;     // the same in the four lanes of a group
                        if (!__any_sync(0xffffffffu, more)) break;
                        const int wr = w0 + 2 * kq;
                        unsigned long long kk[2] = {0ull, 0ull};
                        if (from_slots) {
                            if (!fetch_keys2(in ? b : 0, wr, n, more, kk[0], kk[1])) ready = false;
                        } else {
#pragma unroll
                            for (int j = 0; j < 2; ++j) {
                                if (more && wr + j < n) {
                                    const unsigned long long k = __ldcg(keys_cur + (size_t)b * p.W + wr + j);
                                    if (k != 0ull) kk[j] = (k & 0xFFFFFFFF00000000ull) | (unsigned long long)(0xFFFFFu - key_label(k));
                                }
                            }
                        }
                        // this lane's two rows: the first non-blank one (row and label in one word) and the first broken one
                        uint32_t fn = 0x7FFFFFFFu, fb = 0x7FFFFFFFu;
#pragma unroll
                        for (int j = 1; j >= 0; --j) {
                            const uint32_t lab = 0xFFFFFu - (uint32_t)(kk[j] & 0xFFFFFull);
                            const bool inside = more && wr + j < n;
                            const bool brk = (kk[j] >> 32) == 0ull || lab >= (uint32_t)p.NV;
                            if (inside && brk) fb = (uint32_t)(wr + j) << 20;
                            if (inside && !brk && (int)lab != p.blank) fn = ((uint32_t)(wr + j) << 20) | lab;
                        }
#pragma unroll
                        for (int o = 1; o <= 2; o <<= 1) {
                            fn = min(fn, __shfl_xor_sync(0xffffffffu, fn, o));
                            fb = min(fb, __shfl_xor_sync(0xffffffffu, fb, o));
                        }
                        if (more) {
                            if (fn != 0x7FFFFFFFu) { first = (int)(fn >> 20); label = (int)(fn & 0xFFFFFu); }
                            bad = bad || (fb >> 20) < (fn >> 20);     // rows after the first non-blank one are not looked at
                        }
                    }
                    if (live) {
                        if (first >= 0) tok = label;
                        if (writer) {
                            int jump, forced_adv = 0, emitted = 0;
                            if (first < 0) {
                                jump = n;
                                t += n;
                                cnt = 0;
                            } else {
                                jump = first;
                                if (first > 0) cnt = 0;
                                t += first;
                                if (pos < p.max_out) {
                                    p.out_tokens[(size_t)b * p.max_out + pos] = label;
                                    p.out_frames[(size_t)b * p.max_out + pos] = t;
                                    p.out_len[b] = pos + 1;
                                    emitted = 1;
                                    cnt += 1;
                                    if (cnt == p.S) { t += 1; cnt = 0; forced_adv = 1; }
                                } else {
                                    set_status(p.ctrl, WIND_ERR_OUTPUT_OVERFLOW);  // this utterance stops here
                                    t = len;
                                    tok = -1;
                                }
                            }
                            if (bad && ready) set_status(p.ctrl, WIND_ERR_INTERNAL);
                            t_nxt[b] = t;
                            t_out = t;
                            p.count[b] = cnt;
                            if (!from_slots)
                                for (int w = 0; w < p.W; ++w) keys_nxt[(size_t)b * p.W + w] = 0ull;
                            atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->jump_hist[jump < 64 ? jump : 64]), 1ull);
                            atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->joint_rows), (unsigned long long)n);
                            if (emitted) atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->tokens), 1ull);
                            if (forced_adv) atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->forced), 1ull);
                        }
                    } else if (in && writer) {
                        t_nxt[b] = t;
                        t_out = t;
                    }
                }
                if (in && writer) {
                    if (p.L > 1 && decode) p.emit_tok[b] = tok;   // the upper layer's CTAs read it in their slot
                    // the next frame goes out at once, stamped with the slot, for the CTAs that build the next window's
                    // operand and for everybody's count of the utterances still decoding (readers need nothing but this
                    // word; the frame and counter arrays are only read a whole step later)
                    if (!forced) asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p.t_pub + b), "l"(((unsigned long long)(n_l + 1u) << 32) | (uint32_t)t_out) : "memory");
                }
                if (!ctl_only && head) tok_s[ju] = tok;
                if (mark_here) mark(TR_L, MK_L_TOK);
            }
            if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_TOK);
            if (ctl_only) continue;
            asm volatile("bar.sync 1, 256;" ::: "memory");     // the tokens of the pass
            const int tok = tok_s[jl];
            // ---- gate-table entries (this thread's gate and unit) of the tokens of this lane half's 16 utterances ----
            float add[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const int ta = __shfl_sync(0xffffffffu, tok, j), tb = __shfl_sync(0xffffffffu, tok, 16 + j);
                const int tj = half ? tb : ta;
                if (layer == 0) {
                    add[j] = tj >= 0 ? g0u[(uint32_t)tj * g0_stride] : 0.f;
                } else {
                    // layer 1: the recurrent term W_hh h computed a slot ahead by the h1 CTAs, plus the biases
                    const int bj2 = b0 + 32 * sub + 16 * half + j;
                    add[j] = (tj >= 0 && bj2 < p.B) ? __ldcg(p.dh + (size_t)bj2 * g0_stride + (size_t)q * p.P + unit) + bias1 : 0.f;
                }
            }
            if (c0 == 0) {
                const bool acc_ok = __all_sync(0xffffffffu, mwait(&acc_full[1], acc_n[1] & 1u, 30));
                ready = ready && acc_ok;
                tc_fence_after();
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_ACC);
                if (e == 0) mark(TR_L, MK_L_ACC);
            }
            if (ready) {
                // lanes 0..15 read their row's 32 columns; columns 16..31 then move to lanes 16..31
                float x[16], hi[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) { x[j] = 0.f; hi[j] = 0.f; }
                const int col = c0 + 32 * sub;
                if (col < p.nl) tmem_ld16(tm_l + lane_off + (uint32_t)col, x);
                if (col + 16 < p.nl) tmem_ld16(tm_l + lane_off + (uint32_t)(col + 16), hi);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float v = __shfl_sync(0xffffffffu, hi[j], u16);
                    if (half) x[j] = v;
                }
                // warp q holds gate q: tanh for the cell candidate (q == 2), logistic for the other three,
                // written as 0.5 tanh(x / 2) + 0.5 so that both are one hardware tanh
                const float sc = q == 2 ? 1.f : 0.5f, of = q == 2 ? 0.f : 0.5f;
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    stage_f[(q * 64 + 32 * sub + 16 * half + j) * 16 + u16] = fmaf(tanh_fast((x[j] + add[j]) * sc), sc, of);
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (ready) {
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int j = half + 2 * q + 8 * sub + 16 * jj;     // 0..63
                    const int bj = b0 + j;
                    if (c0 + j < p.nl && bj < p.B) {
                        if (tok_s[j] >= 0) {
                            const float gi = stage_f[(0 * 64 + j) * 16 + u16], gf = stage_f[(1 * 64 + j) * 16 + u16];
                            const float gg = stage_f[(2 * 64 + j) * 16 + u16], go = stage_f[(3 * 64 + j) * 16 + u16];
                            const float cc = gf * cold[jj] + gi * gg;
                            cst[(size_t)bj * p.P] = cc;
                            hout[(size_t)bj * p.P] = __float2bfloat16_rn(go * tanh_fast(cc));
                        } else {
                            hout[(size_t)bj * p.P] = hin[(size_t)bj * p.P];
                        }
                    }
                }
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
        }
        if (ctl_only) {
            // this CTA's 64 utterances are recorded: one arrival on every utterance group they belong to
            asm volatile("bar.sync 1, 256;" ::: "memory");
            const int lo = base, hi = min(lo + 64, p.B);
            if (e == 0 && hi > lo)
                for (int g = lo / p.nl; g <= (hi - 1) / p.nl; ++g) red_release_add(f_h0 + g, 1u);
            return true;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[1]);
        ++acc_n[1];
        // the new state is complete for this CTA's units: visible to TMA reads, then one arrival for the group
        fence_proxy_async_all();
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (e == 0) red_release_add((layer == 0 ? f_h0 : f_h1) + r_ql, 1u);
        if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_EPI_DONE);
        return ready;
    };

    // b_pred of this thread's accumulator row: constant for the whole decode, read once
    const float p_bias = (res_p && e >= 0) ? p.b_pred[r_ht * 64 + 16 * q + (lane & 15)] : 0.f;
    // projection epilogue of a P CTA: pred_proj rows [r_ht*64, +64) of utterances [r_qp*np, +np), published as
    // (value, stamp) pairs: a reader that finds the stamp of this slot has the value
    auto epilogue_res_P = [&](uint32_t stamp) -> bool {
        const int h0 = r_ht * 64;
        if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_TOK);
        const bool ready = __all_sync(0xffffffffu, mwait(&acc_full[2], acc_n[2] & 1u, 31));
        tc_fence_after();
        if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_ACC);
        if (e == 0) mark(TR_P, MK_P_ACC);
        if (ready) {
            const int hl = 16 * q + (lane & 15);
            for (int c0 = 16 * sub; c0 < p.np; c0 += 32) {
                float g[16], more[16];
                tmem_ld16(tm_p + lane_off + (uint32_t)c0, g);
                tmem_ld16(tm_p + lane_off + (uint32_t)(p.np + c0), more);   // the other issuing thread's K blocks
                if (p.kb_p < 2) {   // a single K block: the first copy's issuer had an empty range and wrote nothing
#pragma unroll
                    for (int j = 0; j < 16; ++j) g[j] = 0.f;
                }
                if (lane < 16) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) stage_f[(c0 + j) * 68 + hl] = g[j] + more[j] + p_bias;
                }
            }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[2]);
        ++acc_n[2];
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (ready) {
            // thread e: four consecutive H rows of utterances (e >> 4), (e >> 4) + 16, ...: 512 contiguous bytes per
            // utterance and 16 threads.  No fence before the stamped pairs: a reader needs nothing but the pair itself,
            // and what this CTA read of other CTAs' writes for this slot (the state box) had arrived in shared memory
            // before the accumulator could be read, so a later overwrite of the state cannot reach it.
            const int hq = (e & 15) * 4;
            for (int bl = e >> 4; bl < p.np; bl += 16) {
                const int b = r_qp * p.np + bl;
                if (b < p.B) {
                    const float4 v = *reinterpret_cast<const float4*>(stage_f + bl * 68 + hq);
                    unsigned long long* dst = p.pred_pub + ((size_t)b * p.H + h0 + hq) / 2;
                    st_relaxed_v2_u64(dst, stamped(v.x, v.y, stamp), stamped(v.z, v.w, stamp));
                }
            }
        }
        if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_EPI_DONE);
        if (e == 0) mark(TR_P, MK_P_PUB);
        return ready;
    };
    // h1 CTAs: the finished recurrent term of layer 1 goes to global memory (fp32 [B][4P], gate-major like the gate
    // table); the x1 CTAs add it in the next decoder-update slot
    auto store_res_h1 = [&]() {
        const bool ready = __all_sync(0xffffffffu, mwait(&acc_full[1], acc_n[1] & 1u, 32));
        tc_fence_after();
        if (ready) {
            const int unit = r_ut * 16 + (lane & 15);
            for (int c0 = 0; c0 < p.nl; c0 += 64) {
                const int col = c0 + 32 * sub;
                float x[16], hi[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) { x[j] = 0.f; hi[j] = 0.f; }
                if (col < p.nl) tmem_ld16(tm_l + lane_off + (uint32_t)col, x);
                if (col + 16 < p.nl) tmem_ld16(tm_l + lane_off + (uint32_t)(col + 16), hi);
                if (lane < 16) {
                    float* dst = p.dh + (size_t)q * p.P + unit;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int ba = r_ql * p.nl + col + j, bb = ba + 16;
                        if (col + j < p.nl && ba < p.B) dst[(size_t)ba * 4 * p.P] = x[j];
                        if (col + 16 + j < p.nl && bb < p.B) dst[(size_t)bb * 4 * p.P] = hi[j];
                    }
                }
            }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[1]);
        ++acc_n[1];
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (e == 0) red_release_add(f_dh + r_ql, 1u);
    };
    // GEMMs that need only the state, issued ahead of the decoder-update slot that uses them: layer 0's (its result
    // waits in tensor memory for the next control step) and, with two layers, layer 1's recurrent term (stored by
    // store_res_h1).  While decoding they are issued right behind the joint's MMAs: the state box then takes over the
    // operand buffer the joint has just read, and the buffer is free for the next window's rows as soon as the
    // decoder-update slot is over (the box and the joint's operand share memory in these CTAs).
    auto early_res = [&]() {
        const bool mine = res_l || res_h1;
        if (warp == 0) {
            if (lane == 0 && mine) {
                // the state of this CTA's utterance group as the last decoder-update slot left it
                const bool ok = res_l ? flag_wait(f_h0 + r_ql, n_l * arr_h0(r_ql), 24) : flag_wait(f_h1 + r_ql, n_l * (uint32_t)p.ut_count, 25);
                mark(TR_P, MK_E_FLAG);
                if (ok) {
                    fence_proxy_async_all();
                    if (produce_box(res_l ? &M.hb_l3[pin] : &M.hb_l3_1[pin], r_ql * p.nl, (uint32_t)p.nl * (uint32_t)p.P * 2u))
                        mma_part(1, tm_l, p.nl, p.kb_p, p.kb_p, false, 0, use0, buf0);   // one accumulator: warp 1 issues all of it
                }
                mark(TR_P, MK_E_ISSUED);
            }
        } else if (warp == 1) {
            if (lane == 0 && mine) mma_part(1, tm_l, p.nl, 0, p.kb_p, false, 0, use0, buf0);
        } else if (res_h1) {
            store_res_h1();
        }
        if (mine) ++use0;
    };

    // =========================================================================================
    // The joint's operand, built by the epilogue warps in the 128-byte swizzled K-major layout the MMA reads:
    // K block kb = 64 columns, nj rows of 128 bytes each, the 16-byte chunk c of row i at chunk position c ^ (i & 7).
    // Work item = (utterance of the row group, chunk of 8 columns); thread e takes items e, e + 256, ...
    // Part A (as soon as the next frames are known): copy the enc_proj chunks of the window rows in, zeros past an
    // utterance's end.  Part B (when pred_proj has arrived): add, activate, convert, in place, by the thread that
    // copied the chunk; then hand the buffer to the issuing threads.
    // =========================================================================================
    const int n_chunks = p.H >> 3;
    auto group_span = [&](int rg, int& u_lo, int& n_utt) {
        const int r_lo = rg * p.nj, r_hi = min(r_lo + p.nj, p.rows);
        u_lo = r_lo / p.W;
        n_utt = r_hi > r_lo ? (r_hi - 1) / p.W - u_lo + 1 : 0;
    };
    // Warp 2, once its CTA's decoder-slot work is over: the frames the recording threads have published for this step,
    // all requested together (relaxed loads).  Gives the count of utterances still decoding (every CTA reads the same
    // words, so all take the same exit) and the frames of the CTA's first row group for the operand copies.
    // A CTA that lags may find a later stamp: the recording threads only go on while utterances are left, so a later
    // stamp means "not finished" (the count itself is then of no interest).
    auto poll_frames = [&](uint32_t want) {
        int u_lo = 0, n_utt = 0;
        if (has_j) group_span(j_first, u_lo, n_utt);
        int alive = 0;
        unsigned long long t0 = 0;
        for (uint32_t it = 1;; ++it) {
            bool all = true;
            alive = 0;
            for (int b = lane; b < p.B; b += 32) {
                const unsigned long long v = ld_relaxed_u64(p.t_pub + b);
                const int32_t ahead = (int32_t)((uint32_t)(v >> 32) - want);
                const int t = (int)(uint32_t)v, len = p.enc_len[b];
                all = all && ahead >= 0;
                alive += (ahead > 0 || t < len) ? 1 : 0;
                if (ahead == 0 && b >= u_lo && b < u_lo + n_utt) {
                    s_jt[b - u_lo] = t < len ? t : 0;
                    s_jrem[b - u_lo] = t < len ? len - t : 0;
                }
            }
            if (__all_sync(0xffffffffu, all)) break;
            if ((it & 15u) == 0u) {
                bool quit = *vabort != 0;
                if (!quit && ld_volatile_i32(&p.ctrl->abort)) { *vabort = 2; quit = true; }
                const unsigned long long now = globaltimer_ns();
                if (t0 == 0) t0 = now;
                else if (!quit && now - t0 > kWaitLimitNs) { give_up(42); quit = true; }
                if (__any_sync(0xffffffffu, quit)) break;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) alive += __shfl_xor_sync(0xffffffffu, alive, o);
        if (lane == 0) s_active = alive;
    };
    // frames_known: s_jt / s_jrem of this row group were filled by poll_frames
    auto prep_A = [&](int rg, uint32_t want, bool frames_known) {
        int u_lo, n_utt;
        group_span(rg, u_lo, n_utt);
        if (!frames_known && e < n_utt) {
            const int b = u_lo + e;
            int t = 0;
            if (forced) {
                t = p.t2[b];
            } else {
                // acquire: what the recording thread wrote before publishing (the cleared keys of the next step
                // among it) is ordered before everything this CTA does with the window
                unsigned long long t0 = 0, v = 0;
                for (uint32_t it = 1;; ++it) {
                    v = ld_acquire_u64(p.t_pub + b);
                    if ((uint32_t)(v >> 32) == want) break;
                    if ((it & 63u) == 0u) {
                        if (*vabort) break;
                        if (ld_volatile_i32(&p.ctrl->abort)) { *vabort = 2; break; }
                        const unsigned long long now = globaltimer_ns();
                        if (t0 == 0) t0 = now;
                        else if (now - t0 > kWaitLimitNs) { give_up(40); break; }
                    }
                }
                t = (int)(uint32_t)v;
            }
            const int len = p.enc_len[b];
            s_jt[e] = t < len ? t : 0;
            s_jrem[e] = t < len ? len - t : 0;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
        // the buffer is free once the MMAs that read it last have completed
        bool ok = use1 == 0 || mwait(&empty_bar[1], (use1 - 1) & 1u, 18);
        if (ok && z_sh && use0 > 0) ok = mwait(&empty_bar[0], (use0 - 1) & 1u, 19);
        if (ok && *vabort == 0) {
            for (int idx = e; idx < n_utt * n_chunks; idx += 256) {
                const int ul = idx / n_chunks, c = idx - ul * n_chunks;
                const int b = u_lo + ul, t = s_jt[ul], rem = s_jrem[ul];
                const int w_lo = max(0, rg * p.nj - b * p.W), w_hi = min(p.W, (rg + 1) * p.nj - b * p.W);
                uint8_t* dst_kb = zbuf + (size_t)(c >> 3) * ((size_t)p.nj * 128);
                const __nv_bfloat16* src = p.enc_proj + ((size_t)b * p.T + t) * p.H + c * 8;
                for (int w = w_lo; w < w_hi; ++w) {
                    const int i = b * p.W + w - rg * p.nj;
                    uint8_t* dst = dst_kb + i * 128 + (((c & 7) ^ (i & 7)) << 4);
                    if (w < rem) {
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src + (size_t)w * p.H) : "memory");
                    } else {
                        *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
                    }
                }
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        if (e == 0) mark(TR_J, MK_J_COPIES);
    };
    auto prep_B = [&](int rg, uint32_t want) {
        int u_lo, n_utt;
        group_span(rg, u_lo, n_utt);
        const int n_items = n_utt * n_chunks;
        bool waited = false;
        for (int base = e; base < n_items; base += 256 * kPrepItems) {
            uint32_t pv[kPrepItems][4];      // pred_proj of the item's eight columns, as four bf16 pairs
            int it_ul[kPrepItems], it_c[kPrepItems];
#pragma unroll
            for (int k = 0; k < kPrepItems; ++k) {
                const int idx = base + k * 256;
                it_ul[k] = -1; it_c[k] = 0;
                if (idx < n_items) {
                    const int ul = idx / n_chunks;
                    if (s_jrem[ul] > 0) { it_ul[k] = ul; it_c[k] = idx - ul * n_chunks; }   // a finished utterance needs nothing
                }
            }
            // pred_proj of this round's items, all requested together, until every stamp is this slot's; between two
            // such requests one word is polled until it carries the stamp (little traffic while the projection CTAs are
            // still at work).  Relaxed loads: the values travel in the same 8-byte words as the stamps, and nothing else
            // that another CTA writes is read behind them.
            unsigned long long t0 = 0;
            for (uint32_t it = 1;; ++it) {
                bool all = true;
                const unsigned long long* miss = nullptr;
#pragma unroll
                for (int k = 0; k < kPrepItems; ++k) {
                    if (it_ul[k] < 0) continue;
                    const unsigned long long* src = p.pred_pub + ((size_t)(u_lo + it_ul[k]) * p.H + it_c[k] * 8) / 2;
                    unsigned long long x[4];
                    ld_relaxed_v2_u64(src, x[0], x[1]);
                    ld_relaxed_v2_u64(src + 2, x[2], x[3]);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if ((uint32_t)(x[j] >> 32) != want) { all = false; miss = src + j; }
                        pv[k][j] = (uint32_t)x[j];
                    }
                }
                if (all) break;
                bool quit = false;
                for (uint32_t spin = 1; !quit; ++spin) {
                    if ((uint32_t)(ld_relaxed_u64(miss) >> 32) == want) break;
                    if ((spin & 15u) == 0u) {
                        if (*vabort) quit = true;
                        else if (ld_volatile_i32(&p.ctrl->abort)) { *vabort = 2; quit = true; }
                        else {
                            const unsigned long long now = globaltimer_ns();
                            if (t0 == 0) t0 = now;
                            else if (now - t0 > kWaitLimitNs) { give_up(41); quit = true; }
                        }
                    }
                }
                if (quit) break;
            }
            if (e == 0 && !waited) mark(TR_J, MK_J_PRED);
            if (!waited) { asm volatile("cp.async.wait_all;" ::: "memory"); waited = true; }
#pragma unroll
            for (int k = 0; k < kPrepItems; ++k) {
                if (it_ul[k] < 0) continue;
                const int b = u_lo + it_ul[k], c = it_c[k], rem = s_jrem[it_ul[k]];
                const int w_lo = max(0, rg * p.nj - b * p.W), w_hi = min(min(p.W, (rg + 1) * p.nj - b * p.W), rem);
                uint8_t* dst_kb = zbuf + (size_t)(c >> 3) * ((size_t)p.nj * 128);
                for (int w = w_lo; w < w_hi; ++w) {
                    const int i = b * p.W + w - rg * p.nj;
                    uint4* dst = reinterpret_cast<uint4*>(dst_kb + i * 128 + (((c & 7) ^ (i & 7)) << 4));
                    const uint4 ev = *dst;
                    *dst = make_uint4(act_add_bf16x2(ev.x, pv[k][0], p.act), act_add_bf16x2(ev.y, pv[k][1], p.act),
                                      act_add_bf16x2(ev.z, pv[k][2], p.act), act_add_bf16x2(ev.w, pv[k][3], p.act));
                }
            }
        }
        if (!waited) asm volatile("cp.async.wait_all;" ::: "memory");
        fence_proxy_async();      // this thread's shared-memory writes, for the MMAs (async proxy)
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (e == 0) mbar_arrive(&full_bar[1]);
        if (e == 0) mark(TR_J, MK_J_HANDOVER);
    };

    // ----- before the loop: layer 0's GEMM on the initial (zero) state -----
    early_res();

    for (;;) {
        // =====================================================================================
        // decoder-update slot: control step + LSTM cell update (layer 0), then layer 1 on its own CTAs
        // =====================================================================================
        if (warp >= 2) {
            if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_START);
            if (res_l) epilogue_res_L(0, false);
            else if (res_w && !forced) epilogue_res_L(0, true);
            if (cta == 0 && e == 0 && step >= 0 && !forced) p.ctrl->step = step + 1;
            if (e == 0 && p.L != 2) slot_done(TR_L);
        }
        ++n_l;
        if (p.L == 2) {
            // layer 1: W_ih[1] . (new layer-0 state) on the x1 CTAs, then their cell update
            if (warp == 0) {
                if (lane == 0 && res_x1) {
                    if (flag_wait(f_h0 + r_ql, n_l * arr_h0(r_ql), 26)) {
                        fence_proxy_async_all();
                        if (produce_box(&M.hb_l3[pin ^ 1], r_ql * p.nl, (uint32_t)p.nl * (uint32_t)p.P * 2u))
                            mma_part(1, tm_l, p.nl, p.kb_p, p.kb_p, false, 0, use0, buf0);
                    }
                }
            } else if (warp == 1) {
                if (lane == 0 && res_x1) mma_part(1, tm_l, p.nl, 0, p.kb_p, false, 0, use0, buf0);
            } else {
                if (res_x1) epilogue_res_L(1, false);
                if (e == 0) slot_done(TR_L);
            }
            if (res_x1) ++use0;
        }
        // The next window's enc_proj rows can be copied in from here on: the frames are published and this CTA's
        // GEMMs on the state box are over.  (A CTA whose projection box shares the buffer does it behind that GEMM.)
        if (warp == 2 && !forced) poll_frames(n_l);
        if (warp >= 2 && has_j && !forced && !(res_p && z_sh)) { prep_A(j_first, n_l, true); prepped = true; }
        pin ^= 1;
        if (forced && step + 1 < p.U) {
            // teacher forcing: more prefix tokens to feed before the window is evaluated
            early_res();
            ++step;
            continue;
        }

        // =====================================================================================
        // projection slot: pred_proj for every utterance; behind it, layer 0's GEMM of the next step
        // =====================================================================================
        if (warp == 0) {
            if (lane == 0 && res_p) {
                // the top layer's state of this CTA's utterances: every utterance group they belong to has arrived
                const uint32_t* f = p.L == 2 ? f_h1 : f_h0;
                const int b_lo = r_qp * p.np, b_hi = min(b_lo + p.np, p.B);
                bool ok = true;
                if (b_hi > b_lo)
                    for (int g = b_lo / p.nl; ok && g <= (b_hi - 1) / p.nl; ++g)
                        ok = flag_wait(f + g, n_l * (p.L == 2 ? (uint32_t)p.ut_count : arr_h0(g)), 27);
                mark(TR_P, MK_P_FLAG);
                if (ok) {
                    fence_proxy_async_all();
                    if constexpr (FULL) trace_event(p, 0, tr_n, step, TR_P, EV_FIRST_ISSUE);
                    if (produce_box(&M.hb_p3[pin], r_qp * p.np, (uint32_t)p.np * (uint32_t)p.P * 2u))
                        mma_part(2, tm_p + (uint32_t)p.np, p.np, p.kb_p / 2, p.kb_p, false, 0, use0, buf0);
                }
            }
        } else if (warp == 1) {
            if (lane == 0 && res_p) mma_part(2, tm_p, p.np, 0, p.kb_p / 2, false, 0, use0, buf0);
        } else {
            if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_START);
            if (res_p) epilogue_res_P(n_p + 1u);
        }
        if (res_p) ++use0;
        ++n_p;
        if (warp >= 2 && e == 0) slot_done(TR_P);
        // the one CTA-wide meeting point of a step: everybody learns whether the kernel is being abandoned and how
        // many utterances are still decoding
        {
            const int ab = __syncthreads_or(*vabort != 0);
            if (ab) goto done;
        }
        if (!forced && s_active == 0) break;
        if (!forced && step + 1 >= p.step_cap) { exit_status = WIND_ERR_INTERNAL; break; }
        ++step;

        // =====================================================================================
        // joint slot: the CTA's vocabulary tile against the window rows of its row group(s)
        // =====================================================================================
        {
            const int n_tile = p.nj;
            unsigned long long* keys_cur = p.keys2 + (size_t)(step & 1) * p.rows_pad;
            const int32_t* t_cur = p.t2 + (size_t)(step & 1) * p.B;
            for (int rg = j_first; rg < p.rg_count; rg += p.rg_stride) {
                if (warp < 2) {
                    if (lane == 0) {
                        if constexpr (FULL) trace_event(p, warp, tr_n, step, TR_J, EV_FIRST_ISSUE);
                        if (warp == 0) mma_part(0, tm_j + (uint32_t)n_tile, n_tile, p.kb_h / 2, p.kb_h, true, 1, use1, zbuf);
                        else mma_part(0, tm_j, n_tile, 0, p.kb_h / 2, true, 1, use1, zbuf);
                        if constexpr (FULL) trace_event(p, warp, tr_n, step, TR_J, EV_COMMIT);
                    }
                } else {
                    if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_START);
                    if (e == 0) mark(TR_J, MK_J_ENTER);
                    if (!prepped) prep_A(rg, n_l, false);
                    prepped = false;
                    prep_B(rg, n_p);
                    if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_TOK);
                    const bool ready = __all_sync(0xffffffffu, mwait(&acc_full[0], acc_n[0] & 1u, 33));
                    tc_fence_after();
                    if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_ACC);
                    if (e == 0) mark(TR_J, MK_J_ACC);
                    unsigned long long* part = reinterpret_cast<unsigned long long*>(stage_f);   // [4 lane quadrants][n_tile]
                    if (ready) joint_epilogue_item<true, FULL>(p, tm_j, lane_off, lane, q, sub, row_in_tile, rg, my_vt, n_tile, t_cur, keys_cur, part);
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[0]);
                    ++acc_n[0];
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                    if (!forced && !(FULL && p.window)) {
                        // This vocabulary tile's key of every row of the group goes out as ONE stamped word per row (no
                        // atomics, no fence): high word the orderable logit (0: no entry), then the joint slot's stamp,
                        // then 0xFFFFF - label.  Readers take the maximum over the tiles once every stamp is this step's.
                        if (e < n_tile) {
                            unsigned long long m = 0ull;
                            if (ready) {
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    const unsigned long long x = part[k * n_tile + e];
                                    m = x > m ? x : m;
                                }
                            }
                            const unsigned long long stamp_bits = (unsigned long long)((n_j + 1u) & 0xFFFu) << 20;
                            const unsigned long long word =
                                m != 0ull ? ((m & 0xFFFFFFFF00000000ull) | stamp_bits | (unsigned long long)(0xFFFFFu - key_label(m))) : stamp_bits;
                            asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p.kslot + ((size_t)rg * p.nj + e) * vt_pad + my_vt), "l"(word) : "memory");
                        }
                        // a hint for the readers' wait (relaxed: nothing is ordered by it), one per storing warp, behind
                        // the warp's stores
                        __syncwarp();
                        if (lane == 0 && e < n_tile) red_relaxed_add(f_keys + rg, 1u);
                    }
                    if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_EPI_DONE);
                }
                ++use1;
            }
            if (!forced) early_res();     // behind the joint's MMAs: the GEMMs of the next decoder-update slot
            ++n_j;
            if (warp >= 2 && e == 0) slot_done(TR_J);
        }
        if (forced) break;
        if (FULL && p.window) {
            // window-based decoding: one warp per window row turns the joint's per-row statistics into the most
            // probable (label, offset) pair of Eq. (1) and leaves it in the keys in the form the control step reads
            if (!grid_sync()) goto done;
            if (warp >= 2) {
                const int32_t* t_cur = p.t2 + (size_t)(step & 1) * p.B;
                unsigned long long* keys_cur = p.keys2 + (size_t)(step & 1) * p.rows_pad;
                window_decision<8>(p, cta, G, warp - 2, lane, t_cur, keys_cur, win_lpb, win_sc, win_key);
            }
            if (!grid_sync()) goto done;
        }
    }
done:
    asm volatile("cp.async.wait_all;" ::: "memory");
    // an accumulator may still hold an unused early GEMM; nothing reads it, but its MMAs must have completed before
    // the tensor memory goes back (a private flag, so that the wait is not cut short; it stays bounded)
    if (warp == 1 && lane == 0 && acc_n[1] > 0) {
        int gave_up = 0;
        mbar_wait(&acc_full[1], (acc_n[1] - 1u) & 1u, &gave_up);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, LOOP_TMEM_COLS);
    }
    if (threadIdx.x == 0) {
        if (s_abort) atomicExch(&p.ctrl->abort, 1);
        if (s_abort == 1) set_status(p.ctrl, WIND_ERR_TIMEOUT);
    }
    if (cta == 0 && e == 0) {
        if (exit_status) set_status(p.ctrl, exit_status);
        p.ctrl->active = s_active;
        for (int k = 0; k < 3; ++k) p.ctrl->phase_cycles[k] = cyc[k];
        p.ctrl->loop_ns = (long long)(globaltimer_ns() - ns0);
    }
}

// ---------------------------------------------------------------------------
// host side of this kernel: shared-memory opt-in per device, launch
// ---------------------------------------------------------------------------
static std::mutex g_res_mutex;
static int g_res_smem[64] = {};

cudaError_t loop_res_set_smem(int bytes) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_res_mutex);
    if (bytes > g_res_smem[dev]) {
        for (const void* fn : {(const void*)loop_res_kernel<false>, (const void*)loop_res_kernel<true>}) {
            e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
            if (e != cudaSuccess) return e;
        }
        g_res_smem[dev] = bytes;
    }
    return cudaSuccess;
}

cudaError_t loop_res_launch(const LoopMaps& maps, const LoopParams& p, int grid, uint32_t smem_bytes, bool full, cudaStream_t stream) {
    // every array the kernel writes through must be there: a missing one is a host-side mistake, not something to find on the device
    if (!p.ctrl || !p.flags || !p.pred_pub || !p.kslot || !p.t_pub || !p.t2 || !p.hb || !p.c_state || !p.enc_proj || !p.g0 || !p.keys2 ||
        (p.L == 2 && (!p.dh || !p.emit_tok)))
        return cudaErrorInvalidValue;
    void* args[2] = {(void*)&maps, (void*)&p};
    const void* fn = full ? (const void*)loop_res_kernel<true> : (const void*)loop_res_kernel<false>;
    return cudaLaunchCooperativeKernel(fn, dim3((unsigned)grid), dim3(LOOP_THREADS_RES), args, smem_bytes, stream);
}

}  // namespace wind
