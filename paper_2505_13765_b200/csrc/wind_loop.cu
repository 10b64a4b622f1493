// The decoding loop of the bf16 path as ONE persistent cooperative kernel (sm_100a) whose phases are separated by
// grid barriers, and the host side of all loop kernels (tile plan, tensor maps, launch).
//
// One CTA per SM stays resident for the whole decode.  A lock step of the batch
// (Algorithm 2 applied to every utterance at once) is three phases separated by grid
// barriers; every phase is a tensor-core GEMM whose operands arrive by TMA and whose
// accumulator lives in tensor memory:
//
//   J  joint      logits^T [vocab tile 128, window rows N] = W_out tile . z^T, epilogue = per-row
//                 argmax over the tile's 128 vocabulary entries by warp shuffles, combined across
//                 vocabulary tiles with a 64-bit atomicMax on (logit, label) keys.  The logits never
//                 leave the chip.  When every CTA owns exactly one tile, its W_out tile is loaded
//                 once and stays in shared or tensor memory for the whole decode.
//   L  decoder    gates [utterances 128, 4 x units] = h . W_hh^T (+ x . W_ih^T for upper layers);
//                 the epilogue first does the control step for its utterances -- first-non-blank
//                 scan of the window's keys, jump, emission, max-symbols rule (one CTA per
//                 utterance tile writes the results, the others only need the token) -- then the
//                 LSTM cell update.  Layer 0's input term W_ih emb[tok] + b comes from a table
//                 computed once per call, so the embedding costs no GEMM work inside the loop.
//   P  projection pred_proj [utterances 128, H slice] = h_top . W_pred^T + b_pred, epilogue =
//                 z[b, w, slice] = act(enc_proj[b, t_b + w, slice] + pred_proj) for the next window.
//
// Roles per CTA: warp 0 issues TMA, warp 1 issues tcgen05.mma, warps 2..5 run the epilogues
// (one thread per tensor-memory lane).  State that one phase reads while another CTA writes it
// is double-buffered by step parity (t, keys), so a phase never reads what it writes.
//
// Two modes (template parameter RES).  The description above is the streaming mode: weights flow
// through a TMA ring every step.  In the resident-weights mode (one or two LSTM layers, shapes whose
// tiles fit) the W_out tile of a CTA lives in tensor memory and 64-row tiles of W_hh / W_pred (and of
// layer 1's matrices) in the shared memory of disjoint CTA sets for the whole decode; the GEMMs are
// transposed (weights on the M axis, utterances on N), every per-step operand is one TMA box, two
// threads issue the MMAs, eight warps run the epilogues, and CTAs without a weight tile record the
// steps (outputs, counters, next frame).  (wind_loop_res.cu holds a second kernel for the resident-weights
// mode, without grid barriers; the tile planner below chooses between the two.)
//
// Two variants (template parameter FULL): teacher forcing with the logits store (wind_eval_joint_window),
// window-based decoding (the best (label, offset) pair of Eq. (1) decides the step: per-row softmax
// statistics in the joint's epilogue and a decision phase after it) and the timeline records are compiled
// into the FULL variant only; a plain decode launches the smaller one.
//
// Every wait is bounded (mbarrier waits and the grid barrier): a CTA that runs out of patience
// flags WIND_ERR_TIMEOUT, raises the global abort word, and every CTA leaves at its next wait.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <cstdlib>
#include <mutex>

#include "wind_loop_dev.cuh"

namespace wind {

constexpr int LOOP_MAX_STAGES = 28;
constexpr uint32_t LOOP_A_BYTES = 128 * BK * 2;  // one K block of a 128-row operand tile
constexpr int kDataflowMaxBatch = 64;             // largest batch for which the planner picks the barrier-free resident kernel (one LSTM layer)
constexpr int kDataflowMaxBatch2 = 0;             // the same with two LSTM layers (measured at 16 and 32 utterances: grid barriers ahead)

// RES: resident-weights mode (compile-time, so that each instantiation carries only its own code paths: the loop
// body runs once per lock step, straight through, and instruction fetch is a visible cost at that scale).
// FULL: the kernel also carries teacher forcing with the logits store, window-based decoding and the timeline; the
// plain decode runs the variant without them (a smaller instruction footprint: the loop is sensitive to it).
template <bool RES, bool FULL>
__global__ void __launch_bounds__(RES ? LOOP_THREADS_RES : LOOP_THREADS, 1) loop_kernel(const __grid_constant__ LoopMaps M, const LoopParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[LOOP_MAX_STAGES], empty_bar[LOOP_MAX_STAGES], stat_bar;
    __shared__ uint64_t acc_full[3], acc_empty[3];   // accumulators: joint, decoder, projection
    __shared__ uint32_t tmem_slot;
    __shared__ int s_abort;      // this CTA has given up
    __shared__ int s_active;     // utterances still decoding (set in the projection phase)
    // window-based decoding: per row of the window in hand, blank log-probability, best non-blank score and key
    __shared__ float win_lpb[FULL ? kMaxWindow : 1], win_sc[FULL ? kMaxWindow : 1];
    __shared__ unsigned long long win_key[FULL ? kMaxWindow : 1];
    __shared__ int s_red[8];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    // a length outside [0, T] (found by the init kernel, which ran before this launch): the status is set, no CTA starts
    if (p.ctrl->bad_input) return;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* stat = smem;                       // W_out tile kept in shared memory (J_SMEM): kb_h blocks of 128 x 64 bf16
    uint8_t* ring = smem + p.stat_bytes;        // operand stages; geometry differs per phase, drained in between

    if (threadIdx.x == 0) {
        s_abort = 0;
        s_active = 0;
        // resident-weights mode: two threads issue the MMAs of a GEMM (each its half of the K blocks), both commit
        const uint32_t issuers = RES ? 2u : 1u;
        for (int s = 0; s < LOOP_MAX_STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], s == 0 ? issuers : 1u);
        }
        mbar_init(&stat_bar, 1);
        for (int k = 0; k < 3; ++k) {
            mbar_init(&acc_full[k], issuers);
            mbar_init(&acc_empty[k], RES ? 8u : 4u);   // one arrival per epilogue warp
        }
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(&tmem_slot, LOOP_TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t tm_j = tmem_base + (uint32_t)p.tm_j, tm_l = tmem_base + (uint32_t)p.tm_l, tm_p = tmem_base + (uint32_t)p.tm_p;

    const int e = threadIdx.x - 64;            // epilogue thread: 0..127 (warps 2..5), 0..255 (warps 2..9) in resident mode
    const int sub = (warp - 2) >> 2;           // resident mode: which of the two warps of a lane quadrant (0 otherwise)
    const int q = warp & 3;                    // tensor-memory lane quadrant of this warp
    const int row_in_tile = q * 32 + lane;     // the tensor-memory lane (accumulator row) of this thread
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    // joint items of this CTA.  Streaming mode: items cta, cta + G, ... of the (row group, vocabulary tile) list.
    // Resident mode: the CTA keeps ONE vocabulary tile (cta % vt_count) and takes the row groups j_first,
    // j_first + rg_stride, ... (one per wave); CTAs beyond vt_count * rg_stride have none.
    const int j_first = RES ? (cta < p.vt_count * p.rg_stride ? cta / p.vt_count : p.rg_count) : 0;
    const bool has_j = RES ? j_first < p.rg_count : cta < p.j_items;
    const int my_vt = cta % p.vt_count;        // vocabulary tile of this CTA's joint item when it has exactly one

    // ----- the joint's W_out tile, loaded once when every CTA owns one joint item -----
    if (p.j_mode == J_SMEM && has_j && threadIdx.x == 0) {
        mbar_expect_tx(&stat_bar, (uint32_t)p.kb_h * LOOP_A_BYTES);
        for (int kb = 0; kb < p.kb_h; ++kb) tma_load_2d(stat + (size_t)kb * LOOP_A_BYTES, &M.w_out, kb * BK, my_vt * 128, &stat_bar);
    }
    // resident-weights mode: CTAs [0, l_items) keep a W_hh tile (4 gates x 16 units), the last p_items CTAs a W_pred
    // tile (64 rows), loaded once; `stat` holds kb_p blocks of 64 rows x 64 columns
    // With two LSTM layers two more CTA sets follow the layer-0 set: "x1" keeps a W_ih[1] tile (layer 1's GEMM on the
    // new layer-0 state, in its own phase) and "h1" a W_hh[1] tile (layer 1's recurrent term, issued a phase ahead
    // like layer 0's GEMM and handed over through global memory).
    const int r_role = RES ? cta / p.l_items : 0;                  // 0 layer 0, 1 x1, 2 h1 (while below the L CTA count)
    const int r_idx = RES ? cta - r_role * p.l_items : 0;
    const bool res_l = RES && cta < p.l_items;
    const bool res_x1 = RES && p.L == 2 && r_role == 1;
    const bool res_h1 = RES && p.L == 2 && r_role == 2;
    const bool res_p = RES && !res_l && !res_x1 && !res_h1 && G - 1 - cta < p.p_items;
    const bool res_w = RES && cta >= p.w_first && cta < p.w_first + p.w_count;   // step-recording CTAs (none of the above)
    const int r_ut = r_idx % p.ut_count, r_ql = r_idx / p.ut_count;                  // unit tile / utterance group of an L CTA
    const int r_ht = (G - 1 - cta) % p.ht_count, r_qp = (G - 1 - cta) / p.ht_count;  // H tile / utterance group of a P CTA
    constexpr uint32_t RES_A_BYTES = 64 * BK * 2;
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
    if (p.j_mode == J_TMEM) {
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
    }

    // ----- pipeline state of the role threads -----
    uint32_t pe_bits = 0xffffffffu;   // TMA issuer: parity to wait for on empty_bar[s]
    uint32_t cf_bits = 0u;            // MMA issuer: parity to wait for on full_bar[s]
    uint32_t acc_n[3] = {0u, 0u, 0u}; // uses of each accumulator so far (MMA issuer and epilogue threads count alike)
    int cur = 0;                      // stage cursor, reset whenever the ring has drained
    uint32_t epoch = 0;               // grid barrier target (thread 0)
    int step = -1;                    // -1: start of sequence
    int pin = 0;                      // hb[pin] holds the current decoder state
    long long clk_last = 0, cyc[3] = {0, 0, 0};
    unsigned long long ns0 = 0;
    if (cta == 0 && threadIdx.x == 0) { clk_last = clock64(); ns0 = globaltimer_ns(); }
    int exit_status = 0;
    int tr_n = 0;                     // trace events written by this thread
    const bool early = p.l_early != 0;   // layer 0's GEMM is issued one phase ahead of its cell update

    const uint32_t sb_lp = p.stage_lp, sb_j = p.stage_j;   // stage bytes of the decoder/projection phases and of the joint phase
    const int S_lp = p.stages_lp, S_j = p.stages_j;

    // Grid barrier for all threads of all CTAs; false when the kernel is being abandoned.
    auto grid_sync = [&](int phase_kind) -> bool {
        __syncthreads();
        if (threadIdx.x == 0) {
            epoch += (uint32_t)(G + p.extra_arrivals);   // extra_arrivals > 0: a test hook, the barrier can then never fill
            if constexpr (FULL) trace_event(p, 3, tr_n, step, phase_kind, EV_ARRIVE);
            if constexpr (FULL) trace_phase_done(p, step, phase_kind);   // when this CTA finished its part of the phase
            if (s_abort) {
                atomicExch(&p.ctrl->abort, 1);
            } else {
                __threadfence();
                atomicAdd(&p.ctrl->bar, 1u);
                unsigned long long t0 = 0;
                for (uint32_t it = 1;; ++it) {
                    if ((int32_t)(ld_acquire_u32(&p.ctrl->bar) - epoch) >= 0) break;
                    if ((it & 63u) == 0u) {
                        if (ld_volatile_i32(&p.ctrl->abort)) { s_abort = 2; break; }
                        const unsigned long long now = globaltimer_ns();
                        if (t0 == 0) t0 = now;
                        else if (now - t0 > kWaitLimitNs) { s_abort = 1; atomicExch(&p.ctrl->abort, 1); break; }
                    }
                }
                // the acquire load orders this thread after every arrival; the block barrier below extends that to
                // the other threads of the CTA
            }
            if constexpr (FULL) trace_event(p, 3, tr_n, step, phase_kind, EV_RELEASE);
            if (cta == 0) {
                const long long now = clock64();
                cyc[phase_kind] += now - clk_last;
                clk_last = now;
            }
        }
        __syncthreads();
        return s_abort == 0;
    };

    // ----- TMA issuer (warp 0, lane 0) -----
    auto acquire = [&](uint32_t sb) -> uint8_t* {   // next free stage, nullptr when giving up
        if (!mbar_wait(&empty_bar[cur], (pe_bits >> cur) & 1u, &s_abort)) return nullptr;
        pe_bits ^= 1u << cur;
        return ring + (size_t)cur * sb;
    };
    // decoder GEMM operands of layer l for this CTA's items
    auto produce_L = [&](int l) -> bool {
        const uint32_t b_bytes = (uint32_t)(4 * p.slots) * BK * 2;
        const int segs = l == 0 ? 1 : 2;
        for (int i = cta; i < p.l_items; i += G) {
            const int mt = i / p.ug_count, ug = i - mt * p.ug_count;
            for (int sg = 0; sg < segs; ++sg) {
                const CUtensorMap* ma = (l == 0 || sg == 1) ? &M.hb[pin][l] : &M.hb[pin ^ 1][l - 1];
                const CUtensorMap* mb = (l == 0 || sg == 1) ? &M.w_hh[l] : &M.w_ih[l];
                for (int kb = 0; kb < p.kb_p; ++kb) {
                    uint8_t* a_dst = acquire(sb_lp);
                    if (!a_dst) return false;
                    uint8_t* b_dst = a_dst + LOOP_A_BYTES;
                    mbar_expect_tx(&full_bar[cur], LOOP_A_BYTES + b_bytes);
                    tma_load_2d(a_dst, ma, kb * BK, mt * 128, &full_bar[cur]);
                    for (int g = 0; g < 4; ++g)
                        tma_load_2d(b_dst + (size_t)g * p.slots * 128, mb, kb * BK, g * p.P + ug * p.ul, &full_bar[cur]);
                    cur = cur + 1 == S_lp ? 0 : cur + 1;
                }
            }
        }
        return true;
    };
    // ----- MMA issuer (warp 1, lane 0) -----
    auto consume = [&]() -> bool {
        if (!mbar_wait(&full_bar[cur], (cf_bits >> cur) & 1u, &s_abort)) return false;
        cf_bits ^= 1u << cur;
        tc_fence_after();
        return true;
    };
    auto begin_acc = [&](int k) -> bool {   // the epilogue has drained the previous use of accumulator k
        if (!mbar_wait(&acc_empty[k], (acc_n[k] & 1u) ^ 1u, &s_abort)) return false;
        tc_fence_after();
        return true;
    };
    auto mma_L = [&](int l) -> bool {
        const uint32_t idesc = idesc_bf16(128, 4 * p.slots);
        const int kbs = (l == 0 ? 1 : 2) * p.kb_p;
        for (int i = cta; i < p.l_items; i += G) {
            if (!begin_acc(1)) return false;
            for (int kb = 0; kb < kbs; ++kb) {
                if (!consume()) return false;
                const uint32_t a_addr = smem_u32(ring + (size_t)cur * sb_lp);
                const uint64_t adesc = smem_desc_sw128(a_addr);
                const uint64_t bdesc = smem_desc_sw128(a_addr + LOOP_A_BYTES);
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)
                    tc_mma_bf16(tm_l, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kb | k) != 0);
                tc_commit(&empty_bar[cur]);
                cur = cur + 1 == S_lp ? 0 : cur + 1;
            }
            tc_commit(&acc_full[1]);
            ++acc_n[1];
        }
        return true;
    };
    // ----- epilogue of the decoder phase of layer l: control step (layer 0 while decoding) + LSTM cell update -----
    auto epilogue_L = [&](int l) -> bool {
        const int32_t* t_cur = p.t2 + (size_t)(step & 1) * p.B;
        int32_t* t_nxt = p.t2 + (size_t)((step + 1) & 1) * p.B;
        const unsigned long long* keys_cur = p.keys2 + (size_t)(step & 1) * p.rows_pad;
        unsigned long long* keys_nxt = p.keys2 + (size_t)((step + 1) & 1) * p.rows_pad;
        const int32_t* len_cur = p.slot_len2 + (size_t)(step & 1) * p.B;
        int32_t* len_nxt = p.slot_len2 + (size_t)((step + 1) & 1) * p.B;
        const int32_t* row_cur = p.slot_row2 + (size_t)(step & 1) * p.B;
        int32_t* row_nxt = p.slot_row2 + (size_t)((step + 1) & 1) * p.B;
        for (int i = cta; i < p.l_items; i += G) {
            const int mt = i / p.ug_count, ug = i - mt * p.ug_count;
            const int b = mt * 128 + row_in_tile;
            const bool in = b < p.B;
            const int bb = in ? b : 0;
            float* cst = p.c_state + ((size_t)l * p.B + bb) * p.P;
            const __nv_bfloat16* hin = p.hb + (((size_t)pin * p.L + l) * p.Bpad + bb) * p.P;
            __nv_bfloat16* hout = p.hb + (((size_t)(pin ^ 1) * p.L + l) * p.Bpad + bb) * p.P;
            const int unit0 = ug * p.ul;
            // ---- which token does utterance b feed to its decoder in this step? ----
            int tok = -1;
            if (in) {
                if (step < 0) {
                    tok = p.blank;
                } else if ((FULL && p.forced)) {
                    tok = step < p.prefix_len[b] ? p.prefix[(size_t)b * p.U + step] : -1;
                    if (tok >= p.NV || tok < -1) { tok = p.blank; set_status(p.ctrl, WIND_ERR_INVALID_ARG); }   // caller's mistake
                } else if (l > 0) {
                    tok = p.emit_tok[b];
                } else {
                    // control step (Algorithm 2's branch): first non-blank row of the window.
                    // Everything it needs is requested at once; the keys of all W rows are readable.
                    int t = t_cur[b];
                    const int len_word = len_cur[b];
                    const int len = len_word & kSlotLenMask;
                    const bool writer = ug == 0;
                    int cnt = 0, pos = 0, s_row = 0, s_utt = 0;
                    if (writer) { cnt = p.count[b]; pos = p.slot_pos[b]; s_row = row_cur[b]; s_utt = p.slot_utt[b]; }
                    int len_out = len, row_out = s_row;
                    unsigned long long kk[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) kk[j] = j < p.W ? keys_cur[(size_t)b * p.W + j] : 0ull;
                    if (len_word & kSlotFresh) {
                        // the row took a new utterance in the last step (its state is zero since then): start of sequence
                        tok = p.blank;
                        if (writer) {
                            t_nxt[b] = t;
                            for (int w = 0; w < p.W; ++w) keys_nxt[(size_t)b * p.W + w] = 0ull;
                        }
                    } else if (t < len) {
                        const int n = min(p.W, len - t);
                        int first = -1, label = p.blank;
                        bool bad = false;
                        for (int w0 = 0; w0 < n && first < 0; w0 += 8) {
                            if (w0 > 0) {
#pragma unroll
                                for (int j = 0; j < 8; ++j) kk[j] = (w0 + j < n) ? keys_cur[(size_t)b * p.W + w0 + j] : 0ull;
                            }
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                if (w0 + j < n && first < 0) {
                                    uint32_t lab = key_label(kk[j]);
                                    if (kk[j] == 0ull || lab >= (uint32_t)p.NV) { bad = true; lab = (uint32_t)p.blank; }
                                    if ((int)lab != p.blank) { first = w0 + j; label = (int)lab; }
                                }
                            }
                        }
                        if (first >= 0) tok = label;
                        if (writer) {
                            // this CTA records the step for its utterances
                            int jump, forced = 0, emitted = 0;
                            if (first < 0) {
                                jump = n;
                                t += n;
                                cnt = 0;
                            } else {
                                jump = first;
                                if (first > 0) cnt = 0;
                                t += first;
                                if (pos < p.max_out) {
                                    p.out_tokens[(size_t)s_utt * p.max_out + pos] = label;
                                    p.out_frames[(size_t)s_utt * p.max_out + pos] = t;
                                    p.out_len[s_utt] = pos + 1;
                                    p.slot_pos[b] = pos + 1;
                                    emitted = 1;
                                    cnt += 1;
                                    if (cnt == p.S) { t += 1; cnt = 0; forced = 1; }
                                } else {
                                    set_status(p.ctrl, WIND_ERR_OUTPUT_OVERFLOW);  // this utterance stops here
                                    t = len;
                                    tok = -1;
                                }
                            }
                            if (bad) set_status(p.ctrl, WIND_ERR_INTERNAL);
                            t_nxt[b] = t;
                            p.count[b] = cnt;
                            for (int w = 0; w < p.W; ++w) keys_nxt[(size_t)b * p.W + w] = 0ull;
                            atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->jump_hist[jump < 64 ? jump : 64]), 1ull);
                            atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->joint_rows), (unsigned long long)n);
                            if (emitted) atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->tokens), 1ull);
                            if (forced) atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->forced), 1ull);
                        }
                    } else {
                        // nothing left of this row's utterance: its decoder state is cleared, so that an utterance that
                        // takes the row over starts from the zero state
                        tok = -2;
                        if (writer) {
                            t_nxt[b] = t;
                            if (ld_volatile_i32(&p.ctrl->next_utt) < p.n_utt) {
                                const int u = atomicAdd(&p.ctrl->next_utt, 1);
                                if (u < p.n_utt) {
                                    // the next waiting utterance moves in; the coming step feeds it start-of-sequence
                                    len_out = min(max(p.enc_len[u], 0), p.T) | kSlotFresh;
                                    row_out = u * p.T;
                                    p.slot_utt[b] = u;
                                    p.slot_pos[b] = 0;
                                    p.count[b] = 0;
                                    t_nxt[b] = 0;
                                }
                            }
                        }
                    }
                    if (writer) {
                        len_nxt[b] = len_out;
                        row_nxt[b] = row_out;
                        p.emit_tok[b] = tok;
                    }
                }
            }
            if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_TOK);
            const bool live = in && tok >= 0;
            // what the cell update needs from memory, requested before the accumulator is waited for
            float add[4][8], cold[8];
            auto load_operands = [&](int u0) {
                if (live) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int unit = unit0 + u0 + j;
                        const bool ok = u0 + j < p.ul && unit < p.P;
                        cold[j] = ok ? cst[unit] : 0.f;
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            if (l == 0) add[g][j] = ok ? p.g0[(size_t)tok * 4 * p.P + (size_t)g * p.P + unit] : 0.f;
                            else add[g][j] = ok ? p.b_ih[l][g * p.P + unit] + p.b_hh[l][g * p.P + unit] : 0.f;
                        }
                    }
                }
            };
            load_operands(0);
            const bool ready = __all_sync(0xffffffffu, mbar_wait(&acc_full[1], acc_n[1] & 1u, &s_abort));
            tc_fence_after();
            if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_ACC);
            if (ready) {
                for (int u0 = 0; u0 < p.ul; u0 += 8) {
                    if (u0 > 0) load_operands(u0);
                    float pre[4][8];
#pragma unroll
                    for (int g = 0; g < 4; ++g) tmem_ld8(tm_l + lane_off + (uint32_t)(g * p.slots + u0), pre[g]);
                    if (in) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int unit = unit0 + u0 + j;
                            if (u0 + j < p.ul && unit < p.P) {
                                if (live) {
                                    const float gi = sigmoid_f(pre[0][j] + add[0][j]);
                                    const float gf = sigmoid_f(pre[1][j] + add[1][j]);
                                    const float gg = tanhf(pre[2][j] + add[2][j]);
                                    const float go = sigmoid_f(pre[3][j] + add[3][j]);
                                    const float cc = gf * cold[j] + gi * gg;
                                    cst[unit] = cc;
                                    hout[unit] = __float2bfloat16_rn(go * tanhf(cc));
                                } else if (tok == -2) {
                                    cst[unit] = 0.f;
                                    hout[unit] = __float2bfloat16_rn(0.f);
                                } else {
                                    hout[unit] = hin[unit];
                                }
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[1]);
            ++acc_n[1];
            if (!ready) return false;
        }
        if (cta == 0 && e == 0 && l == 0 && step >= 0 && !(FULL && p.forced)) p.ctrl->step = step + 1;
        fence_proxy_async_all();
        if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_EPI_DONE);
        return true;
    };

    // =========================================================================================
    // resident-weights mode.  Every per-step operand is ONE three-dimensional TMA box (all K blocks at once) into
    // the single operand buffer, and every GEMM is one wait, kb x 4 MMAs back to back, two commits: the issuing
    // threads pay for as few asynchronous instructions as possible.
    //   decoder:    D[4 gates x 16 units, nl utterances] = W_hh tile . h^T   (warp q of the epilogue = gate q)
    //   projection: D[64 H rows, np utterances] = W_pred tile . h^T
    // With 64 accumulator rows, row m sits in lane (m % 16) of quadrant m / 16.
    // =========================================================================================
    float* stage_f = reinterpret_cast<float*>(smem + p.stage_off);   // epilogue staging
    auto produce_one = [&](const CUtensorMap* map, int row0, uint32_t bytes) -> bool {
        cur = 0;
        uint8_t* dst = acquire(0);
        if (!dst) return false;
        mbar_expect_tx(&full_bar[0], bytes);
        tma_load_3d(dst, map, 0, row0, 0, &full_bar[0]);
        return true;
    };
    // One issuing thread's share of a GEMM: K blocks [kb_lo, kb_hi) into the accumulator at tm_d.  Two threads call
    // this for every GEMM (warp 1 and, after it has issued the TMA box, warp 0), with disjoint K ranges and
    // separate accumulator copies that the epilogue adds; an empty range only takes part in the commits.
    auto mma_part = [&](int k_acc, uint32_t tm_d, int n_tile, int kb_lo, int kb_hi, bool a_tmem) -> bool {
        const uint32_t idesc = idesc_bf16(a_tmem ? 128 : 64, n_tile);
        if (!a_tmem && !mbar_wait(&stat_bar, 0, &s_abort)) return false;
        if (!begin_acc(k_acc)) return false;
        cur = 0;
        if (!consume()) return false;
        const uint32_t b_addr = smem_u32(ring);
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
        tc_commit(&empty_bar[0]);
        tc_commit(&acc_full[k_acc]);
        ++acc_n[k_acc];
        return true;
    };
    // control step + LSTM cell update of an L CTA: units [r_ut*16, +16), utterances [r_ql*nl, +nl), 64 utterances per
    // pass.  Warp (q, sub) of the epilogue owns gate q and the pass's utterances [32 sub, 32 sub + 32).  All global reads
    // of a pass are requested together: first everything the control step needs, then the gate-table rows of the
    // chosen tokens.  Lanes 16..31 hold no accumulator row (64-row tile); they take the second 16 utterances.
    struct ScanIn { int t, len, cnt, pos; unsigned long long kk[8]; };
    // ctl_only: the CTA is one of the step-recording CTAs (see the plan): it takes the control step of 64 utterances,
    // records it (outputs, counters, next frame) and has no cell update; the L CTAs then record nothing.
    auto epilogue_res_L = [&](const int layer, const bool ctl_only) -> bool {
        if (ctl_only && q != 0) return true;
        const int32_t* t_cur = p.t2 + (size_t)(step & 1) * p.B;
        int32_t* t_nxt = p.t2 + (size_t)((step + 1) & 1) * p.B;
        const unsigned long long* keys_cur = p.keys2 + (size_t)(step & 1) * p.rows_pad;
        unsigned long long* keys_nxt = p.keys2 + (size_t)((step + 1) & 1) * p.rows_pad;
        const int cur_off = (step & 1) * p.B, nxt_off = p.B - cur_off;   // the slot arrays' copy of this step and of the next
        const int u16 = lane & 15, half = lane >> 4;
        const int unit = r_ut * 16 + u16;        // this thread's hidden unit; its gate is q
        // without recording CTAs, the two gate-0 warps of one CTA per utterance group record the step
        const bool writer = ctl_only ? true : (p.w_count == 0 && layer == 0 && r_ut == 0 && q == 0);
        const int n_here = ctl_only ? 64 : p.nl;
        const int base = ctl_only ? (cta - p.w_first) * 64 : r_ql * p.nl;
        const bool decode = step >= 0 && !(FULL && p.forced) && layer == 0;
        float* cst = p.c_state + (size_t)layer * p.B * p.P + unit;
        const __nv_bfloat16* hin = p.hb + ((size_t)(pin * p.L + layer) * p.Bpad) * p.P + unit;
        __nv_bfloat16* hout = p.hb + ((size_t)((pin ^ 1) * p.L + layer) * p.Bpad) * p.P + unit;
        const float bias1 = layer == 0 ? 0.f : p.b_ih[1][q * p.P + unit] + p.b_hh[1][q * p.P + unit];
        const float* g0u = p.g0 + (size_t)q * p.P + unit;
        const uint32_t g0_stride = 4u * (uint32_t)p.P;
        bool ready = true;
        for (int c0 = 0; c0 < n_here; c0 += 64) {
            const int b0 = base + c0;
            // ---- lane j decides for utterance b0 + 32 sub + j ----
            const int jl = 32 * sub + lane;
            const int b = b0 + jl;
            const bool in = c0 + jl < n_here && b < p.B;
            ScanIn si;
            si.t = 0; si.len = 0; si.cnt = 0; si.pos = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) si.kk[j] = 0ull;
            int s_row = 0;
            if (in && decode) {
                si.t = t_cur[b];
                si.len = p.slot_len2[cur_off + b];
                if (writer) { si.cnt = p.count[b]; si.pos = p.slot_pos[b]; s_row = p.slot_row2[cur_off + b]; }
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (j < p.W) si.kk[j] = keys_cur[(size_t)b * p.W + j];
            }
            // old cell state of the four (utterance, unit) pairs this thread finishes
            float cold[4];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int j = half + 2 * q + 8 * sub + 16 * jj;     // 0..63 over the CTA's 256 epilogue threads
                cold[jj] = (!ctl_only && c0 + j < p.nl && b0 + j < p.B) ? cst[(size_t)(b0 + j) * p.P] : 0.f;
            }
            // the token utterance b feeds to its decoder in this step (-1: none)
            int tok = -1, t_out = 0, t_left = 0;
            uint32_t t_row = 0u;
            if (in) {
                if (step < 0) {
                    tok = p.blank;
                    if (writer) { t_row = (uint32_t)p.slot_row2[cur_off + b]; t_left = p.slot_len2[cur_off + b] & kSlotLenMask; }   // frame 0 of the row's first utterance
                } else if ((FULL && p.forced)) {
                    tok = step < p.prefix_len[b] ? p.prefix[(size_t)b * p.U + step] : -1;
                    if (tok >= p.NV || tok < -1) { tok = p.blank; set_status(p.ctrl, WIND_ERR_INVALID_ARG); }   // caller's mistake
                } else if (layer > 0) {
                    tok = p.emit_tok[b];     // decided by layer 0's CTAs one phase earlier
                } else {
                    int t = si.t;
                    const int len = si.len & kSlotLenMask;
                    int len_out = len, row_out = s_row;
                    if (si.len & kSlotFresh) {
                        // the row took a new utterance in the last step (its state is zero since then): start of sequence
                        tok = p.blank;
                        if (writer) {
                            t_nxt[b] = t;
                            t_out = t;
                            for (int w = 0; w < p.W; ++w) keys_nxt[(size_t)b * p.W + w] = 0ull;
                        }
                    } else if (t < len) {
                        // control step (Algorithm 2's branch): first non-blank row of the window
                        const int n = min(p.W, len - t);
                        int first = -1, label = p.blank;
                        bool bad = false;
                        for (int w0 = 0; w0 < n && first < 0; w0 += 8) {
                            if (w0 > 0) {
#pragma unroll
                                for (int j = 0; j < 8; ++j) si.kk[j] = (w0 + j < n) ? keys_cur[(size_t)b * p.W + w0 + j] : 0ull;
                            }
                            // the eight rows side by side: which are inside the window, broken, non-blank
                            uint32_t nonblank = 0u, broken = 0u;
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const uint32_t lab = key_label(si.kk[j]);
                                const bool inside = w0 + j < n;
                                const bool brk = si.kk[j] == 0ull || lab >= (uint32_t)p.NV;
                                broken |= (uint32_t)(inside && brk) << j;
                                nonblank |= (uint32_t)(inside && !brk && (int)lab != p.blank) << j;
                            }
                            if (nonblank) {
                                const int j = __ffs((int)nonblank) - 1;
                                first = w0 + j;
                                uint32_t lab = 0u;
#pragma unroll
                                for (int jj = 0; jj < 8; ++jj)
                                    if (jj == j) lab = key_label(si.kk[jj]);
                                label = (int)lab;
                                broken &= (1u << j) - 1u;   // rows after the first non-blank one are not looked at
                            }
                            bad = bad || broken != 0u;
                        }
                        if (first >= 0) tok = label;
                        if (writer) {
                            int cnt = si.cnt, jump, forced = 0, emitted = 0;
                            if (first < 0) {
                                jump = n;
                                t += n;
                                cnt = 0;
                            } else {
                                jump = first;
                                if (first > 0) cnt = 0;
                                t += first;
                                if (si.pos < p.max_out) {
                                    const int s_utt = p.slot_utt[b];   // which utterance the row decodes (index into the outputs)
                                    p.out_tokens[(size_t)s_utt * p.max_out + si.pos] = label;
                                    p.out_frames[(size_t)s_utt * p.max_out + si.pos] = t;
                                    p.out_len[s_utt] = si.pos + 1;
                                    p.slot_pos[b] = si.pos + 1;
                                    emitted = 1;
                                    cnt += 1;
                                    if (cnt == p.S) { t += 1; cnt = 0; forced = 1; }
                                } else {
                                    set_status(p.ctrl, WIND_ERR_OUTPUT_OVERFLOW);  // this utterance stops here
                                    t = len;
                                    tok = -1;
                                }
                            }
                            if (bad) set_status(p.ctrl, WIND_ERR_INTERNAL);
                            t_nxt[b] = t;
                            t_out = t;
                            p.count[b] = cnt;
                            for (int w = 0; w < p.W; ++w) keys_nxt[(size_t)b * p.W + w] = 0ull;
                            atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->jump_hist[jump < 64 ? jump : 64]), 1ull);
                            atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->joint_rows), (unsigned long long)n);
                            if (emitted) atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->tokens), 1ull);
                            if (forced) atomicAdd(reinterpret_cast<unsigned long long*>(&p.ctrl->forced), 1ull);
                        }
                    } else {
                        // nothing left of this row's utterance: its decoder state is cleared, so that an utterance that
                        // takes the row over starts from the zero state
                        tok = -2;
                        if (writer) {
                            t_nxt[b] = t;
                            t_out = t;
                            if (ld_volatile_i32(&p.ctrl->next_utt) < p.n_utt) {
                                const int u = atomicAdd(&p.ctrl->next_utt, 1);
                                if (u < p.n_utt) {
                                    // the next waiting utterance moves in; the coming step feeds it start-of-sequence
                                    len_out = min(max(p.enc_len[u], 0), p.T) | kSlotFresh;
                                    row_out = u * p.T;
                                    p.slot_utt[b] = u;
                                    p.slot_pos[b] = 0;
                                    p.count[b] = 0;
                                    t_nxt[b] = 0;
                                    t_out = 0;
                                }
                            }
                        }
                    }
                    if (writer) {
                        p.slot_len2[nxt_off + b] = len_out;
                        p.slot_row2[nxt_off + b] = row_out;
                        t_row = (uint32_t)row_out + (uint32_t)t_out;
                        t_left = (len_out & kSlotLenMask) - t_out;
                    }
                }
                // the next frame goes out at once, stamped with the step, for the projection CTAs (which fetch their
                // enc_proj rows while this phase is still running): enc_proj row of the frame, frames left (capped)
                if (writer && !(FULL && p.forced))
                    p.t_pub[b] = ((unsigned long long)(((uint32_t)(step + 2) << 8) | (uint32_t)min(max(t_left, 0), 255)) << 32) | t_row;
                if (writer && p.L > 1 && decode) p.emit_tok[b] = tok;   // the upper layer's CTAs read it in their phase
            }
            if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_TOK);
            if (ctl_only) continue;
            // ---- gate-table entries (this thread's gate and unit) of the tokens of this lane half's 16 utterances ----
            float add[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const int ta = __shfl_sync(0xffffffffu, tok, j), tb = __shfl_sync(0xffffffffu, tok, 16 + j);
                const int tj = half ? tb : ta;
                if (layer == 0) {
                    add[j] = tj >= 0 ? g0u[(uint32_t)tj * g0_stride] : 0.f;
                } else {
                    // layer 1: the recurrent term W_hh h computed a phase ahead by the h1 CTAs, plus the biases
                    const int bj2 = b0 + 32 * sub + 16 * half + j;
                    add[j] = (tj >= 0 && bj2 < p.B) ? p.dh[(size_t)bj2 * g0_stride + (size_t)q * p.P + unit] + bias1 : 0.f;
                }
            }
            // the other warps need the tokens for the cell update below: through shared memory
            int* tok_s = reinterpret_cast<int*>(stage_f + 4 * 64 * 16);
            if (q == 0) tok_s[jl] = tok;
            if (c0 == 0) {
                ready = __all_sync(0xffffffffu, mbar_wait(&acc_full[1], acc_n[1] & 1u, &s_abort));
                tc_fence_after();
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_ACC);
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
                        } else if (tok_s[j] == -2) {
                            cst[(size_t)bj * p.P] = 0.f;
                            hout[(size_t)bj * p.P] = __float2bfloat16_rn(0.f);
                        } else {
                            hout[(size_t)bj * p.P] = hin[(size_t)bj * p.P];
                        }
                    }
                }
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");
        }
        if (ctl_only) return true;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[1]);
        ++acc_n[1];
        fence_proxy_async_all();
        if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_EPI_DONE);
        return ready;
    };
    // z rows of a P CTA: row r = (utterance bl = r / W of the CTA's group, window row w = r % W), 64 columns = 128 bytes =
    // eight 16-byte chunks.  Thread e owns chunk (e & 7) of rows (e >> 3) + 32 i, so that eight neighbouring lanes
    // read and write one whole 128-byte row segment.  Row kinds: 0 nothing to write (outside the batch, or the
    // utterance is done), 1 zeros (past the utterance's end), 2 act(enc_proj row + pred_proj).
    //
    // During the decoder-update phase a P CTA has nothing else to do: it waits for the next frame of its
    // utterances to be published and starts copying the enc_proj chunks of its first 256 rows into a shared-memory
    // stash (asynchronous copies, collected in the projection epilogue).  pre_kinds: 2 bits per row, -1 = no prefetch.
    uint8_t* stash = ring + (size_t)p.np * p.P * 2;   // behind the projection's own operand box
    int pre_kinds = -1;
    const int p_chunk = e & 7, p_row0 = e >> 3;
    // the (utterance, window row) of this thread's first eight rows never changes: worked out once, so that the
    // per-step code has no integer division; -1 = no such row
    int p_bw[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        p_bw[i] = -1;
        if (res_p && e >= 0) {
            const int r = p_row0 + 32 * i;
            const int bl = r / p.W, w = r - bl * p.W, b = r_qp * p.np + bl;
            if (r < p.np * p.W && b < p.B) p_bw[i] = (b << 8) | w;
        }
    }
    // b_pred of this thread's accumulator row: constant for the whole decode, read once
    const float p_bias = (res_p && e >= 0) ? p.b_pred[r_ht * 64 + 16 * q + (lane & 15)] : 0.f;
    // kind of a row at frame position t of its utterance, and the row's enc_proj frame
    auto row_kind = [&](int w, int left) -> int { return left <= 0 ? 0 : (w >= left ? 1 : 2); };
    auto prefetch_res_P = [&]() {
        pre_kinds = -1;
        if ((FULL && p.forced)) return;
        const uint32_t want = (uint32_t)(step + 2) & 0xFFFFFFu;
        // the published frames of this thread's rows, all requested together, until every stamp is this step's
        unsigned long long v[8];
        unsigned long long t0 = 0;
        for (uint32_t it = 1;; ++it) {
            bool all = true;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                v[i] = (unsigned long long)want << 40;
                if (p_bw[i] >= 0) asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(v[i]) : "l"(p.t_pub + (p_bw[i] >> 8)) : "memory");
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) all = all && (uint32_t)(v[i] >> 40) == want;
            if (all) break;
            if ((it & 15u) == 0u) {
                if (s_abort || ld_volatile_i32(&p.ctrl->abort)) return;
                const unsigned long long now = globaltimer_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > kWaitLimitNs) { s_abort = 1; return; }
            }
        }
        int kinds = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (p_bw[i] < 0) continue;
            const int w = p_bw[i] & 255;
            const int kind = row_kind(w, (int)((v[i] >> 32) & 255u));
            kinds |= kind << (2 * i);
            if (kind == 2) {
                const __nv_bfloat16* src = p.enc_proj + ((size_t)(uint32_t)v[i] + w) * p.H + r_ht * 64 + p_chunk * 8;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(stash + (size_t)(p_row0 + 32 * i) * 128 + p_chunk * 16)),
                             "l"(src)
                             : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        pre_kinds = kinds;
    };
    // projection epilogue of a P CTA: pred_proj rows [r_ht*64, +64) of utterances [r_qp*np, +np), then z
    auto epilogue_res_P = [&]() -> bool {
        const int32_t* t_new = p.t2 + (size_t)((step + 1) & 1) * p.B;
        const int32_t* len_new = p.slot_len2 + (size_t)((step + 1) & 1) * p.B;
        const int32_t* row_new = p.slot_row2 + (size_t)((step + 1) & 1) * p.B;
        const int h0 = r_ht * 64;
        const int rows_here = p.np * p.W;
        // one 16-byte chunk of a z row: act(enc_proj chunk + pred_proj chunk), zeros past the utterance's end
        // (pred_proj is rounded to bf16 and the sum is taken in bf16 arithmetic, one rounding: the same instruction
        // sequence as in the resident kernel without grid barriers, so that the two give the same transcripts)
        auto z_chunk = [&](int bl, int kind, uint4 ev) -> uint4 {
            const float4* gs = reinterpret_cast<const float4*>(stage_f + bl * 68 + p_chunk * 8);
            const float4 ga = gs[0], gb = gs[1];
            if (kind != 2) return make_uint4(0, 0, 0, 0);
            return make_uint4(act_add_bf16x2(ev.x, pack_bf16x2(ga.x, ga.y), p.act), act_add_bf16x2(ev.y, pack_bf16x2(ga.z, ga.w), p.act),
                              act_add_bf16x2(ev.z, pack_bf16x2(gb.x, gb.y), p.act), act_add_bf16x2(ev.w, pack_bf16x2(gb.z, gb.w), p.act));
        };
        // the chunks of this thread's first eight rows: prefetched, or requested now before the accumulator is ready
        uint4 ev[8];
        int kinds = pre_kinds;
        if (kinds < 0) {
            kinds = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                ev[i] = make_uint4(0, 0, 0, 0);
                if (p_bw[i] >= 0) {
                    const int b = p_bw[i] >> 8, w = p_bw[i] & 255;
                    const int t = t_new[b];
                    const int kind = row_kind(w, (len_new[b] & kSlotLenMask) - t);
                    kinds |= kind << (2 * i);
                    if (kind == 2) ev[i] = *reinterpret_cast<const uint4*>(p.enc_proj + ((size_t)row_new[b] + t + w) * p.H + h0 + p_chunk * 8);
                }
            }
        } else {
            asm volatile("cp.async.wait_all;" ::: "memory");
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                ev[i] = make_uint4(0, 0, 0, 0);
                if (((kinds >> (2 * i)) & 3) == 2) ev[i] = *reinterpret_cast<const uint4*>(stash + (size_t)(p_row0 + 32 * i) * 128 + p_chunk * 16);
            }
        }
        if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_TOK);
        const bool ready = __all_sync(0xffffffffu, mbar_wait(&acc_full[2], acc_n[2] & 1u, &s_abort));
        tc_fence_after();
        if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_ACC);
        if (ready) {
            const int hl = 16 * q + (lane & 15);
            const float bias = p_bias;
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
                    for (int j = 0; j < 16; ++j) stage_f[(c0 + j) * 68 + hl] = g[j] + more[j] + bias;
                }
            }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[2]);
        ++acc_n[2];
        asm volatile("bar.sync 1, 256;" ::: "memory");
        if (ready) {
            uint4 out[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int bl = p_bw[i] >= 0 ? (p_bw[i] >> 8) - r_qp * p.np : 0;
                out[i] = z_chunk(bl, (kinds >> (2 * i)) & 3, ev[i]);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (p_bw[i] >= 0 && ((kinds >> (2 * i)) & 3) != 0) {
                    const int b = p_bw[i] >> 8, w = p_bw[i] & 255;
                    *reinterpret_cast<uint4*>(p.z + ((size_t)b * p.W + w) * p.H + h0 + p_chunk * 8) = out[i];
                }
            }
            // rows beyond the first 256 of this CTA (wide windows): same chunking, fetched here
            // (four rows at a time, their loads requested together)
            for (int r0 = p_row0 + 256; r0 < rows_here; r0 += 128) {
                uint4 x[4];
                int kinds4[4], bls[4];
                size_t zoff[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int r = r0 + 32 * i;
                    const int bl = r / p.W, w = r - bl * p.W, b = r_qp * p.np + bl;
                    x[i] = make_uint4(0, 0, 0, 0);
                    kinds4[i] = 0; bls[i] = 0; zoff[i] = 0;
                    if (r < rows_here && b < p.B) {
                        const int t = t_new[b];
                        kinds4[i] = row_kind(w, (len_new[b] & kSlotLenMask) - t);
                        bls[i] = bl;
                        zoff[i] = ((size_t)b * p.W + w) * p.H + h0 + p_chunk * 8;
                        if (kinds4[i] == 2)
                            x[i] = *reinterpret_cast<const uint4*>(p.enc_proj + ((size_t)row_new[b] + t + w) * p.H + h0 + p_chunk * 8);
                    }
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (kinds4[i] != 0) *reinterpret_cast<uint4*>(p.z + zoff[i]) = z_chunk(bls[i], kinds4[i], x[i]);
            }
        }
        fence_proxy_async_all();
        if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_EPI_DONE);
        return ready;
    };
    // the decoder GEMM of the next step, on the state hb[pin] (TMA and MMA issuers of an L CTA)
    // h1 CTAs: the finished recurrent term of layer 1 goes to global memory (fp32 [B][4P], gate-major like the gate
    // table); the x1 CTAs add it one or two phases later
    auto store_res_h1 = [&]() {
        const bool ready = __all_sync(0xffffffffu, mbar_wait(&acc_full[1], acc_n[1] & 1u, &s_abort));
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
    };
    // GEMMs that need only the state, issued a phase ahead: layer 0's (its result waits in tensor memory for the
    // next control step) and, with two layers, layer 1's recurrent term (stored by store_res_h1)
    auto early_res = [&]() {
        if (warp == 0) {
            if (lane == 0 && (res_l || res_h1)) {
                fence_proxy_async_all();
                if (produce_one(res_l ? &M.hb_l3[pin] : &M.hb_l3_1[pin], r_ql * p.nl, (uint32_t)p.nl * (uint32_t)p.P * 2u))
                    mma_part(1, tm_l, p.nl, p.kb_p, p.kb_p, false);   // one accumulator: warp 1 issues all of it
            }
        } else if (warp == 1) {
            if (lane == 0 && (res_l || res_h1)) mma_part(1, tm_l, p.nl, 0, p.kb_p, false);
        } else if (res_h1) {
            store_res_h1();
        }
    };

    // Measurement aid (FULL variant): the joint phase alone, joint_iters times back to back on the z rows the workspace
    // holds, every CTA for itself (no barrier in between).
    const bool jo = FULL && p.joint_iters > 0;
    int jo_it = 0;
    if (jo) { step = 0; goto joint_only_entry; }
    // ----- before the loop: layer 0's GEMM on the initial (zero) state -----
    if constexpr (RES) {
        early_res();
    } else if (early) {
        if (warp == 0) {
            if (lane == 0) { fence_proxy_async_all(); cur = 0; produce_L(0); }
        } else if (warp == 1) {
            if (lane == 0) { cur = 0; mma_L(0); }
        }
    }

    for (;;) {
        // =====================================================================================
        // decoder phases: control step + LSTM cell update (layer 0), then one GEMM + update phase per upper layer
        // =====================================================================================
        if constexpr (RES) {
            if (warp >= 2) {
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_START);
                if (res_l) epilogue_res_L(0, false);
                else if (res_w) epilogue_res_L(0, true);
                else if (res_p) prefetch_res_P();
                if (cta == 0 && e == 0 && step >= 0 && !(FULL && p.forced)) p.ctrl->step = step + 1;
            }
            if (!grid_sync(TR_L)) goto done;
            if (p.L == 2) {
                // layer 1: W_ih[1] . (new layer-0 state) on the x1 CTAs, then their cell update
                if (warp == 0) {
                    if (lane == 0 && res_x1) {
                        fence_proxy_async_all();
                        if (produce_one(&M.hb_l3[pin ^ 1], r_ql * p.nl, (uint32_t)p.nl * (uint32_t)p.P * 2u))
                            mma_part(1, tm_l, p.nl, p.kb_p, p.kb_p, false);
                    }
                } else if (warp == 1) {
                    if (lane == 0 && res_x1) mma_part(1, tm_l, p.nl, 0, p.kb_p, false);
                } else if (res_x1) {
                    epilogue_res_L(1, false);
                }
                if (!grid_sync(TR_L)) goto done;
            }
        }
        for (int l = 0; l < p.L && !RES; ++l) {
            const bool gemm_here = l > 0 || !early;
            if (warp == 0) {
                if (lane == 0 && gemm_here) { fence_proxy_async_all(); cur = 0; produce_L(l); }
            } else if (warp == 1) {
                if (lane == 0 && gemm_here) { cur = 0; mma_L(l); }
            } else {
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_L, EV_START);
                epilogue_L(l);
            }
            if (!grid_sync(TR_L)) goto done;
        }
        pin ^= 1;
        if ((FULL && p.forced) && step + 1 < p.U) {
            // teacher forcing: more prefix tokens to feed before the window is evaluated
            if constexpr (RES) {
                early_res();
            } else if (early) {
                if (warp == 0) {
                    if (lane == 0) { fence_proxy_async_all(); cur = 0; produce_L(0); }
                } else if (warp == 1) {
                    if (lane == 0) { cur = 0; mma_L(0); }
                }
            }
            ++step;
            continue;
        }

        // =====================================================================================
        // projection phase: pred_proj for every utterance, then the next window's joint activations z;
        // behind it, layer 0's GEMM of the next step (its result waits in tensor memory)
        // =====================================================================================
        {
            const int n_tile = p.np;
            const uint32_t b_bytes = (uint32_t)n_tile * BK * 2;
            const int32_t* t_new = p.t2 + (size_t)((step + 1) & 1) * p.B;
            const int32_t* len_new = p.slot_len2 + (size_t)((step + 1) & 1) * p.B;
            const int32_t* row_new = p.slot_row2 + (size_t)((step + 1) & 1) * p.B;
            const int i0 = p.p_items <= G ? G - 1 - cta : cta;   // projection items start at the far end of the grid
            if constexpr (RES) {
                if (warp == 0) {
                    if (lane == 0 && res_p) {
                        fence_proxy_async_all();
                        if (produce_one(&M.hb_p3[pin], r_qp * p.np, (uint32_t)p.np * (uint32_t)p.P * 2u))
                            mma_part(2, tm_p + (uint32_t)p.np, p.np, p.kb_p / 2, p.kb_p, false);
                    }
                } else if (warp == 1) {
                    if (lane == 0 && res_p) mma_part(2, tm_p, p.np, 0, p.kb_p / 2, false);
                } else {
                    if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_START);
                    // rows still decoding, plus one while utterances wait for a row
                    int cnt = (e == 0 && ld_volatile_i32(&p.ctrl->next_utt) < p.n_utt) ? 1 : 0;
                    for (int b = e; b < p.B; b += 256) cnt += t_new[b] < (len_new[b] & kSlotLenMask);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
                    if (lane == 0) s_red[warp - 2] = cnt;
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                    if (e == 0) s_active = s_red[0] + s_red[1] + s_red[2] + s_red[3] + s_red[4] + s_red[5] + s_red[6] + s_red[7];
                    if (res_p) epilogue_res_P();
                }
                early_res();
            } else if (warp == 0) {
                if (lane == 0) {
                    fence_proxy_async_all();
                    cur = 0;
                    bool ok = true;
                    for (int i = i0; i < p.p_items && ok; i += G) {
                        const int mt = i / p.hg_count, hg = i - mt * p.hg_count;
                        for (int kb = 0; kb < p.kb_p; ++kb) {
                            uint8_t* a_dst = acquire(sb_lp);
                            if (!a_dst) { ok = false; break; }
                            mbar_expect_tx(&full_bar[cur], LOOP_A_BYTES + b_bytes);
                            tma_load_2d(a_dst, &M.hb[pin][p.L - 1], kb * BK, mt * 128, &full_bar[cur]);
                            tma_load_2d(a_dst + LOOP_A_BYTES, &M.w_pred, kb * BK, hg * p.np, &full_bar[cur]);
                            cur = cur + 1 == S_lp ? 0 : cur + 1;
                        }
                    }
                    if (ok && early) produce_L(0);
                }
            } else if (warp == 1) {
                if (lane == 0) {
                    const uint32_t idesc = idesc_bf16(128, n_tile);
                    cur = 0;
                    bool ok = true;
                    for (int i = i0; i < p.p_items && ok; i += G) {
                        if (!begin_acc(2)) { ok = false; break; }
                        for (int kb = 0; kb < p.kb_p; ++kb) {
                            if (!consume()) { ok = false; break; }
                            const uint32_t a_addr = smem_u32(ring + (size_t)cur * sb_lp);
                            const uint64_t adesc = smem_desc_sw128(a_addr);
                            const uint64_t bdesc = smem_desc_sw128(a_addr + LOOP_A_BYTES);
#pragma unroll
                            for (int k = 0; k < BK / 16; ++k)
                                tc_mma_bf16(tm_p, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kb | k) != 0);
                            tc_commit(&empty_bar[cur]);
                            cur = cur + 1 == S_lp ? 0 : cur + 1;
                        }
                        if (ok) { tc_commit(&acc_full[2]); ++acc_n[2]; }
                    }
                    if (ok && early) mma_L(0);
                }
            } else {
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_START);
                // utterances still decoding, counted by every CTA (they all take the same exit)
                {
                    int cnt = (e == 0 && ld_volatile_i32(&p.ctrl->next_utt) < p.n_utt) ? 1 : 0;   // utterances waiting for a row
                    for (int b = e; b < p.B; b += 128) cnt += t_new[b] < (len_new[b] & kSlotLenMask);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
                    if (lane == 0) s_red[warp - 2] = cnt;
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (e == 0) s_active = s_red[0] + s_red[1] + s_red[2] + s_red[3];
                }
                // Projection epilogue of the streaming mode.  The accumulator holds pred_proj[utterance (lane), np columns];
                // it goes through shared memory, and the z rows are then built by ALL epilogue threads: work item =
                // (utterance, window row), 2 x 16 bytes of enc_proj each, four items per thread and round with their
                // loads requested together.  (One thread per utterance, as the accumulator is laid out, left three
                // quarters of the threads idle for batches of 32 and took W dependent rounds of loads.)
                if (p.W > 4) {
                float* pst = stage_f;                                                   // [128][np] pred_proj + b_pred
                for (int i = i0; i < p.p_items; i += G) {
                    const int mt = i / p.hg_count, hg = i - mt * p.hg_count;
                    const int h0 = hg * p.np;
                    const int rows_here = min(128, p.B - mt * 128);
                    const int total = rows_here * p.W;
                    // this thread's first four items, requested before the accumulator is ready
                    uint4 ev[4][2];
                    int it_r[4], it_w[4], it_n[4];
                    auto fetch = [&](int base) {
                        int t[4], len[4], row[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int idx = base + k * 128 + e;
                            it_n[k] = 0; it_r[k] = 0; it_w[k] = 0;
                            t[k] = 0; len[k] = 0; row[k] = 0;
                            if (idx < total) {
                                it_r[k] = idx / p.W;
                                it_w[k] = idx - it_r[k] * p.W;
                                const int b = mt * 128 + it_r[k];
                                t[k] = t_new[b]; len[k] = len_new[b]; row[k] = row_new[b];
                            }
                        }
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int idx = base + k * 128 + e;
                            if (idx < total) {
                                it_n[k] = min(p.W, (len[k] & kSlotLenMask) - t[k]);   // <= 0 when the utterance is done
                                if (it_w[k] < it_n[k]) {
                                    const uint4* src = reinterpret_cast<const uint4*>(
                                        p.enc_proj + ((size_t)row[k] + t[k] + it_w[k]) * p.H + h0);
                                    ev[k][0] = src[0];
                                    ev[k][1] = src[1];
                                }
                            }
                        }
                    };
                    fetch(0);
                    if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_TOK);
                    const bool ready = __all_sync(0xffffffffu, mbar_wait(&acc_full[2], acc_n[2] & 1u, &s_abort));
                    tc_fence_after();
                    if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_ACC);
                    if (ready) {
                        float g[16];
                        tmem_ld16(tm_p + lane_off, g);
#pragma unroll
                        for (int j = 0; j < 16; ++j) pst[row_in_tile * 16 + j] = g[j] + p.b_pred[h0 + j];
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[2]);
                    ++acc_n[2];
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (ready) {
                        for (int base = 0; base < total; base += 512) {
                            if (base > 0) fetch(base);
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                if (it_n[k] <= 0) continue;            // outside the batch, or the utterance is done: nothing to write
                                uint4 o0 = make_uint4(0, 0, 0, 0), o1 = make_uint4(0, 0, 0, 0);
                                if (it_w[k] < it_n[k]) {
                                    const float* g = pst + it_r[k] * 16;
                                    const __nv_bfloat162* eb = reinterpret_cast<const __nv_bfloat162*>(&ev[k][0]);
                                    uint32_t wds[8];
#pragma unroll
                                    for (int c = 0; c < 8; ++c) {
                                        const float2 e2 = __bfloat1622float2(eb[c]);
                                        float z0 = e2.x + g[2 * c], z1 = e2.y + g[2 * c + 1];
                                        z0 = p.act == WIND_ACT_RELU ? fmaxf(z0, 0.f) : tanh_fast(z0);
                                        z1 = p.act == WIND_ACT_RELU ? fmaxf(z1, 0.f) : tanh_fast(z1);
                                        wds[c] = pack_bf16x2(z0, z1);
                                    }
                                    o0 = make_uint4(wds[0], wds[1], wds[2], wds[3]);
                                    o1 = make_uint4(wds[4], wds[5], wds[6], wds[7]);
                                }
                                uint4* dst = reinterpret_cast<uint4*>(p.z + ((size_t)(mt * 128 + it_r[k]) * p.W + it_w[k]) * p.H + h0);
                                dst[0] = o0;
                                dst[1] = o1;
                            }
                        }
                    }
                    asm volatile("bar.sync 1, 128;" ::: "memory");   // the staging arrays are reused by the CTA's next item
                    if (s_abort) break;                               // the same decision in all four warps
                }
                } else {
                // narrow windows: one thread per utterance (its accumulator lane), every load requested before the
                // accumulator is ready; the staging above would only add a block barrier
                for (int i = i0; i < p.p_items; i += G) {
                    const int mt = i / p.hg_count, hg = i - mt * p.hg_count;
                    const int b = mt * 128 + row_in_tile;
                    const int h0 = hg * p.np;
                    int t = 0, n = 0;
                    size_t row0 = 0;
                    if (b < p.B) {
                        t = t_new[b];
                        n = min(p.W, (len_new[b] & kSlotLenMask) - t);   // <= 0 when the utterance is done
                        row0 = (size_t)row_new[b] + t;                   // enc_proj row of the window's first frame
                    }
                    // the first rows of the window, requested before the accumulator is ready (np == 16)
                    uint4 ev[4][2];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (j < n) {
                            const uint4* src = reinterpret_cast<const uint4*>(p.enc_proj + (row0 + j) * p.H + h0);
                            ev[j][0] = src[0];
                            ev[j][1] = src[1];
                        }
                    }
                    if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_TOK);
                    const bool ready = __all_sync(0xffffffffu, mbar_wait(&acc_full[2], acc_n[2] & 1u, &s_abort));
                    tc_fence_after();
                    if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_ACC);
                    if (ready) {
                        for (int c0 = 0; c0 < n_tile; c0 += 16) {
                            float g[16];
                            tmem_ld16(tm_p + lane_off + (uint32_t)c0, g);
                            if (b < p.B && n > 0) {
#pragma unroll
                                for (int j = 0; j < 16; ++j) g[j] += p.b_pred[h0 + c0 + j];
                                for (int w0 = 0; w0 < p.W; w0 += 4) {
                                    if (w0 > 0 || c0 > 0) {
#pragma unroll
                                        for (int j = 0; j < 4; ++j) {
                                            if (w0 + j < n) {
                                                const uint4* src = reinterpret_cast<const uint4*>(
                                                    p.enc_proj + (row0 + w0 + j) * p.H + h0 + c0);
                                                ev[j][0] = src[0];
                                                ev[j][1] = src[1];
                                            }
                                        }
                                    }
#pragma unroll
                                    for (int j = 0; j < 4; ++j) {
                                        if (w0 + j < p.W) {
                                            uint4 o0 = make_uint4(0, 0, 0, 0), o1 = make_uint4(0, 0, 0, 0);
                                            if (w0 + j < n) {
                                                const __nv_bfloat162* eb = reinterpret_cast<const __nv_bfloat162*>(&ev[j][0]);
                                                uint32_t wds[8];
#pragma unroll
                                                for (int k = 0; k < 8; ++k) {
                                                    const float2 e2 = __bfloat1622float2(eb[k]);
                                                    float z0 = e2.x + g[2 * k], z1 = e2.y + g[2 * k + 1];
                                                    z0 = p.act == WIND_ACT_RELU ? fmaxf(z0, 0.f) : tanh_fast(z0);
                                                    z1 = p.act == WIND_ACT_RELU ? fmaxf(z1, 0.f) : tanh_fast(z1);
                                                    wds[k] = pack_bf16x2(z0, z1);
                                                }
                                                o0 = make_uint4(wds[0], wds[1], wds[2], wds[3]);
                                                o1 = make_uint4(wds[4], wds[5], wds[6], wds[7]);
                                            }
                                            uint4* dst = reinterpret_cast<uint4*>(p.z + ((size_t)b * p.W + w0 + j) * p.H + h0 + c0);
                                            dst[0] = o0;
                                            dst[1] = o1;
                                        }
                                    }
                                }
                            }
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[2]);
                    ++acc_n[2];
                    if (!ready) break;
                }
                }
                fence_proxy_async_all();
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_P, EV_EPI_DONE);
            }
            if (!grid_sync(TR_P)) goto done;
        }
        if (!(FULL && p.forced) && s_active == 0) break;
        if (!(FULL && p.forced) && step + 1 >= p.step_cap) { exit_status = WIND_ERR_INTERNAL; break; }
        ++step;

        // =====================================================================================
        // joint phase: window logits on tensor cores, per-row argmax in the epilogue
        // =====================================================================================
joint_only_entry:
        {
            const int n_tile = p.nj;
            const uint32_t z_bytes = (uint32_t)n_tile * BK * 2;
            unsigned long long* keys_cur = p.keys2 + (size_t)(step & 1) * p.rows_pad;
            if (RES && warp < 2) {
                // one box for the whole z tile, then every MMA back to back (A = W_out tile in tensor memory)
                if (lane == 0 && has_j) {
                    if (warp == 0) {
                        fence_proxy_async_all();
                        if constexpr (FULL) trace_event(p, 0, tr_n, step, TR_J, EV_FIRST_ISSUE);
                        for (int rg = j_first; rg < p.rg_count; rg += p.rg_stride) {
                            const bool ok = produce_one(&M.z3, rg * n_tile, (uint32_t)n_tile * (uint32_t)p.H * 2u);
                            if constexpr (FULL) trace_event(p, 0, tr_n, step, TR_J, EV_LAST_ISSUE);
                            if (!ok || !mma_part(0, tm_j + (uint32_t)n_tile, n_tile, p.kb_h / 2, p.kb_h, true)) break;
                        }
                        if constexpr (FULL) trace_event(p, 0, tr_n, step, TR_J, EV_COMMIT);
                    } else {
                        for (int rg = j_first; rg < p.rg_count; rg += p.rg_stride)
                            if (!mma_part(0, tm_j, n_tile, 0, p.kb_h / 2, true)) break;
                        if constexpr (FULL) trace_event(p, 1, tr_n, step, TR_J, EV_COMMIT);
                    }
                }
            } else if (!RES && warp == 0) {
                if (lane == 0) {
                    fence_proxy_async_all();
                    cur = 0;
                    bool ok = true;
                    if constexpr (FULL) trace_event(p, 0, tr_n, step, TR_J, EV_FIRST_ISSUE);
                    for (int i = cta; i < p.j_items && ok; i += G) {
                        const int rg = i / p.vt_count, vt = i - rg * p.vt_count;
                        for (int kb = 0; kb < p.kb_h; ++kb) {
                            uint8_t* dst = acquire(sb_j);
                            if (!dst) { ok = false; break; }
                            if (p.j_mode != J_STREAM) {
                                mbar_expect_tx(&full_bar[cur], z_bytes);
                                tma_load_2d(dst, &M.z, kb * BK, rg * n_tile, &full_bar[cur]);
                            } else {
                                mbar_expect_tx(&full_bar[cur], LOOP_A_BYTES + z_bytes);
                                tma_load_2d(dst, &M.w_out, kb * BK, vt * 128, &full_bar[cur]);
                                tma_load_2d(dst + LOOP_A_BYTES, &M.z, kb * BK, rg * n_tile, &full_bar[cur]);
                            }
                            cur = cur + 1 == S_j ? 0 : cur + 1;
                        }
                    }
                    if constexpr (FULL) trace_event(p, 0, tr_n, step, TR_J, EV_LAST_ISSUE);
                }
            } else if (!RES && warp == 1) {
                if (lane == 0) {
                    const uint32_t idesc = idesc_bf16(128, n_tile);
                    cur = 0;
                    bool ok = true;
                    if (p.j_mode == J_SMEM && has_j) ok = mbar_wait(&stat_bar, 0, &s_abort);
                    for (int i = cta; i < p.j_items && ok; i += G) {
                        if (!begin_acc(0)) { ok = false; break; }
                        for (int kb = 0; kb < p.kb_h; ++kb) {
                            if (!consume()) { ok = false; break; }
                            if (kb == 0) if constexpr (FULL) trace_event(p, 1, tr_n, step, TR_J, EV_FIRST_DATA);
                            const uint32_t st_addr = smem_u32(ring + (size_t)cur * sb_j);
                            if (p.j_mode == J_TMEM) {
                                const uint64_t bdesc = smem_desc_sw128(st_addr);
#pragma unroll
                                for (int k = 0; k < BK / 16; ++k)
                                    tc_mma_bf16_ts(tm_j, tmem_base + (uint32_t)(kb * (BK / 2) + k * 8), bdesc + (uint64_t)(k * 2), idesc,
                                                   (kb | k) != 0);
                            } else {
                                const uint64_t adesc =
                                    smem_desc_sw128(p.j_mode == J_SMEM ? smem_u32(stat + (size_t)kb * LOOP_A_BYTES) : st_addr);
                                const uint64_t bdesc = smem_desc_sw128(p.j_mode == J_SMEM ? st_addr : st_addr + LOOP_A_BYTES);
#pragma unroll
                                for (int k = 0; k < BK / 16; ++k)
                                    tc_mma_bf16(tm_j, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kb | k) != 0);
                            }
                            tc_commit(&empty_bar[cur]);
                            cur = cur + 1 == S_j ? 0 : cur + 1;
                        }
                        if (ok) { tc_commit(&acc_full[0]); ++acc_n[0]; if constexpr (FULL) trace_event(p, 1, tr_n, step, TR_J, EV_COMMIT); }
                    }
                }
            } else {
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_START);
                const int32_t* t_cur = p.t2 + (size_t)(step & 1) * p.B;
                for (int i = RES ? j_first : cta; i < (RES ? p.rg_count : p.j_items); i += RES ? p.rg_stride : G) {
                    const int rg = RES ? i : i / p.vt_count, vt = RES ? my_vt : i - rg * p.vt_count;
                    const int v = vt * 128 + row_in_tile;            // this thread's vocabulary entry
                    const bool v_ok = v < p.NV;
                    const float bias = v_ok ? p.b_out[v] : 0.f;
                    const bool ready = __all_sync(0xffffffffu, mbar_wait(&acc_full[0], acc_n[0] & 1u, &s_abort));
                    tc_fence_after();
                    if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_ACC);
                    if (ready) {
                        for (int c0 = RES ? 32 * sub : 0; c0 < n_tile; c0 += RES ? 64 : 32) {
                            float val[32];
                            tmem_ld16(tm_j + lane_off + (uint32_t)c0, val);
                            if (c0 + 16 < n_tile) {
                                tmem_ld16(tm_j + lane_off + (uint32_t)(c0 + 16), val + 16);
                            } else {
#pragma unroll
                                for (int j = 16; j < 32; ++j) val[j] = -INFINITY;
                            }
                            if (RES) {   // second accumulator copy (the other issuing thread's K blocks)
                                float more[16];
                                if (p.kb_h < 2) {   // a single K block: nothing was written to the first copy
#pragma unroll
                                    for (int j = 0; j < 32; ++j) val[j] = (j < 16 || c0 + 16 < n_tile) ? 0.f : val[j];
                                }
                                tmem_ld16(tm_j + lane_off + (uint32_t)(n_tile + c0), more);
#pragma unroll
                                for (int j = 0; j < 16; ++j) val[j] += more[j];
                                if (c0 + 16 < n_tile) {
                                    tmem_ld16(tm_j + lane_off + (uint32_t)(n_tile + c0 + 16), more);
#pragma unroll
                                    for (int j = 0; j < 16; ++j) val[16 + j] += more[j];
                                }
                            }
#pragma unroll
                            for (int j = 0; j < 32; ++j) val[j] = v_ok ? val[j] + bias : -INFINITY;
                            const int row = rg * n_tile + c0 + lane;      // the window row whose result this lane ends up with
                            if (FULL && p.logits_out) {
                                // teacher-forced evaluation: store the logits of the rows inside the window
                                bool row_ok = false;
                                if (row < p.rows && c0 + lane < n_tile) {
                                    const int b = row / p.W, w = row - b * p.W;
                                    row_ok = t_cur[b] + w < p.enc_len[b];
                                }
                                const uint32_t okmask = __ballot_sync(0xffffffffu, row_ok);
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (((okmask >> j) & 1u) && v_ok)
                                        p.logits_out[(size_t)(rg * n_tile + c0 + j) * p.NV + v] = val[j];
                            } else {
                                unsigned long long* key_dst = keys_cur;
                                if (FULL && p.window) {
                                    // window-based decoding: this warp's 32 vocabulary entries give, per row, a partial
                                    // (maximum, sum of exponentials) for the row's log-sum-exp; the blank's logit is
                                    // stored on its own and the blank leaves the maximum search
                                    float tmp[32];
#pragma unroll
                                    for (int j = 0; j < 32; ++j) tmp[j] = val[j];
                                    reduce_exchange<16, false>(tmp, lane);
                                    reduce_exchange<8, false>(tmp, lane);
                                    reduce_exchange<4, false>(tmp, lane);
                                    reduce_exchange<2, false>(tmp, lane);
                                    reduce_exchange<1, false>(tmp, lane);
                                    const float m_keep = tmp[0];           // this lane's row: maximum over the warp's 32 entries
#pragma unroll
                                    for (int j = 0; j < 32; ++j) {
                                        const float mj = __shfl_sync(0xffffffffu, m_keep, j);
                                        tmp[j] = val[j] > -INFINITY ? __expf(val[j] - mj) : 0.f;
                                    }
                                    reduce_exchange<16, true>(tmp, lane);
                                    reduce_exchange<8, true>(tmp, lane);
                                    reduce_exchange<4, true>(tmp, lane);
                                    reduce_exchange<2, true>(tmp, lane);
                                    reduce_exchange<1, true>(tmp, lane);
                                    const float s_keep = tmp[0];
                                    if (row < p.rows && c0 + lane < n_tile)
                                        p.jpart[(size_t)row * p.parts + vt * 4 + q] = make_float2(m_keep, s_keep);
                                    if (v == p.blank) {
#pragma unroll
                                        for (int j = 0; j < 32; ++j) {
                                            const int rj = rg * n_tile + c0 + j;
                                            if (rj < p.rows && c0 + j < n_tile) p.jblank[rj] = val[j];
                                            val[j] = -INFINITY;
                                        }
                                    }
                                    key_dst = p.nbkeys;
                                }
                                int id[32];
#pragma unroll
                                for (int j = 0; j < 32; ++j) id[j] = v;
                                argmax_exchange<16>(val, id, lane);
                                argmax_exchange<8>(val, id, lane);
                                argmax_exchange<4>(val, id, lane);
                                argmax_exchange<2>(val, id, lane);
                                argmax_exchange<1>(val, id, lane);
                                if (row < p.rows && c0 + lane < n_tile && val[0] > -INFINITY)
                                    atomicMax(&key_dst[row], pack_key(val[0], (uint32_t)id[0]));
                            }
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[0]);
                    ++acc_n[0];
                    if (!ready) break;
                }
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_EPI_DONE);
            }
            if (!jo && !grid_sync(TR_J)) goto done;
        }
        if (jo) {
            if (++jo_it < p.joint_iters) goto joint_only_entry;
            goto done;
        }
        if ((FULL && p.forced)) break;
        if (FULL && p.window) {
            // =================================================================================
            // window-based decoding: one warp per utterance turns the joint phase's per-row statistics into the
            // most probable (label, offset) pair of Eq. (1) and leaves it in the keys in the form the control step
            // reads (the chosen row carries its label, every other row the blank)
            // =================================================================================
            if (warp >= 2) {
                constexpr int n_ew = RES ? 8 : 4;
                const int ew = warp - 2;
                const int32_t* t_cur = p.t2 + (size_t)(step & 1) * p.B;
                unsigned long long* keys_cur = p.keys2 + (size_t)(step & 1) * p.rows_pad;
                const unsigned long long blank_key = pack_key(0.f, (uint32_t)p.blank);
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_START);
                // one utterance per CTA at a time; each epilogue warp takes the rows ew, ew + n_ew, ... of its window
                for (int b = cta; b < p.B; b += G) {
                    int t = 0, len = 0;
                    if (ew == 0) { t = t_cur[b]; len = p.enc_len[b]; }
                    for (int j = ew; j < p.W; j += n_ew) {
                        const size_t row = (size_t)b * p.W + j;
                        float bl = 0.f;
                        unsigned long long key = 0ull;
                        if (lane == 0) { bl = p.jblank[row]; key = p.nbkeys[row]; }
                        // the row's log-sum-exp from its partial (maximum, sum) pairs, spread over the lanes
                        float m = -INFINITY, sm = 0.f;
                        for (int k = lane; k < p.parts; k += 32) {
                            const float2 pr = p.jpart[row * p.parts + k];
                            if (pr.y > 0.f) {
                                if (pr.x > m) { sm = sm * __expf(m - pr.x) + pr.y; m = pr.x; }
                                else sm += pr.y * __expf(pr.x - m);
                            }
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
                            const float om = __shfl_xor_sync(0xffffffffu, m, o), os = __shfl_xor_sync(0xffffffffu, sm, o);
                            const float mx = fmaxf(m, om);
                            const float a = sm > 0.f ? sm * __expf(m - mx) : 0.f;
                            const float c = os > 0.f ? os * __expf(om - mx) : 0.f;
                            m = mx; sm = a + c;
                        }
                        if (lane == 0) {
                            const float lse = m + __logf(sm);
                            win_lpb[j] = bl - lse;
                            win_sc[j] = key != 0ull ? key_logit(key) - lse : -INFINITY;
                            win_key[j] = key;
                            p.nbkeys[row] = 0ull;
                        }
                    }
                    asm volatile("bar.sync 1, %0;" ::"n"(n_ew * 32) : "memory");
                    if (ew == 0) {
                        const int n = t < len ? min(p.W, len - t) : 0;
                        // lane j looks at rows j and j + 32: blank log-probabilities of the rows before each row
                        float lpb0 = lane < n ? win_lpb[lane] : 0.f, lpb1 = lane + 32 < n ? win_lpb[lane + 32] : 0.f;
                        float sc0 = lane < n ? win_sc[lane] : -INFINITY, sc1 = lane + 32 < n ? win_sc[lane + 32] : -INFINITY;
                        float incl0 = lpb0, incl1 = lpb1;
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) {
                            const float a0 = __shfl_up_sync(0xffffffffu, incl0, o), a1 = __shfl_up_sync(0xffffffffu, incl1, o);
                            if (lane >= o) { incl0 += a0; incl1 += a1; }
                        }
                        const float tot0 = __shfl_sync(0xffffffffu, incl0, 31), tot1 = __shfl_sync(0xffffffffu, incl1, 31);
                        sc0 += incl0 - lpb0;
                        sc1 += tot0 + incl1 - lpb1;
                        // first strict maximum in row order; "all blank" (tot0 + tot1) wins only when strictly larger
                        float top = sc0;
                        int pick = lane;
                        if (sc1 > top) { top = sc1; pick = lane + 32; }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
                            const float ot = __shfl_xor_sync(0xffffffffu, top, o);
                            const int op = __shfl_xor_sync(0xffffffffu, pick, o);
                            if (ot > top || (ot == top && op < pick)) { top = ot; pick = op; }
                        }
                        if (!(top > -INFINITY) || tot0 + tot1 > top) pick = -1;
                        for (int j = lane; j < n; j += 32) keys_cur[(size_t)b * p.W + j] = j == pick ? win_key[j] : blank_key;
                    }
                    if (b + G < p.B) asm volatile("bar.sync 1, %0;" ::"n"(n_ew * 32) : "memory");   // the arrays are reused
                }
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_EPI_DONE);
            }
            if (!grid_sync(TR_J)) goto done;
        }
    }
done:
    // an accumulator may still hold an unused early GEMM; nothing reads it, the MMAs have completed
    // before the last barrier (the issuing thread waited for none of them, so wait for them here)
    // (also when the kernel is being abandoned: a private flag, so that the wait is not cut short; it stays bounded)
    if (early && warp == 1 && lane == 0) {
        int gave_up = 0;
        mbar_wait(&acc_full[1], acc_n[1] & 1u ? 0u : 1u, &gave_up);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, LOOP_TMEM_COLS);
    }
    if (threadIdx.x == 0) {
        if (s_abort == 1) set_status(p.ctrl, WIND_ERR_TIMEOUT);
        if (cta == 0) {
            if (exit_status) set_status(p.ctrl, exit_status);
            p.ctrl->active = s_active;
            for (int k = 0; k < 3; ++k) p.ctrl->phase_cycles[k] = cyc[k];
            p.ctrl->loop_ns = (long long)(globaltimer_ns() - ns0);
        }
    }
}


// ---------------------------------------------------------------------------
// host side: tile plan, tensor maps, launch
// ---------------------------------------------------------------------------
static PFN_cuTensorMapEncodeTiled g_encode_loop = nullptr;
static std::mutex g_loop_mutex;
static int g_sm_count[64] = {};
static int g_smem_optin[64] = {};
static int g_attr_smem[64] = {};       // opt-in shared memory already granted to the streaming kernel, per device
static int g_loop_extra_arrivals = 0;
static LoopOptions g_loop_options = {1, -1, 4, -1};
int loop_set_extra_arrivals(int n) { int prev = g_loop_extra_arrivals; g_loop_extra_arrivals = n > 0 ? n : 0; return prev; }
void loop_set_options(const LoopOptions& o) { g_loop_options = o; }
LoopOptions loop_get_options() { return g_loop_options; }

static cudaError_t loop_device_info(int* sms, int* smem_optin, int* dev_out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_loop_mutex);
    if (!g_sm_count[dev]) {
        int n = 0, sm = 0;
        if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&sm, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess) return e;
        g_sm_count[dev] = n;
        g_smem_optin[dev] = sm;
    }
    *sms = g_sm_count[dev];
    *smem_optin = g_smem_optin[dev];
    if (dev_out) *dev_out = dev;
    return cudaSuccess;
}

cudaError_t loop_sm_count(int* sms) {
    int optin = 0;
    return loop_device_info(sms, &optin, nullptr);
}

static cudaError_t get_encode_loop() {
    std::lock_guard<std::mutex> lock(g_loop_mutex);
    if (g_encode_loop) return cudaSuccess;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    g_encode_loop = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(fn);
    return cudaSuccess;
}

// bf16 matrix [rows, cols] row-major, box = box_rows x 64 columns, 128-byte swizzle, zero fill outside
static cudaError_t loop_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode_loop(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// the same matrix seen as (64 columns, rows, cols / 64 blocks): one box of (64, box_rows, all blocks) lands in shared
// memory as cols / 64 consecutive K blocks of box_rows x 128 bytes, each with the 128-byte swizzle
static cudaError_t loop_map3(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    cuuint64_t dims[3] = {(cuuint64_t)BK, rows, cols / BK};
    cuuint64_t strides[2] = {cols * 2, (cuuint64_t)BK * 2};
    cuuint32_t box[3] = {(cuuint32_t)BK, box_rows, (cuuint32_t)(cols / BK)};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode_loop(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// Tile plan: how each phase's GEMM is cut into items (one item = one accumulator), sized so that a phase is one wave
// over the grid whenever the shapes allow.  A pure function of the shapes, the SM count and the opt-in shared memory
// per block (so that it can be checked on the host over many shapes); cudaErrorInvalidConfiguration when nothing fits.
cudaError_t loop_plan_for(const wind_model_t& m, int B, int W, int sms, int smem_optin, LoopPlan* out, bool refill) {
    LoopPlan pl{};
    LoopOptions opt = g_loop_options;
    if (refill) opt.dataflow = 0;   // rows are refilled by loop_kernel only
    if (sms < 1 || m.H % BK || m.P % BK || m.H < BK || m.P < BK || B < 1 || W < 1) return cudaErrorInvalidConfiguration;
    const int G = sms;
    const int rows = B * W;
    const int NV = m.V + 1;
    pl.grid = G;
    pl.kb_h = m.H / BK;
    pl.kb_p = m.P / BK;
    // joint: vocabulary tiles of 128 x window-row groups of nj
    pl.vt_count = (NV + 127) / 128;
    pl.nj = 256;
    for (int cand : {16, 32, 64, 96, 128, 160, 192, 224, 256}) {
        if ((long long)pl.vt_count * ((rows + cand - 1) / cand) <= G) { pl.nj = cand; break; }
    }
    pl.rg_count = (rows + pl.nj - 1) / pl.nj;
    pl.j_items = pl.vt_count * pl.rg_count;
    // projection: utterance tiles of 128 x H slices of np, placed at the far end of the grid
    pl.mt_count = (B + 127) / 128;
    pl.np = 16;
    pl.hg_count = m.H / pl.np;
    pl.p_items = pl.mt_count * pl.hg_count;
    // decoder: utterance tiles of 128 x unit groups of ul (4 gates x `slots` rows per item), on the
    // CTAs the projection leaves free when there are enough of them
    int free_ctas = G - pl.p_items;
    if (free_ctas < G / 2) free_ctas = G;
    int groups_wanted = free_ctas / pl.mt_count;
    if (groups_wanted < 1) groups_wanted = 1;
    pl.ul = (m.P + groups_wanted - 1) / groups_wanted;
    if (pl.ul > 64) pl.ul = 64;
    pl.slots = 8;
    while (pl.slots < pl.ul) pl.slots *= 2;
    pl.ug_count = (m.P + pl.ul - 1) / pl.ul;
    pl.l_items = pl.mt_count * pl.ug_count;
    pl.l_early = pl.l_items <= G;
    // where the joint's W_out tile lives, tensor-memory columns, shared-memory ring
    const int budget = smem_optin - 4096 - 1024;   // static shared memory of the kernels, 1 KB alignment slack
    if (budget < 32768) return cudaErrorInvalidConfiguration;
    const uint32_t small_ops = (uint32_t)(4 * pl.slots > pl.np ? 4 * pl.slots : pl.np) * BK * 2;
    pl.stage_lp = LOOP_A_BYTES + (small_ops + 1023u) / 1024u * 1024u;
    const uint32_t stat_bytes = (uint32_t)pl.kb_h * LOOP_A_BYTES;
    const bool one_wave = pl.j_items <= G;
    const bool tmem_fits = m.H / 2 + pl.nj + 4 * pl.slots + pl.np <= (int)LOOP_TMEM_COLS;
    const bool smem_fits = pl.nj <= 128 && (long long)stat_bytes + 3ll * pl.stage_lp <= budget;
    pl.j_mode = one_wave && tmem_fits ? J_TMEM : (one_wave && smem_fits ? J_SMEM : J_STREAM);
    {   // a forced placement (wind_set_loop_options) is taken when it is feasible
        const int want = opt.joint_placement;
        if (want == J_STREAM || (want == J_SMEM && one_wave && smem_fits) || (want == J_TMEM && one_wave && tmem_fits)) pl.j_mode = want;
    }
    pl.stat_bytes = pl.j_mode == J_SMEM ? stat_bytes : 0;
    pl.stage_j = ((pl.j_mode == J_STREAM ? LOOP_A_BYTES : 0u) + (uint32_t)pl.nj * BK * 2 + 1023u) / 1024u * 1024u;
    // behind the ring: staging of the projection epilogue (pred_proj of a 128-utterance tile, np = 16 columns)
    const uint32_t p_staging = 128u * (uint32_t)pl.np * 4u;
    // (this mode's kernels have 1.6 KB of static shared memory, not the 4 KB the budget sets aside: half of the difference goes to the ring)
    const long long ring = (long long)budget + 2048 - pl.stat_bytes - p_staging;
    pl.stages_lp = (int)(ring / pl.stage_lp);
    pl.stages_j = (int)(ring / pl.stage_j);
    if (pl.stages_lp > LOOP_MAX_STAGES) pl.stages_lp = LOOP_MAX_STAGES;
    if (pl.stages_j > LOOP_MAX_STAGES) pl.stages_j = LOOP_MAX_STAGES;
    bool streaming_ok = pl.stages_lp >= 2 && pl.stages_j >= 2;
    pl.tm_j = pl.j_mode == J_TMEM ? m.H / 2 : 0;
    pl.tm_l = pl.tm_j + pl.nj;
    pl.tm_p = pl.tm_l + 4 * pl.slots;
    if (pl.tm_p + pl.np > (int)LOOP_TMEM_COLS) streaming_ok = false;
    const uint32_t ring_lp = (uint32_t)(pl.stages_lp > 0 ? pl.stages_lp : 0) * pl.stage_lp, ring_j = (uint32_t)(pl.stages_j > 0 ? pl.stages_j : 0) * pl.stage_j;
    pl.stage_off = pl.stat_bytes + (ring_lp > ring_j ? ring_lp : ring_j);
    pl.smem_bytes = pl.stage_off + p_staging + 1024;

    // Resident-weights mode (one or two LSTM layers): the W_out tile of a CTA in tensor memory, W_hh in tiles of 4 gates x
    // 16 units and W_pred in tiles of 64 rows in the shared memory of disjoint CTA sets, for the whole decode; per step a
    // CTA fetches only its utterance group's rows of the state, as one box, and builds the joint's operand in place.
    // Its joint: every CTA keeps one vocabulary tile; G / vt_count CTAs share a tile and take one row group each per
    // wave.  Row-group sizes are tried in order of preference -- the smallest that needs one wave, else from the largest
    // down (fewest waves, at most four) -- until the whole plan fits shared and tensor memory.
    const int per_wave = pl.vt_count <= G ? G / pl.vt_count : 0;
    int cands[5], n_cands = 0;
    {
        const int max_waves = opt.max_joint_waves >= 1 && opt.max_joint_waves <= 4 ? opt.max_joint_waves : 4;
        int one = 0;
        for (int cand : {16, 32, 64, 96})
            if (per_wave >= 1 && ((rows + cand - 1) / cand + per_wave - 1) / per_wave == 1) { one = cand; break; }
        if (one) cands[n_cands++] = one;
        for (int cand : {96, 64, 32, 16})
            if (per_wave >= 1 && cand != one && ((rows + cand - 1) / cand + per_wave - 1) / per_wave <= max_waves && !one)
                cands[n_cands++] = cand;
    }
    bool resident_done = false;
    for (int ci = 0; ci < n_cands && !resident_done; ++ci) {
        const int r_nj = cands[ci];
        if (!(m.L <= 2 && m.H / 2 + 2 * r_nj <= (int)LOOP_TMEM_COLS && opt.resident != 0)) continue;
        LoopPlan r = pl;
        r.nj = r_nj;
        r.rg_count = (rows + r_nj - 1) / r_nj;
        r.j_items = r.vt_count * r.rg_count;
        r.rg_stride = per_wave;
        const int l_sets = m.L == 2 ? 3 : 1;   // layer 0; with two layers also layer 1's input and recurrent halves
        r.ut_count = m.P / 16;
        r.ht_count = m.H / 64;
        bool found = false;
        for (int nl : {16, 32, 64, 128}) {
            for (int npr : {16, 32, 64, 128}) {
                const int ql = (B + nl - 1) / nl, qp = (B + npr - 1) / npr;
                if (l_sets * r.ut_count * ql + r.ht_count * qp <= G) {
                    r.nl = nl; r.np = npr; r.ql_count = ql; r.qp_count = qp;
                    found = true;
                    break;
                }
            }
            if (found) break;
        }
        if (!found) continue;
        // Which resident kernel: the one with grid barriers between the phases, or the one in which CTAs hand their
        // results on through arrival counters and stamped data.  Measured on B200: the second is ahead while a lock step
        // is mostly latency (config 3's model with 1 / 16 / 64 utterances: 12.1 / 13.4 / 14.8 against 13.2 / 13.9 / 15.4 us per
        // lock step), the first once every CTA has work in every phase (128 utterances: 16.7 against 17.6 us).
        r.dataflow = opt.dataflow >= 0 ? (opt.dataflow != 0) : (B <= (m.L == 1 ? kDataflowMaxBatch : kDataflowMaxBatch2));
        if (NV > (1 << 20)) r.dataflow = 0;    // labels take 20 bits of a stamped key slot
        auto up = [](uint32_t x) { return (x + 1023u) / 1024u * 1024u; };
        if (!r.dataflow) {
            // shared memory of a CTA: [weight tile][operand buffer][epilogue staging]; the buffer holds the step's one
            // operand box (the joint's z rows, or the state rows) and, in CTAs with a W_pred tile, behind the state box
            // the prefetched enc_proj rows of their first 256 z rows
            const uint32_t staging = r.np > 64 ? (uint32_t)r.np * 68u * 4u : 17408u;
            const uint32_t tile = (uint32_t)r.kb_p * 64u * BK * 2u;
            uint32_t buf = (uint32_t)r.nj * (uint32_t)m.H * 2u;
            if ((uint32_t)r.nl * m.P * 2u > buf) buf = (uint32_t)r.nl * m.P * 2u;
            const uint32_t stash_rows = (uint32_t)(r.np * W < 256 ? r.np * W : 256);
            if ((uint32_t)r.np * m.P * 2u + stash_rows * 128u > buf) buf = (uint32_t)r.np * m.P * 2u + stash_rows * 128u;
            buf = up(buf);
            r.resident = 1;
            r.j_mode = J_TMEM;
            r.stat_bytes = tile;
            r.buf_off = tile;
            r.z_off = r.z_off_p = tile;
            r.stage_off = tile + buf;
            r.smem_bytes = tile + buf + staging + 1024;
        } else {
        // shared memory of a CTA: [weight tile][state box | joint operand][epilogue staging].  The joint's operand
        // (nj rows x H) shares the state box's memory where a CTA needs both; the CTAs with a W_pred tile (smaller box)
        // get an operand buffer of their own when it fits, so that they can start on the next window a slot earlier.
        // epilogue staging: 64 utterances x 4 gates x 16 units (+ their tokens) in the decoder slot, np utterances x
        // (64 + 4 padding) pred_proj values in the projection slot
        const uint32_t staging = r.np > 64 ? (uint32_t)r.np * 68u * 4u : 17408u;
        const uint32_t tile = (uint32_t)r.kb_p * 64u * BK * 2u;
        const uint32_t box_l = up((uint32_t)r.nl * m.P * 2u), box_p = up((uint32_t)r.np * m.P * 2u);
        const uint32_t zb = up((uint32_t)r.nj * (uint32_t)m.H * 2u);
        const uint32_t end_l = tile + (box_l > zb ? box_l : zb);
        const uint32_t end_p_own = tile + box_p + zb, end_p_shared = tile + (box_p > zb ? box_p : zb);
        const bool own = (long long)(end_l > end_p_own ? end_l : end_p_own) + staging <= (long long)budget;
        const uint32_t end_p = own ? end_p_own : end_p_shared;
        r.resident = 1;
        r.j_mode = J_TMEM;
        r.stat_bytes = tile;
        r.buf_off = tile;
        r.z_off = tile;
        r.z_off_p = own ? tile + box_p : tile;
        r.stage_off = end_l > end_p ? end_l : end_p;
        r.smem_bytes = r.stage_off + staging + 1024;
        }
        r.stages_lp = r.stages_j = 1;
        r.stage_lp = r.stage_j = 0;
        r.tm_j = m.H / 2;
        r.tm_l = r.tm_p = r.tm_j + 2 * r.nj;   // two copies of the joint accumulator, then decoder / projection
        r.l_items = r.ut_count * r.ql_count;
        r.p_items = r.ht_count * r.qp_count;
        // CTAs that hold no decoder or projection tile record the steps (outputs, counters, next frame), 64
        // utterances each, so that no L CTA carries that work between its control step and its cell update
        r.w_first = l_sets * r.l_items;
        r.w_count = (B + 63) / 64;
        if (r.w_first + r.w_count + r.p_items > G) r.w_count = 0;
        r.l_early = 1;
        const int acc_cols = r.nl > 2 * r.np ? r.nl : 2 * r.np;
        if ((long long)r.smem_bytes <= (long long)budget + 1024 && r.tm_l + acc_cols <= (int)LOOP_TMEM_COLS) {
            pl = r;
            resident_done = true;
        }
    }
    if (!resident_done && !streaming_ok) return cudaErrorInvalidConfiguration;
    *out = pl;
    return cudaSuccess;
}

cudaError_t loop_plan(const Call& c, LoopPlan* out) {
    int sms = 0, smem_optin = 0;
    cudaError_t e = loop_device_info(&sms, &smem_optin, nullptr);
    if (e != cudaSuccess) return e;
    return loop_plan_for(c.m, c.B, c.W, sms, smem_optin, out, c.N > 0);
}

// whether the loop kernels have a plan for these shapes on the current device
bool loop_plan_ok(const wind_model_t& m, int B, int W) {
    int sms = 0, smem_optin = 0;
    if (loop_device_info(&sms, &smem_optin, nullptr) != cudaSuccess) return false;
    LoopPlan pl;
    return loop_plan_for(m, B, W, sms, smem_optin, &pl) == cudaSuccess;
}

static thread_local LoopMaps t_loop_maps;
static thread_local LoopPlan t_loop_plan;

cudaError_t loop_prepare(Call& c) {
    cudaError_t e = get_encode_loop();
    if (e != cudaSuccess) return e;
    LoopPlan& pl = t_loop_plan;
    if ((e = loop_plan(c, &pl)) != cudaSuccess) return e;
    LoopMaps& M = t_loop_maps;
    const wind_model_t& m = c.m;
#define WIND_MAP(call_) do { e = (call_); if (e != cudaSuccess) return e; } while (0)
    if (pl.resident) {
        WIND_MAP(loop_map(&M.w_hh_r, c.w_hh[0], 4ull * m.P, m.P, 16));
        WIND_MAP(loop_map(&M.w_pred_r, m.w_pred, m.H, m.P, 64));
        if (m.L == 2) {
            WIND_MAP(loop_map(&M.w_ih1_r, c.w_ih[1], 4ull * m.P, m.P, 16));
            WIND_MAP(loop_map(&M.w_hh1_r, c.w_hh[1], 4ull * m.P, m.P, 16));
        }
        for (int par = 0; par < 2; ++par) {
            WIND_MAP(loop_map3(&M.hb_l3[par], c.hb(par, 0), c.lay.Bpad, m.P, pl.nl));
            if (m.L == 2) WIND_MAP(loop_map3(&M.hb_l3_1[par], c.hb(par, 1), c.lay.Bpad, m.P, pl.nl));
            WIND_MAP(loop_map3(&M.hb_p3[par], c.hb(par, m.L - 1), c.lay.Bpad, m.P, pl.np));
        }
        if (!pl.dataflow) WIND_MAP(loop_map3(&M.z3, c.z(), (uint64_t)c.lay.rows_pad, m.H, pl.nj));
    } else {
        WIND_MAP(loop_map(&M.w_out, m.w_out, (uint64_t)m.V + 1, m.H, 128));
        WIND_MAP(loop_map(&M.z, c.z(), (uint64_t)c.lay.rows_pad, m.H, pl.nj));
        WIND_MAP(loop_map(&M.w_pred, m.w_pred, m.H, m.P, pl.np));
        for (int l = 0; l < m.L; ++l) {
            if (l > 0) WIND_MAP(loop_map(&M.w_ih[l], c.w_ih[l], 4ull * m.P, m.P, pl.slots));
            WIND_MAP(loop_map(&M.w_hh[l], c.w_hh[l], 4ull * m.P, m.P, pl.slots));
            for (int par = 0; par < 2; ++par) WIND_MAP(loop_map(&M.hb[par][l], c.hb(par, l), c.lay.Bpad, m.P, 128));
        }
    }
#undef WIND_MAP
    if (pl.resident && pl.dataflow) return loop_res_set_smem((int)pl.smem_bytes);
    int sms = 0, optin = 0, dev = 0;
    if ((e = loop_device_info(&sms, &optin, &dev)) != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(g_loop_mutex);
    if ((int)pl.smem_bytes > g_attr_smem[dev]) {
        for (const void* fn : {(const void*)loop_kernel<false, false>, (const void*)loop_kernel<false, true>,
                               (const void*)loop_kernel<true, false>, (const void*)loop_kernel<true, true>}) {
            e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem_bytes);
            if (e != cudaSuccess) return e;
        }
        g_attr_smem[dev] = (int)pl.smem_bytes;
    }
    return cudaSuccess;
}

cudaError_t tc_loop(const Call& c, const int32_t* prefix, int U, const int32_t* prefix_len, float* logits_out,
                    int trace_step) {
    const LoopPlan& pl = t_loop_plan;
    LoopParams p{};
    p.ctrl = c.ctrl();
    p.B = c.B; p.T = c.T; p.W = c.W; p.S = c.S; p.max_out = c.max_out;
    p.H = c.m.H; p.P = c.m.P; p.NV = c.m.V + 1; p.blank = c.m.blank_id; p.act = c.m.act; p.L = c.m.L;
    p.rows = c.B * c.W; p.rows_pad = c.lay.rows_pad; p.Bpad = c.lay.Bpad;
    long long cap = (long long)c.T * (c.S + 1) + 2;
    if (c.N > 0) cap = (cap + 1) * c.N;    // refilled rows: at worst one utterance after the other
    p.step_cap = cap > 0x7fffffff ? 0x7fffffff : (int)cap;
    p.nj = pl.nj; p.vt_count = pl.vt_count; p.rg_count = pl.rg_count; p.j_items = pl.j_items; p.j_mode = pl.j_mode;
    p.rg_stride = pl.rg_stride > 0 ? pl.rg_stride : 1;
    p.tm_j = pl.tm_j; p.tm_l = pl.tm_l; p.tm_p = pl.tm_p; p.l_early = pl.l_early;
    p.resident = pl.resident; p.nl = pl.nl; p.ut_count = pl.ut_count > 0 ? pl.ut_count : 1; p.ht_count = pl.ht_count > 0 ? pl.ht_count : 1;
    p.w_first = pl.w_first; p.w_count = pl.resident ? pl.w_count : 0;
    p.ql_count = pl.ql_count; p.qp_count = pl.qp_count; p.buf_off = pl.buf_off; p.stage_off = pl.stage_off;
    p.z_off = pl.z_off; p.z_off_p = pl.z_off_p;
    p.stage_lp = pl.stage_lp; p.stage_j = pl.stage_j; p.stages_lp = pl.stages_lp; p.stages_j = pl.stages_j;
    p.slots = pl.slots; p.ul = pl.ul; p.ug_count = pl.ug_count; p.mt_count = pl.mt_count; p.l_items = pl.l_items;
    p.np = pl.np; p.hg_count = pl.hg_count; p.p_items = pl.p_items;
    p.kb_h = pl.kb_h; p.kb_p = pl.kb_p;
    p.stat_bytes = pl.stat_bytes;
    p.slot_len2 = c.slot(); p.slot_row2 = c.slot() + 2 * (size_t)c.B; p.slot_utt = c.slot() + 4 * (size_t)c.B;
    p.slot_pos = c.slot() + 5 * (size_t)c.B; p.n_utt = c.N > 0 ? c.N : c.B;
    p.enc_len = c.enc_len; p.t2 = c.t(); p.t_pub = c.t_pub(); p.count = c.count(); p.emit_tok = c.emit_tok(); p.keys2 = c.keys();
    p.out_tokens = c.out_tokens; p.out_frames = c.out_frames; p.out_len = c.out_len;
    p.c_state = c.c(); p.dh = c.dh(); p.hb = c.hb(0, 0); p.z = c.z(); p.enc_proj = (const __nv_bfloat16*)c.enc_proj(); p.g0 = c.g0();
    for (int l = 0; l < c.m.L; ++l) { p.b_ih[l] = c.b_ih[l]; p.b_hh[l] = c.b_hh[l]; }
    p.b_pred = c.m.b_pred; p.b_out = c.m.b_out; p.w_out = (const __nv_bfloat16*)c.m.w_out;
    p.forced = logits_out != nullptr; p.prefix = prefix; p.U = U; p.prefix_len = prefix_len; p.logits_out = logits_out;
    p.trace = trace_step >= -1 ? c.trace() : nullptr; p.trace_step = trace_step;
    p.extra_arrivals = g_loop_extra_arrivals;
    p.window = c.mode == WIND_MODE_WINDOW && !logits_out;
    p.nbkeys = c.keys() + 2 * (size_t)c.lay.rows_pad; p.jpart = c.jpart(); p.jblank = c.jblank(); p.parts = 4 * pl.vt_count;
    p.flags = c.flags(); p.pred_pub = c.pred_pub(); p.kslot = c.kslot();
    p.joint_iters = c.joint_iters;
    const bool full = p.forced || p.window || p.trace || p.joint_iters > 0;
    if (pl.resident && pl.dataflow) return loop_res_launch(t_loop_maps, p, pl.grid, pl.smem_bytes, full, c.stream);
    void* args[2] = {(void*)&t_loop_maps, (void*)&p};
    const void* fn = pl.resident ? (full ? (const void*)loop_kernel<true, true> : (const void*)loop_kernel<true, false>)
                                 : (full ? (const void*)loop_kernel<false, true> : (const void*)loop_kernel<false, false>);
    return cudaLaunchCooperativeKernel(fn, dim3((unsigned)pl.grid), dim3(pl.resident ? LOOP_THREADS_RES : LOOP_THREADS), args, pl.smem_bytes,
                                       c.stream);
}

}  // namespace wind
