// The decoding loop of the bf16 path as ONE persistent cooperative kernel (sm_100a): streaming mode, and the host
// side of both modes (tile plan, tensor maps, launch).
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
// This file's kernel is the streaming mode: weights flow through a TMA ring every step (large vocabularies,
// more than two LSTM layers, batches whose tiles outnumber the SMs).  Shapes whose weight tiles fit on chip run
// the resident-weights kernel of wind_loop_res.cu instead (no grid barriers, operands built in place).
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
// FULL: the kernel also carries teacher forcing with the logits store, window-based decoding and the timeline; the
// plain decode runs the variant without them (a smaller instruction footprint: the loop is sensitive to it).
template <bool FULL>
__global__ void __launch_bounds__(LOOP_THREADS, 1) loop_kernel(const __grid_constant__ LoopMaps M, const LoopParams p) {
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
        for (int s = 0; s < LOOP_MAX_STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&stat_bar, 1);
        for (int k = 0; k < 3; ++k) {
            mbar_init(&acc_full[k], 1);
            mbar_init(&acc_empty[k], 4);   // one arrival per epilogue warp
        }
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(&tmem_slot, LOOP_TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    const uint32_t tm_j = tmem_base + (uint32_t)p.tm_j, tm_l = tmem_base + (uint32_t)p.tm_l, tm_p = tmem_base + (uint32_t)p.tm_p;

    const int e = threadIdx.x - 64;            // epilogue thread: 0..127 (warps 2..5)
    const int q = warp & 3;                    // tensor-memory lane quadrant of this warp
    const int row_in_tile = q * 32 + lane;     // the tensor-memory lane (accumulator row) of this thread
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    // joint items of this CTA: items cta, cta + G, ... of the (row group, vocabulary tile) list
    const bool has_j = cta < p.j_items;
    const int my_vt = cta % p.vt_count;        // vocabulary tile of this CTA's joint item when it has exactly one

    // ----- the joint's W_out tile, loaded once when every CTA owns one joint item -----
    if (p.j_mode == J_SMEM && has_j && threadIdx.x == 0) {
        mbar_expect_tx(&stat_bar, (uint32_t)p.kb_h * LOOP_A_BYTES);
        for (int kb = 0; kb < p.kb_h; ++kb) tma_load_2d(stat + (size_t)kb * LOOP_A_BYTES, &M.w_out, kb * BK, my_vt * 128, &stat_bar);
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
            if constexpr (FULL) trace_phase_done(p, step, phase_kind);   // when every CTA finished its part of the phase
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
                    const int len = p.enc_len[b];
                    const bool writer = ug == 0;
                    int cnt = 0, pos = 0;
                    if (writer) { cnt = p.count[b]; pos = p.out_len[b]; }
                    unsigned long long kk[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) kk[j] = j < p.W ? keys_cur[(size_t)b * p.W + j] : 0ull;
                    if (t < len) {
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
                                    p.out_tokens[(size_t)b * p.max_out + pos] = label;
                                    p.out_frames[(size_t)b * p.max_out + pos] = t;
                                    p.out_len[b] = pos + 1;
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
                    } else if (writer) {
                        t_nxt[b] = t;
                    }
                    if (writer) p.emit_tok[b] = tok;
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

    // ----- before the loop: layer 0's GEMM on the initial (zero) state -----
    if (early) {
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
        for (int l = 0; l < p.L; ++l) {
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
            if (early) {
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
            const int i0 = p.p_items <= G ? G - 1 - cta : cta;   // projection items start at the far end of the grid
            if (warp == 0) {
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
                    int cnt = 0;
                    for (int b = e; b < p.B; b += 128) cnt += t_new[b] < p.enc_len[b];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
                    if (lane == 0) s_red[warp - 2] = cnt;
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (e == 0) s_active = s_red[0] + s_red[1] + s_red[2] + s_red[3];
                }
                for (int i = i0; i < p.p_items; i += G) {
                    const int mt = i / p.hg_count, hg = i - mt * p.hg_count;
                    const int b = mt * 128 + row_in_tile;
                    const int h0 = hg * p.np;
                    int t = 0, n = 0;
                    if (b < p.B) {
                        t = t_new[b];
                        n = min(p.W, p.enc_len[b] - t);   // <= 0 when the utterance is done
                    }
                    // the first rows of the window, requested before the accumulator is ready (np == 16)
                    uint4 ev[4][2];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (j < n) {
                            const uint4* src = reinterpret_cast<const uint4*>(p.enc_proj + ((size_t)b * p.T + t + j) * p.H + h0);
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
                                                    p.enc_proj + ((size_t)b * p.T + t + w0 + j) * p.H + h0 + c0);
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
        {
            const int n_tile = p.nj;
            const uint32_t z_bytes = (uint32_t)n_tile * BK * 2;
            unsigned long long* keys_cur = p.keys2 + (size_t)(step & 1) * p.rows_pad;
            if (warp == 0) {
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
            } else if (warp == 1) {
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
                for (int i = cta; i < p.j_items; i += G) {
                    const int rg = i / p.vt_count, vt = i - rg * p.vt_count;
                    const bool ready = __all_sync(0xffffffffu, mbar_wait(&acc_full[0], acc_n[0] & 1u, &s_abort));
                    tc_fence_after();
                    if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_ACC);
                    if (ready) joint_epilogue_item<false, FULL>(p, tm_j, lane_off, lane, q, 0, row_in_tile, rg, vt, n_tile, t_cur, keys_cur);
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[0]);
                    ++acc_n[0];
                    if (!ready) break;
                }
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_EPI_DONE);
            }
            if (!grid_sync(TR_J)) goto done;
        }
        if ((FULL && p.forced)) break;
        if (FULL && p.window) {
            // =================================================================================
            // window-based decoding: one warp per utterance turns the joint phase's per-row statistics into the
            // most probable (label, offset) pair of Eq. (1) and leaves it in the keys in the form the control step
            // reads (the chosen row carries its label, every other row the blank)
            // =================================================================================
            if (warp >= 2) {
                const int32_t* t_cur = p.t2 + (size_t)(step & 1) * p.B;
                unsigned long long* keys_cur = p.keys2 + (size_t)(step & 1) * p.rows_pad;
                if (e == 0) if constexpr (FULL) trace_event(p, 2, tr_n, step, TR_J, EV_START);
                window_decision<4>(p, cta, G, warp - 2, lane, t_cur, keys_cur, win_lpb, win_sc, win_key);
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
static LoopOptions g_loop_options = {1, -1, 4};
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
cudaError_t loop_plan_for(const wind_model_t& m, int B, int W, int sms, int smem_optin, LoopPlan* out) {
    LoopPlan pl{};
    const LoopOptions opt = g_loop_options;
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
    const long long ring = (long long)budget - pl.stat_bytes;
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
    pl.smem_bytes = pl.stat_bytes + (ring_lp > ring_j ? ring_lp : ring_j) + 1024;

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
        if (!(m.L <= 2 && m.H / 2 + 2 * r_nj <= (int)LOOP_TMEM_COLS && opt.resident != 0 && NV <= (1 << 20))) continue;   // (labels take 20 bits of a key slot)
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
        // shared memory of a CTA: [weight tile][state box | joint operand][epilogue staging].  The joint's operand
        // (nj rows x H) shares the state box's memory where a CTA needs both; the CTAs with a W_pred tile (smaller box)
        // get an operand buffer of their own when it fits, so that they can start on the next window a slot earlier.
        auto up = [](uint32_t x) { return (x + 1023u) / 1024u * 1024u; };
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
    return loop_plan_for(c.m, c.B, c.W, sms, smem_optin, out);
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
    if (pl.resident) return loop_res_set_smem((int)pl.smem_bytes);
    int sms = 0, optin = 0, dev = 0;
    if ((e = loop_device_info(&sms, &optin, &dev)) != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(g_loop_mutex);
    if ((int)pl.smem_bytes > g_attr_smem[dev]) {
        for (const void* fn : {(const void*)loop_kernel<false>, (const void*)loop_kernel<true>}) {
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
    const bool full = p.forced || p.window || p.trace;
    if (pl.resident) return loop_res_launch(t_loop_maps, p, pl.grid, pl.smem_bytes, full, c.stream);
    void* args[2] = {(void*)&t_loop_maps, (void*)&p};
    const void* fn = full ? (const void*)loop_kernel<true> : (const void*)loop_kernel<false>;
    return cudaLaunchCooperativeKernel(fn, dim3((unsigned)pl.grid), dim3(LOOP_THREADS), args, pl.smem_bytes, c.stream);
}

}  // namespace wind
