// Device-side pieces shared by the two persistent decoding-loop kernels (streaming mode in wind_loop.cu,
// resident-weights mode in wind_loop_res.cu): memory-ordering wrappers, tensor-memory loads and stores, the
// transposing warp reductions of the joint's epilogue, the joint's epilogue itself, the timeline records.
#pragma once

#include "wind_internal.cuh"
#include "wind_loop.cuh"
#include "wind_ptx.cuh"

namespace wind {

constexpr int LOOP_THREADS = 192;       // streaming mode: TMA warp, MMA warp, 4 epilogue warps
constexpr int LOOP_THREADS_RES = 320;   // resident-weights mode: 8 epilogue warps (two per tensor-memory lane quadrant)
constexpr uint32_t LOOP_TMEM_COLS = 512;

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_volatile_i32(const int* p) {
    int v;
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// release: every write this thread has made or observed is visible device-wide before the counter moves
__device__ __forceinline__ void red_relaxed_add(uint32_t* p, uint32_t v) {
    asm volatile("red.relaxed.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_release_add(uint32_t* p, uint32_t v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// generic-proxy writes of this thread become visible to later async-proxy (TMA) reads
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// 32 lanes x 8 consecutive columns
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
// 32 lanes x 16 consecutive columns, registers -> tensor memory
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
        "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D[tmem] (+)= A[tmem] * B[smem]^T: A rows on lanes, two bf16 K elements per 32-bit column
__device__ __forceinline__ void tc_mma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(tmem_d),
        "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

enum { J_STREAM = 0, J_SMEM = 1, J_TMEM = 2 };   // where the joint's W_out tile lives

// z = act(e + g) on two bf16 pairs at once: one rounding for the sum (fused multiply-add with 1), then ReLU or tanh
__device__ __forceinline__ uint32_t act_add_bf16x2(uint32_t e, uint32_t g, int act) {
    const __nv_bfloat162 one = __floats2bfloat162_rn(1.f, 1.f);
    __nv_bfloat162 s = __hfma2(*reinterpret_cast<const __nv_bfloat162*>(&e), one, *reinterpret_cast<const __nv_bfloat162*>(&g));
    uint32_t r;
    if (act == WIND_ACT_RELU) {
        s = __hmax2(s, __floats2bfloat162_rn(0.f, 0.f));
        r = *reinterpret_cast<uint32_t*>(&s);
    } else {
        asm("tanh.approx.bf16x2 %0, %1;" : "=r"(r) : "r"(*reinterpret_cast<uint32_t*>(&s)));
    }
    return r;
}

// One stage of the exchange that turns "every lane holds 2*HALF columns" into "every lane holds HALF
// columns, reduced over lane pairs": lanes with bit HALF set keep the upper columns.
template <int HALF>
__device__ __forceinline__ void argmax_exchange(float* v, int* id, int lane) {
    const bool up = (lane & HALF) != 0;
#pragma unroll
    for (int c = 0; c < HALF; ++c) {
        const float sv = up ? v[c] : v[c + HALF];
        const int si = up ? id[c] : id[c + HALF];
        const float kv = up ? v[c + HALF] : v[c];
        const int ki = up ? id[c + HALF] : id[c];
        const float rv = __shfl_xor_sync(0xffffffffu, sv, HALF);
        const int ri = __shfl_xor_sync(0xffffffffu, si, HALF);
        const bool take = (rv > kv) || (rv == kv && ri < ki);   // lowest label on equal logits
        v[c] = take ? rv : kv;
        id[c] = take ? ri : ki;
    }
}

// The same exchange for a plain maximum or a plain sum of 32 columns: after the five calls (HALF = 16 .. 1) lane L
// holds column L's result over the warp in v[0].
template <int HALF, bool SUM>
__device__ __forceinline__ void reduce_exchange(float* v, int lane) {
    const bool up = (lane & HALF) != 0;
#pragma unroll
    for (int c = 0; c < HALF; ++c) {
        const float send = up ? v[c] : v[c + HALF];
        const float keep = up ? v[c + HALF] : v[c];
        const float recv = __shfl_xor_sync(0xffffffffu, send, HALF);
        v[c] = SUM ? keep + recv : fmaxf(keep, recv);
    }
}

// Timeline record of CTA 0 and of the last CTA (a role thread calls this; n is that thread's event counter).
__device__ __forceinline__ void trace_event(const LoopParams& p, int role, int& n, int step, int phase, int ev) {
    if (p.trace && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1) && step >= p.trace_step && step < p.trace_step + 2 &&
        n < kTraceEvents) {
        if (blockIdx.x != 0) role += 4;   // the last CTA's records go to the second half of the table
        TraceEvent t;
        t.tag = (uint32_t)(phase * 16 + ev);
        t.step = step;
        long long now;
        asm volatile("mov.u64 %0, %%clock64;" : "=l"(now)::"memory");   // not to be moved across the memory operations around it
        t.clock = now;
        p.trace[role * kTraceEvents + n] = t;
        ++n;
    }
}
// Marks of every CTA in the first traced step, on the global timer (comparable across SMs): role 8 + mark, one
// record per CTA (`step` holds the CTA index).  Joint: 0 slot entered, 1 copies of the window's enc_proj rows issued,
// 2 pred_proj has arrived, 3 operand handed to the issuing threads, 4 accumulator ready, 5 keys out (slot done).
// Decoder update: 6 keys of the CTA's utterances complete, 7 tokens known, 8 accumulator ready, 9 state written (slot
// done).  Projection: 10 state counters seen by the TMA thread, 11 accumulator ready, 12 pred_proj published, 13
// state counters seen for the GEMM issued a slot ahead, 14 that GEMM issued, 15 slot done.
enum { MK_J_ENTER = 0, MK_J_COPIES = 1, MK_J_PRED = 2, MK_J_HANDOVER = 3, MK_J_ACC = 4, MK_J_DONE = 5, MK_L_KEYS = 6, MK_L_TOK = 7,
       MK_L_ACC = 8, MK_L_DONE = 9, MK_P_FLAG = 10, MK_P_ACC = 11, MK_P_PUB = 12, MK_E_FLAG = 13, MK_E_ISSUED = 14, MK_P_DONE = 15 };
__device__ __forceinline__ void trace_mark(const LoopParams& p, int step, int phase_kind, int mark) {
    if (p.trace && step == p.trace_step && (int)blockIdx.x < kTraceEvents) {
        TraceEvent t;
        t.tag = (uint32_t)(phase_kind * 16 + 8);
        t.step = (int)blockIdx.x;
        t.clock = (long long)globaltimer_ns();
        p.trace[(8 + mark) * kTraceEvents + blockIdx.x] = t;
    }
}
// when this CTA finished its part of a phase
__device__ __forceinline__ void trace_phase_done(const LoopParams& p, int step, int phase_kind) {
    trace_mark(p, step, phase_kind, phase_kind == 0 ? MK_J_DONE : (phase_kind == 1 ? MK_L_DONE : MK_P_DONE));
}
enum { TR_J = 0, TR_L = 1, TR_P = 2 };
enum { EV_START = 0, EV_FIRST_ISSUE = 1, EV_LAST_ISSUE = 2, EV_FIRST_DATA = 3, EV_COMMIT = 4, EV_TOK = 5, EV_ACC = 6, EV_EPI_DONE = 7,
       EV_ARRIVE = 8, EV_RELEASE = 9 };

// Epilogue of one joint item: the accumulator holds logits^T [128 vocabulary entries of tile vt (lanes), n_tile window
// rows of row group rg (columns)].  Adds b_out, then per window row the argmax over the tile's 128 entries by a
// five-stage transposing exchange (lane L ends with the winner of column L; lowest label on ties) and a 64-bit
// atomicMax of (logit, label) across the vocabulary tiles.  FULL adds the logits store of teacher forcing and the
// per-row softmax statistics of window-based decoding.  RES: two accumulator copies (one per issuing thread) are
// added, and the eight epilogue warps split the columns in two (sub).
template <bool RES, bool FULL>
__device__ __forceinline__ void joint_epilogue_item(const LoopParams& p, uint32_t tm_j, uint32_t lane_off, int lane, int q, int sub,
                                                    int row_in_tile, int rg, int vt, int n_tile, const int32_t* t_cur,
                                                    unsigned long long* keys_cur, unsigned long long* part = nullptr) {
    const int v = vt * 128 + row_in_tile;            // this thread's vocabulary entry
    const bool v_ok = v < p.NV;
    const float bias = v_ok ? p.b_out[v] : 0.f;
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
                if (((okmask >> j) & 1u) && v_ok) p.logits_out[(size_t)(rg * n_tile + c0 + j) * p.NV + v] = val[j];
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
                if (row < p.rows && c0 + lane < n_tile) p.jpart[(size_t)row * p.parts + vt * 4 + q] = make_float2(m_keep, s_keep);
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
            if (part && !(FULL && p.window)) {
                // this warp's winner of row c0 + lane (over its 32 vocabulary entries) goes to shared memory; the caller
                // combines the four lane quadrants and puts the tile's key out
                if (c0 + lane < n_tile) part[q * n_tile + c0 + lane] = (row < p.rows && val[0] > -INFINITY) ? pack_key(val[0], (uint32_t)id[0]) : 0ull;
            } else if (row < p.rows && c0 + lane < n_tile && val[0] > -INFINITY) {
                atomicMax(&key_dst[row], pack_key(val[0], (uint32_t)id[0]));
            }
        }
    }
}

// Window-based decoding, decision phase (after every vocabulary tile has left its statistics): for the utterances
// b = first, first + stride, ... one warp per window row turns the partial (maximum, sum) pairs into the row's
// log-sum-exp, then one warp takes the most probable (label, offset) pair of Eq. (1) against "all blank" and leaves it
// in the keys in the form the control step reads (the chosen row carries its label, every other row the blank).
// n_ew epilogue warps take part (ew = index of this warp); win_* are shared arrays of kMaxWindow entries.
template <int n_ew>
__device__ __forceinline__ void window_decision(const LoopParams& p, int first, int stride, int ew, int lane, const int32_t* t_cur,
                                                unsigned long long* keys_cur, float* win_lpb, float* win_sc,
                                                unsigned long long* win_key) {
    const unsigned long long blank_key = pack_key(0.f, (uint32_t)p.blank);
    for (int b = first; b < p.B; b += stride) {
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
        if (b + stride < p.B) asm volatile("bar.sync 1, %0;" ::"n"(n_ew * 32) : "memory");   // the arrays are reused
    }
}

}  // namespace wind
