// Parameter blocks of the persistent decoding-loop kernel.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "wind_internal.cuh"

namespace wind {

// Tensor maps of one call; all bf16, 64-column boxes, 128-byte swizzle.
struct LoopMaps {
    CUtensorMap w_out;                 // [V+1, H], box 128 rows
    CUtensorMap z;                     // [rows_pad, H], box nj rows
    CUtensorMap w_pred;                // [H, P], box np rows
    CUtensorMap w_ih[kMaxLayers];      // [4P, P], box `slots` rows (layers > 0)
    CUtensorMap w_hh[kMaxLayers];      // [4P, P], box `slots` rows
    CUtensorMap hb[2][kMaxLayers];     // [Bpad, P], box 128 rows
    // resident-weights mode (one LSTM layer): weight tiles of 64 rows loaded once; per-step operands as ONE
    // three-dimensional box each (64 columns, rows, all K blocks)
    CUtensorMap w_hh_r;                // [4P, P], box 16 rows (one gate's 16 units)
    CUtensorMap w_pred_r;              // [H, P], box 64 rows
    CUtensorMap w_ih1_r, w_hh1_r;      // layer 1 (two-layer models): [4P, P], box 16 rows
    CUtensorMap hb_l3[2];              // layer 0 state [Bpad, P] as (64, rows, P/64), box (64, nl, P/64)
    CUtensorMap hb_l3_1[2];            // layer 1 state, same box
    CUtensorMap hb_p3[2];              // same, box (64, np, P/64)
    CUtensorMap z3;                    // [rows_pad, H] as (64, rows, H/64), box (64, nj, H/64) (resident kernel with grid barriers)
};

// How the three phases are cut into items and how shared memory is used (host-chosen).
struct LoopPlan {
    int grid;
    int kb_h, kb_p;                        // K blocks of 64 in H and in P
    int nj, vt_count, rg_count, j_items;   // joint: window rows per item, vocabulary tiles, row groups
    int rg_stride;                         // resident mode: row groups taken per wave (CTAs per vocabulary tile)
    int j_mode;                            // where the joint's W_out tile lives: 0 streamed through the ring, 1 kept in
                                           // shared memory, 2 kept in tensor memory (1, 2: every CTA owns one joint item)
    int tm_j, tm_l, tm_p;                  // tensor-memory columns of the joint / decoder / projection accumulators
    int l_early;                           // layer 0's GEMM runs one phase ahead of its cell update
    // resident-weights mode: W_hh tiles (4 gates x 16 units) and W_pred tiles (64 rows) stay in the shared memory of
    // disjoint CTA sets; accumulators are [64 weight rows, nl or np utterances]
    int resident, nl, ut_count, ht_count, ql_count, qp_count;
    int dataflow;                          // resident mode: the kernel without grid barriers (wind_loop_res.cu)
    int w_first, w_count;                  // step-recording CTAs [w_first, w_first + w_count), 64 utterances each (0: the L CTAs record)
    uint32_t buf_off, stage_off;           // the per-step operand buffer and the epilogue staging area (after the tile)
    uint32_t z_off, z_off_p;               // resident mode: the joint's operand buffer (z_off_p: in CTAs with a W_pred tile);
                                           // equal to buf_off where it shares the state box's memory
    int slots, ul, ug_count, mt_count, l_items;  // decoder: rows per gate block, units per item, unit groups, utterance tiles
    int np, hg_count, p_items;             // projection: H columns per item, H slices
    int stages_lp, stages_j;               // ring stages in the decoder/projection phases and in the joint phase
    uint32_t stage_lp, stage_j, stat_bytes, smem_bytes;
};

constexpr int kSlotFresh = 1 << 30;          // flag in a slot_len2 word
constexpr int kSlotLenMask = kSlotFresh - 1;

struct LoopParams {
    Ctrl* ctrl;
    int B, T, W, S, max_out, H, P, NV, blank, act, L;
    int rows, rows_pad, Bpad, step_cap;
    int nj, vt_count, rg_count, j_items, j_mode, rg_stride;
    int tm_j, tm_l, tm_p, l_early;
    int resident, nl, ut_count, ht_count, ql_count, qp_count;
    int w_first, w_count;
    uint32_t buf_off, stage_off, z_off, z_off_p;
    int slots, ul, ug_count, mt_count, l_items;
    int np, hg_count, p_items;
    int kb_h, kb_p;
    int stages_lp, stages_j;
    uint32_t stage_lp, stage_j, stat_bytes;
    const int32_t* enc_len;        // [n_utt]
    // Which utterance a batch row decodes (loop_kernel; the other kernels take row b = utterance b).  With more
    // utterances than rows, a row whose utterance is finished takes the next waiting one.  Double-buffered by step
    // parity like t2: a step's control threads write the copy the next step reads.
    int n_utt;
    int32_t* slot_len2;            // [2][B] frames of the row's utterance; kSlotFresh set in the step after it moved in
    int32_t* slot_row2;            // [2][B] enc_proj row of the utterance's first frame
    int32_t* slot_utt;             // [B] the utterance (index into the outputs); recording threads only
    int32_t* slot_pos;             // [B] tokens emitted so far for it; recording threads only
    int32_t* t2;                   // [2][B]
    unsigned long long* t_pub;     // [B]
    int32_t* count;                // [B]
    int32_t* emit_tok;             // [B]
    unsigned long long* keys2;     // [2][rows_pad]
    int32_t* out_tokens;
    int32_t* out_frames;
    int32_t* out_len;
    float* c_state;                // [L][B][P]
    float* dh;                     // [B][4P] layer 1's recurrent term W_hh[1] h (two-layer resident mode)
    __nv_bfloat16* hb;             // [2][L][Bpad][P]
    __nv_bfloat16* z;              // [rows_pad][H]
    const __nv_bfloat16* enc_proj; // [B*T][H]
    const float* g0;               // [V+1][4P]
    const float* b_ih[kMaxLayers];
    const float* b_hh[kMaxLayers];
    const float* b_pred;
    const float* b_out;
    const __nv_bfloat16* w_out;    // [V+1][H]
    // teacher forcing (wind_eval_joint_window): feed prefix tokens, then store the window logits
    int forced;
    const int32_t* prefix;
    int U;
    const int32_t* prefix_len;
    float* logits_out;
    // timeline of CTA 0 for lock steps [trace_step, trace_step + 2); trace == nullptr: off
    TraceEvent* trace;
    int trace_step;
    // window-based decoding (the most probable pair of Eq. (1) per step instead of the first non-blank row)
    int window, parts;             // parts = 4 per vocabulary tile: one (maximum, sum of exponentials) pair per epilogue warp
    unsigned long long* nbkeys;    // [rows_pad] best non-blank (logit, label) per window row
    float2* jpart;                 // [rows_pad][parts]
    float* jblank;                 // [rows_pad] blank logit per window row
    int extra_arrivals;            // test hook: arrivals the first cross-CTA wait asks for beyond those that come (0 in normal use)
    // resident-weights mode: arrival counters between CTA groups (keys of a row group complete, state of an utterance
    // group written, ...) and the stamped pred_proj values
    uint32_t* flags;
    unsigned long long* pred_pub;  // [B][H / 2] (two bf16 values, stamp)
    int joint_iters;               // measurement aid: > 0 runs only the joint phase, that many times (kernel with grid barriers, FULL)
    unsigned long long* kslot;     // [window rows][vocabulary tiles, padded to even] the tiles' stamped (logit, label) keys
};

// Options of the tile planner (process-wide; wind_set_loop_options): whether the resident-weights mode may be chosen,
// a forced placement of the streaming mode's W_out tile (-1: the planner's own choice; 0 streamed, 1 shared memory,
// 2 tensor memory, taken when feasible), the most waves the resident joint may run in (1..4), and which resident kernel
// (-1: the planner's choice by batch size; 0 the one with grid barriers; 1 the one with arrival counters).
struct LoopOptions { int resident; int joint_placement; int max_joint_waves; int dataflow; };
void loop_set_options(const LoopOptions& o);
LoopOptions loop_get_options();
bool loop_plan_ok(const wind_model_t& m, int B, int W);
cudaError_t loop_plan(const Call& c, LoopPlan* out);
cudaError_t loop_sm_count(int* sms);   // SMs of the current device (cached per device)
// the plan as a pure function of the shapes and of the device's SM count and opt-in shared memory per block
cudaError_t loop_plan_for(const wind_model_t& m, int B, int W, int sms, int smem_optin, LoopPlan* out, bool refill = false);
// launchers of the two kernels (wind_loop.cu: streaming mode; wind_loop_res.cu: resident-weights mode)
cudaError_t loop_res_set_smem(int bytes);
cudaError_t loop_res_launch(const LoopMaps& maps, const LoopParams& p, int grid, uint32_t smem_bytes, bool full, cudaStream_t stream);
int loop_set_extra_arrivals(int n);  // returns the previous value
cudaError_t loop_prepare(Call& c);   // plan + tensor maps + shared-memory opt-in (host only; not inside a capture)

}  // namespace wind
