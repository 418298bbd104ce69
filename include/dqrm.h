/*
 * dqrm.h - C ABI of the B200 (sm_100a) library for the embedding half of a DQRM
 * training step: quantisation-aware training of DLRM embedding tables
 * ("DQRM: Deep Quantized Recommendation Models", arXiv 2410.20046).
 *
 * The calls follow the paper's statement of the problem:
 *   - Section 3.1 / Figure 2(b): run the embedding lookup first, then quantise only
 *     the rows the batch uses                                   -> dqrm_emb_fwd
 *   - Section 3.2: the per-table scale is found by traversing the whole table and is
 *     refreshed only every P iterations                         -> dqrm_scale_refresh
 *   - Section 4.3 / Appendix B.1: the embedding gradient is a sparse (indices, values)
 *     tensor over the touched rows, duplicates coalesced        -> dqrm_emb_bwd
 *   - Appendix B.1: only the values are quantised to INT8, with a scale fixed by the
 *     bit width and the tensor's distribution                   -> dqrm_grad_quant_int8
 *   - Appendix B.1: the local step uses the dequantised gradient; Section 3.1: the FP32
 *     master copy is what is updated                            -> dqrm_row_update
 *
 * Quantiser (the paper prints no formula; Section 4.1 gives every table a single scale,
 * Appendix A describes a uniform quantiser whose clipping range is the table's fixed
 * minimum and maximum):
 *     n(b) = 2^(b-1) - 1
 *     scale(absmax, b) = max(absmax, 1e-8f) / (float)n(b)                 one FP32 divide
 *     Q(x; s, b) = clamp(round_half_even(x / s), -2^(b-1), 2^(b-1) - 1)   one FP32 divide
 *     DQ(q; s)   = (float)q * s                                           one FP32 multiply
 * These are the results every call reproduces bit for bit: each FP32 operation above is a
 * single IEEE round-to-nearest operation, and no fused multiply-add stands where two
 * roundings are specified.  Where one scale serves many elements the kernels reach the
 * same codes through a reciprocal multiply that is provably equal away from rounding
 * ties and redo the rare element near a tie with the IEEE division (see
 * dqrm_selfcheck_quantizer).
 *
 * Conventions
 *   - All array arguments are DEVICE pointers unless the name starts with h_ (host).
 *     The caller owns every buffer.  After dqrm_create the library allocates nothing;
 *     scratch comes from a caller-provided workspace (see dqrm_workspace_bytes).
 *   - `stream` is a cudaStream_t passed as void*; calls are asynchronous on it.  Calls
 *     that share a context or a workspace must be ordered on one stream.
 *   - Tables live in one arena [sum_t R_t, D] float32, row-major, base aligned to 16
 *     bytes; row_off[t] is the first arena row of table t.  D is a multiple of 4,
 *     4 <= D <= 1024.  sum_t R_t < 2^31.
 *   - indices[L] int32: row numbers within their table, 0 <= idx < R_t, table-major
 *     (all lookups of table 0 in sample order, then table 1, ...).
 *   - offsets[T*B + 1] int32, non-decreasing, offsets[0] = 0, offsets[T*B] = L:
 *     bag g = t*B + i owns indices[offsets[g] .. offsets[g+1]).  Empty bags are allowed.
 *   - out and grad_out are [B, T, D] float32 (sample-major).  T*B < 2^31.
 *   - bits[T] int32, each in 2..16.  scales[T] float32.
 *   - Return value: DQRM_OK or a negative error.  Invalid arguments are detected on the
 *     host before anything is launched.  Conditions only the device can see (an index
 *     outside its table, offsets that decrease or leave [0, L]) never trap: the
 *     offending value is clamped into range, an error code is recorded in the context's
 *     device status word, and dqrm_check_status reports it.
 */
#ifndef DQRM_H_
#define DQRM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DQRM_OK                 0
#define DQRM_ERR_INVALID_ARG   (-1)  /* null pointer, bad T/D/B/L, bits outside 2..16 */
#define DQRM_ERR_WORKSPACE     (-2)  /* workspace null, misaligned (256 B) or too small */
#define DQRM_ERR_CUDA          (-3)  /* a CUDA runtime call failed; see dqrm_last_cuda_error */
#define DQRM_ERR_INDEX_RANGE   (-4)  /* device saw an index outside [0, R_t) or a bad offset */
#define DQRM_ERR_TIMEOUT       (-5)  /* reserved: a bounded device-side wait ran out */
#define DQRM_ERR_STATIC_LIMIT  (-6)  /* size exceeds the built-in scratch of a *_static call */
#define DQRM_ERR_NOT_SORTED    (-7)  /* dqrm_train_step_sorted: the workspace holds no unconsumed sorted batch of this L, B */

typedef struct dqrm_ctx dqrm_ctx;

/* Creates a context for T tables of feature size D on the current device.
 * h_row_off: HOST array [T+1], h_row_off[0] = 0, strictly increasing.
 * Allocates a few KB of device memory (row offsets, status word).  Not stream-ordered:
 * synchronises the device. */
int dqrm_create(dqrm_ctx **ctx, int T, int D, const int64_t *h_row_off);

/* Frees what dqrm_create allocated.  The caller must have synchronised its streams. */
int dqrm_destroy(dqrm_ctx *ctx);

/* Bytes of scratch the calls below need for at most max_lookups lookups and max_bags
 * bags per call.  The workspace must be 256-byte aligned.  Contents need not be
 * preserved between calls and need no initialisation. */
size_t dqrm_workspace_bytes(const dqrm_ctx *ctx, int64_t max_lookups, int64_t max_bags);

/* Synchronises `stream`, returns DQRM_OK or the first device-detected error since the
 * last check, and clears the status word. */
int dqrm_check_status(dqrm_ctx *ctx, void *stream);

/* The cudaError_t (as int) of the last failed runtime call on this context, 0 if none. */
int dqrm_last_cuda_error(const dqrm_ctx *ctx);

/* Static text for a DQRM_* code. */
const char *dqrm_status_string(int status);

/* Scale refresh (Section 3.2): for every table, min and max over all R_t*D elements,
 * a = max(|min|, |max|), scales[t] = scale(a, bits[t]).
 *   tables  in   [sum R_t, D]
 *   bits    in   [T]
 *   scales  out  [T]
 *   minmax  out  [T][2] (min, max), may be NULL
 * Reads the arena once.  Bit-exact: min/max do not depend on the order of evaluation. */
int dqrm_scale_refresh(dqrm_ctx *ctx, const float *tables, const int32_t *bits,
                       float *scales, float *minmax,
                       void *workspace, size_t workspace_bytes, void *stream);

/* Row summaries (no counterpart in the paper; Section 3.2 states the cost they remove: finding a
 * table's range means reading the whole table, which is why the paper refreshes the scales
 * only every P iterations).  A training step changes only the rows it touches, so the library
 * can keep (min, max) of every row, 8 bytes per row in memory the caller provides, current as
 * it writes rows; dqrm_scale_refresh then reads the summaries, 8 bytes per row instead of 4*D,
 * and returns the same scales and minmax as the scan of the tables (min and max do not depend
 * on how the elements are grouped).
 *   dqrm_row_summary_bytes   bytes the summary needs: 8 * sum R_t
 *   dqrm_row_summary_attach  scans `tables` once, writes every row's (min, max) to `summary`
 *                            (device memory, 8-byte aligned, owned by the caller, kept until
 *                            detach or dqrm_destroy); from then on dqrm_row_update,
 *                            dqrm_train_step*, dqrm_dp_merge_update keep the entries of the rows
 *                            they write current and dqrm_scale_refresh ignores its `tables`
 *                            argument's contents and reads the summary.  The calls that follow
 *                            must be ordered behind `stream` by the caller.  Rows changed by
 *                            anyone else make the summary stale: attach again.
 *   dqrm_row_summary_detach  dqrm_scale_refresh scans the tables again
 * Errors: DQRM_ERR_INVALID_ARG (null or misaligned), DQRM_ERR_WORKSPACE (summary too small). */
size_t dqrm_row_summary_bytes(const dqrm_ctx *ctx);
int dqrm_row_summary_attach(dqrm_ctx *ctx, const float *tables, void *summary,
                            size_t summary_bytes, void *stream);
int dqrm_row_summary_detach(dqrm_ctx *ctx);

/* Forward (Section 3.1, Figure 2(b)): for every bag, gather its rows from the FP32
 * master table, fake-quantise each gathered row with its table's stored scale and bit
 * width, and sum over the bag (in bag order, FP64 accumulator, rounded once):
 *   out[i][t][:] = sum_{j in bag (t,i)} DQ(Q(W_t[indices[j]][:]; scales[t], bits[t]); scales[t])
 *   codes_out    out [L][D] int8, the integer codes of every gathered row; may be NULL;
 *                only meaningful when every bits[t] <= 8.
 * The table is not modified and no low-precision copy of it is ever made. */
int dqrm_emb_fwd(dqrm_ctx *ctx, const float *tables, const int32_t *indices,
                 const int32_t *offsets, const float *scales, const int32_t *bits,
                 float *out, int8_t *codes_out, int B, int64_t L, void *stream);

/* Backward (Section 4.3, Appendix B.1): sum pooling and a straight-through quantiser
 * hand every lookup its bag's upstream gradient unchanged; lookups of the same
 * (table, row) are summed (FP64 accumulator, rounded once to FP32).
 *   grad_out     in   [B][T][D]
 *   unique_rows  out  [>= L] int32: per table ascending distinct row numbers, table-major
 *   uniq_off     out  [T+1] int32: table t owns unique_rows[uniq_off[t] .. uniq_off[t+1])
 *   grad_rows    out  [>= L][D] float32: summed gradient of each unique row
 * Takes neither tables nor scales: the pass-through backward needs neither.
 * Entries of unique_rows / grad_rows at and beyond uniq_off[T] are left untouched.
 * Deterministic: the same inputs give the same bits on every run. */
int dqrm_emb_bwd(dqrm_ctx *ctx, const float *grad_out, const int32_t *indices,
                 const int32_t *offsets, int32_t *unique_rows, int32_t *uniq_off,
                 float *grad_rows, int B, int64_t L,
                 void *workspace, size_t workspace_bytes, void *stream);

/* INT8 gradient quantiser (Appendix B.1): per table t over its U_t*D summed gradients,
 *   grad_scales[t] = scale(max |grad_rows|, 8);  codes = Q(grad_rows; grad_scales[t], 8).
 * A table that touched no row gets scale(0, 8) and no codes.
 *   grad_rows in [U][D], uniq_off in [T+1], codes out [U][D] int8, grad_scales out [T]. */
int dqrm_grad_quant_int8(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off,
                         int8_t *codes, float *grad_scales,
                         void *workspace, size_t workspace_bytes, void *stream);

/* Touched-row SGD update (Appendix B.1, Section 3.1): for every unique row u of table t,
 *   g = (float)codes[u][d] * grad_scales[t];  step = lr * g;  W[row][d] = W[row][d] - step
 * (three separately rounded FP32 operations).  Rows not listed are not read or written.
 * Rows are distinct, so the update is free of conflicts. */
int dqrm_row_update(dqrm_ctx *ctx, float *tables, const int32_t *unique_rows,
                    const int32_t *uniq_off, const int8_t *codes, const float *grad_scales,
                    float lr, void *stream);

/* One training iteration of the embedding path in the order the paper's loop takes it:
 * forward, backward, INT8 gradient quantisation, touched-row update.  Results equal
 * those of the four separate calls; the gradient abs-max is folded into the backward
 * and the quantiser is fused with the update, which saves launches and one read of
 * grad_rows.  grad_out is an input (in training it comes from the dense layers). */
int dqrm_train_step(dqrm_ctx *ctx, float *tables, const int32_t *indices,
                    const int32_t *offsets, const float *grad_out,
                    const float *scales, const int32_t *bits,
                    float *out, int32_t *unique_rows, int32_t *uniq_off, float *grad_rows,
                    int8_t *codes, float *grad_scales, float lr, int B, int64_t L,
                    void *workspace, size_t workspace_bytes, void *stream);

/* dqrm_train_step in two calls, for a training loop that knows the next batch's indices
 * while the current batch trains (no counterpart in the paper; Section 4.3 only fixes what the
 * sparse gradient holds).  dqrm_sort_batch does the part of the backward that needs the
 * indices alone: it orders the lookups by row and finds where every row's run begins.
 * dqrm_train_step_sorted then runs forward, gradient summation, INT8 quantisation and update
 * for the same batch.  unique_rows and uniq_off are outputs of the PAIR of calls: pass the same
 * buffers to both; they are complete when dqrm_train_step_sorted is (the sort numbers each
 * table's rows by itself, and the tables' bases are added where the gradients are summed).  The sorted order travels in `workspace` (dqrm_workspace_bytes): pass
 * the same workspace to both calls and to nothing in between; two workspaces used alternately
 * let batch k+1 be sorted on one stream while batch k trains on another.  dqrm_sort_batch
 * records an event behind the sort and dqrm_train_step_sorted puts its gradient summation (not
 * its forward, which does not need the sorted order) behind that event, so the step's stream
 * need not wait for the sort's stream.  Exception: when the two calls are made inside different
 * stream captures, or one inside a capture and one outside, the event cannot connect them and
 * the caller orders the calls itself (join the sort's stream before the capture ends).  A
 * workspace is written by the sort and read by the step: the next sort into the same workspace
 * must be ordered, by the caller, behind the step that used it.  One dqrm_sort_batch serves ONE
 * dqrm_train_step_sorted: the step uses up counters that only the sort resets.  The context
 * keeps, on the host, which workspaces hold a sorted batch that no step has taken yet;
 * dqrm_train_step_sorted on a workspace that holds none (never sorted, already used, or sorted
 * for another B or L) returns DQRM_ERR_NOT_SORTED and launches nothing.  A step replayed from
 * a captured CUDA graph is outside that bookkeeping: capture each step together with its sort.
 * Outputs equal those of dqrm_train_step. */
int dqrm_sort_batch(dqrm_ctx *ctx, const int32_t *indices, const int32_t *offsets,
                    int32_t *unique_rows, int32_t *uniq_off, int B, int64_t L,
                    void *workspace, size_t workspace_bytes, void *stream);
int dqrm_train_step_sorted(dqrm_ctx *ctx, float *tables, const int32_t *indices,
                           const int32_t *offsets, const float *grad_out,
                           const float *scales, const int32_t *bits, float *out,
                           int32_t *unique_rows, int32_t *uniq_off, float *grad_rows,
                           int8_t *codes, float *grad_scales, float lr, int B, int64_t L,
                           void *workspace, size_t workspace_bytes, void *stream);

/* Makes `stream` wait until the forward of the last dqrm_train_step_sorted enqueued on this
 * context has finished (no counterpart in the paper).  For the pipelined loop above: the sort of
 * batch k+1 shares the SMs with whatever runs beside it, so a loop may hold the sort back until
 * batch k's forward is done and let it run beside the gradient summation and the update instead
 * (whether that pays depends on the shapes: it helped 64-byte rows and hurt 256-byte rows when
 * measured on a B200):
 *   dqrm_train_step_sorted(batch k, stream A); dqrm_stream_wait_forward(ctx, stream B);
 *   dqrm_sort_batch(batch k+1, stream B).
 * Before the first dqrm_train_step_sorted the wait returns at once.  Inside a stream capture both
 * calls must belong to the same capture. */
int dqrm_stream_wait_forward(dqrm_ctx *ctx, void *stream);

/* Bytes of workspace dqrm_train_step_host needs (device staging for the host buffers,
 * the step's intermediate outputs and the scratch of dqrm_train_step). */
size_t dqrm_host_step_workspace_bytes(const dqrm_ctx *ctx, int64_t max_lookups, int64_t max_bags);

/* dqrm_train_step for callers whose batch lives in HOST memory: copies h_indices [L],
 * h_offsets [T*B+1] and h_grad_out [B][T][D] to the device, runs the step, and copies
 * the pooled output back to h_out [B][T][D]; asynchronously when the host buffers are
 * pinned.  The call is ordered on `stream`: it starts behind the work already on `stream`,
 * and work put on `stream` afterwards starts once the step and both copies are complete.
 * Inside the call the inputs come in and the pooled output goes out on two streams owned by
 * the context, beside the index sort and the forward (the two large transfers run in opposite
 * directions).  The workspace holds two sets of staging buffers that consecutive calls use in
 * turn, so the inputs of a call are copied while the call before it is still computing and
 * sending its output; a caller that issues calls back to back therefore keeps both directions
 * of the host link busy.  With dqrm_set_overlap(ctx, 0) everything stays on `stream`.
 * tables, scales and bits stay on the device.  The sparse gradient (unique rows, codes,
 * scales) stays in the workspace.  h_grad_out and h_out must stay valid and untouched
 * until the call's work on `stream` is complete. */
int dqrm_train_step_host(dqrm_ctx *ctx, float *tables, const int32_t *h_indices,
                         const int32_t *h_offsets, const float *h_grad_out,
                         const float *scales, const int32_t *bits, float *h_out,
                         float lr, int B, int64_t L,
                         void *workspace, size_t workspace_bytes, void *stream);

/* ---- allocation-free gradient quantiser (the paper has no counterpart) -------------
 * Same result as dqrm_grad_quant_int8, for callers that must not allocate device memory
 * when they quantise: code that runs inside a host framework which has already claimed
 * the GPU's memory for its own pool, or a serving / real-time loop that cannot afford the
 * device-wide synchronisation a cudaMalloc or cudaFree implies.  It needs no context and
 * no workspace: T and D are passed directly, and the per-table abs-max scratch lives in a
 * fixed array inside the library image (DQRM_STATIC_MAX_TABLES 32-bit words = 4 KB, held
 * by every GPU that loads the library until the process exits).  The call performs no
 * cudaMalloc / cudaFree and uses no allocating library routine.
 *   T            number of tables, 1 .. DQRM_STATIC_MAX_TABLES; larger T returns
 *                DQRM_ERR_STATIC_LIMIT and launches nothing
 *   D            feature size, multiple of 4, 4 .. 1024
 *   grad_rows in [U][D], uniq_off in [T+1], codes out [U][D] int8, grad_scales out [T]
 *                (device pointers, caller-owned, as for dqrm_grad_quant_int8)
 * The first call on each device looks up the array's device address (the device that is
 * current at the call is used); make that first call outside any stream capture.
 * All calls on a device share the one array, which still holds the previous call's maxima:
 * each call clears the T entries it uses on `stream` before its kernels run.  Two calls
 * that can overlap on the GPU (different streams, no dependency) race on it; order them. */
#define DQRM_STATIC_MAX_TABLES 1024
int dqrm_grad_quant_int8_static(int T, int D, const float *grad_rows, const int32_t *uniq_off,
                                int8_t *codes, float *grad_scales, void *stream);

/* ---- data-parallel exchange of the sparse INT8 gradient (Appendix B.1) --------------
 * The paper's data-parallel step, for every parameter tensor: compute the quantisation
 * scale locally, unify it across ranks, quantise locally with the unified scale, sum the
 * integer gradients over the ranks, apply the dequantised sum on every rank.  The three
 * calls below are the local pieces; the two collectives between them (a MAX all-reduce of
 * T floats, an all-gather of each rank's rows and codes) are the caller's, e.g. NCCL.
 * Readings: scales are unified by MAX of the abs-max (no rank clips); the integers are
 * summed exactly in 32 bits; the update uses the sum over ranks, not the mean.
 *
 * dqrm_grad_absmax: absmax[t] = max |grad_rows| over table t's rows (0 if none); [T] floats.
 * dqrm_grad_quant_int8_unified: grad_scales[t] = scale(unified_absmax[t], 8) and
 *   codes = Q(grad_rows; grad_scales[t], 8).  With unified_absmax = this rank's own abs-max
 *   it equals dqrm_grad_quant_int8.
 * dqrm_dp_merge_update: rank r's sparse gradient sits at rows_cat + r*rank_stride (ascending
 *   distinct rows per table, uoff_cat + r*(T+1) as in dqrm_emb_bwd) with codes at
 *   codes_cat + r*rank_stride*D.  n_entries = sum of the ranks' row counts and
 *   max_table_entries = the largest per-table sum over ranks (both from the host copy of
 *   uoff_cat).  Writes the ascending union of rows per table to union_rows [>= n_entries] /
 *   union_off [T+1], optionally the int32 sums to sums_out [>= n_entries][D] (may be NULL),
 *   and updates W[row] -= lr * ((float)sum * grad_scales[t]) with three rounded operations.
 *   Workspace: dqrm_dp_workspace_bytes(ctx, max n_entries). */
int dqrm_grad_absmax(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off, float *absmax, void *stream);
int dqrm_grad_quant_int8_unified(dqrm_ctx *ctx, const float *grad_rows, const int32_t *uniq_off,
                                 const float *unified_absmax, int8_t *codes, float *grad_scales, void *stream);
size_t dqrm_dp_workspace_bytes(const dqrm_ctx *ctx, int64_t max_entries);
int dqrm_dp_merge_update(dqrm_ctx *ctx, float *tables, int W, int64_t rank_stride, const int32_t *rows_cat,
                         const int32_t *uoff_cat, const int8_t *codes_cat, const float *grad_scales, float lr,
                         int64_t n_entries, int64_t max_table_entries, int32_t *union_rows, int32_t *union_off,
                         int32_t *sums_out, void *workspace, size_t workspace_bytes, void *stream);

/* ---- bit-packed export and inference (Appendix C) ----------------------------------
 * The deployed model stores the embedding codes bit-packed (Appendix C; Table "res_tab":
 * 2.161 GB -> 0.270 GB at 4 bits).  The paper gives no layout; here element d of a row sits
 * in byte (d*bits)/8 at bit offset (d*bits)%8, lowest bits first, as a two's-complement code;
 * a row takes D*bits/8 bytes and rows follow the arena order.  bits is 2, 4 or 8 for all tables.
 * dqrm_packed_bytes: size of the packed arena (0 for an unsupported width).
 * dqrm_pack_tables: packed = Q(tables; scales[t], bits), one pass over the arena.
 * dqrm_packed_fwd: out[i][t][:] = sum over bag (t,i) of code * scales[t] (bag order, FP64
 *   accumulator, rounded once) - equal, bit for bit, to dqrm_emb_fwd on the weights and
 *   scales the tables were packed from. */
size_t dqrm_packed_bytes(const dqrm_ctx *ctx, int bits);
int dqrm_pack_tables(dqrm_ctx *ctx, const float *tables, const float *scales, int bits, uint8_t *packed, void *stream);
int dqrm_packed_fwd(dqrm_ctx *ctx, const uint8_t *packed, const int32_t *indices, const int32_t *offsets,
                    const float *scales, int bits, float *out, int B, int64_t L, void *stream);

/* ---- table-sharded forward payload (Section 4.3, the remark on hybrid parallelism) -----------
 * With the tables sharded over ranks, the all-to-all that carries embedding vectors shrinks with
 * the code width: for one-index bags the pooled vector is the dequantised row, so a table's owner
 * sends the row's bit-packed codes (layout of dqrm_pack_tables, bits in {2, 4, 8} for all tables)
 * and the samples' owner multiplies by the table's scale.
 * dqrm_emb_fwd_codes: payload[i][t][D*bits/8] = packed Q(row of bag (t, i)) for the context's T
 *   tables and B bags per table; every bag must hold exactly one index (L == T*B, else
 *   DQRM_ERR_INVALID_ARG; a bag that does not is reported as DQRM_ERR_INDEX_RANGE and left unwritten).
 * dqrm_decode_payload: out[i][t0 + j][:] = code * scales[j] for a payload block [B][T_blk][D*bits/8]
 *   of T_blk consecutive tables starting at table t0 of an output [B][T_total][D] (D is the
 *   context's; its tables are not used).  Decoding every sender's block gives, bit for bit, what
 *   dqrm_emb_fwd computes on the unsharded problem. */
int dqrm_emb_fwd_codes(dqrm_ctx *ctx, const float *tables, const int32_t *indices, const int32_t *offsets,
                       const float *scales, int bits, uint8_t *payload, int B, int64_t L, void *stream);
int dqrm_decode_payload(dqrm_ctx *ctx, const uint8_t *payload, const float *scales, int bits, float *out, int B,
                        int T_blk, int T_total, int t0, void *stream);

/* ---- choice of the backward's sort (no counterpart in the paper) --------------------
 * dqrm_emb_bwd and dqrm_train_step order the batch's lookups by row before they sum
 * duplicates.  path 0 (default): one thread-block cluster per table (eight blocks, sixteen
 * when the batch has very few tables) sorts that table's lookups in distributed shared
 * memory; a batch with more lookups per table than such a cluster holds takes path 1 by
 * itself.  path 1: one global least-significant-digit radix sort over all tables.  Both give
 * identical outputs; the choice only affects speed. */
int dqrm_set_sort_path(dqrm_ctx *ctx, int path);

/* dqrm_train_step and dqrm_train_step_sorted run the backward up to the summed gradient (index
 * sort, gradient summation: neither needs the tables or the forward's output) on a second
 * stream owned by the context (created by dqrm_create), beside the forward on the caller's
 * stream, and join the two before the touched rows are updated; the caller's stream sees one
 * ordered step.  dqrm_train_step_sorted also moves its forward to a third, lowest-priority
 * stream of the context (forked from and joined to the caller's stream), so that the forward's
 * many blocks do not keep a sort of the next batch, running elsewhere, off the SMs.
 * on = 0 keeps every launch on the caller's stream.  Default: 1. */
int dqrm_set_overlap(dqrm_ctx *ctx, int on);

/* ---- quantiser self-check (no counterpart in the paper) ----------------------------
 * The kernels evaluate Q(x; s, b) without the IEEE division sequence where a scale is
 * shared by many elements, and fall back to the division near rounding ties.  This call
 * compares that evaluation with the plain definition clamp(round_half_even(x / s)) for
 * the `count` FP32 bit patterns first_bits, first_bits+1, ... (count <= 2^32, wrapping)
 * and ADDS the number of disagreements to *mismatches (device uint64, caller-zeroed).
 * NaN patterns are skipped.  Expected result: 0 for every scale and bit width. */
int dqrm_selfcheck_quantizer(dqrm_ctx *ctx, float scale, int bits, uint32_t first_bits, uint64_t count,
                             uint64_t *mismatches, void *stream);

/* ---- launch accounting and timing aid (no counterpart in the paper) ----------------
 * dqrm_launch_count: kernels this context has launched since it was created (memsets
 * and copies are not counted).
 * dqrm_profile_begin / dqrm_profile_end: between the two, every launch of this context
 * is followed by a cudaEvent on its stream; _end synchronises the stream and returns,
 * per kernel id (0 .. dqrm_kernel_count()-1), the summed milliseconds between the event
 * before and the event after its launches, and the number of launches.  Both arrays are
 * HOST arrays of at least dqrm_kernel_count() entries.  At most 4096 launches are
 * recorded per begin/end pair; later ones are counted but not timed.  Event recording
 * perturbs back-to-back launches slightly, so headline timings are taken with profiling
 * off.  dqrm_kernel_name gives the kernel's name for an id. */
int64_t dqrm_launch_count(const dqrm_ctx *ctx);
int dqrm_profile_begin(dqrm_ctx *ctx, void *stream);
int dqrm_profile_end(dqrm_ctx *ctx, void *stream, float *h_ms_per_kernel,
                     int32_t *h_launches_per_kernel, int n);
const char *dqrm_kernel_name(int kernel_id);
int dqrm_kernel_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DQRM_H_ */
