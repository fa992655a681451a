/*
 * eb.h - C ABI of the cross-layer MoE step (EasyBalance) for NVIDIA B200 (sm_100a).
 *
 * One step takes N micro-batches, each sitting at its own MoE layer l_j, and
 *   1. routes their tokens (top-k gating, Section 2.1),
 *   2. chooses the subset that runs now and the subset that is deferred (Schedule(S, m) of
 *      Algorithm 1; Section 4.2 and Section 5.2),
 *   3. groups the routed tokens of the chosen micro-batches by (virtual device, layer, expert)
 *      (the dispatch of Section 2.2 with D expert-parallel devices emulated on one GPU),
 *   4. runs every group through its expert in one grouped pass (expert_i of Eq. 1, SwiGLU),
 *   5. aggregates the expert outputs back per token (Eq. 1).
 *
 * Conventions
 *   - All tensor arguments are DEVICE pointers borrowed from the caller, 16-byte aligned,
 *     row-major, and must stay valid until the work enqueued on `stream` has finished.
 *     Host pointers are marked "host".  The library never frees or reallocates caller memory.
 *   - `stream` is a cudaStream_t passed as void*.  Every call only enqueues work and returns,
 *     except where stated.  Calls on one context must not overlap on the GPU (they share the
 *     context's workspace).
 *   - Errors are reported through the return code only.  Arguments are checked before any
 *     launch.  Device-side waits are bounded; if one gives up the kernel records
 *     EB_ERR_TIMEOUT in the context's status word (eb_device_status) and exits cleanly.
 *   - Limits: n_mb <= EB_MAX_MB, D <= EB_MAX_D, E <= EB_MAX_E, 1 <= K <= EB_MAX_K <= E,
 *     S <= EB_MAX_S, H % 8 == 0, I % 8 == 0.  Anything else gives EB_ERR_UNSUPPORTED.
 *   - Packed token layout: micro-batch j owns tokens tok_off[j] .. tok_off[j+1]-1.
 *   - Group table of a step: active layers = distinct layers of the chosen micro-batches,
 *     ascending.  Groups are enumerated device-major: for d in 0..D-1, for each active layer,
 *     the routed experts hosted by d (ascending) followed by the S shared experts.  Rows inside
 *     a group are ordered by (micro-batch, token).  Shared experts are replicated on every
 *     virtual device and serve the tokens whose home device floor(t_local * D / T_j) is d.
 */
#ifndef EB_H_
#define EB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct eb_ctx eb_ctx; /* opaque; created by eb_create, owned by the library */

typedef enum {
  EB_OK = 0,
  EB_ERR_INVALID_ARG = 1,
  EB_ERR_UNSUPPORTED = 2,
  EB_ERR_WORKSPACE = 3,
  EB_ERR_CUDA = 4,
  EB_ERR_TIMEOUT = 5
} eb_status;

/* Scheduling policies: MaxUtil (Section 4.2), CumUtil and DiffPeak (Section 5.2); ALL runs the
 * whole pool (lock-step execution, the no-deferral baseline). */
typedef enum {
  EB_POLICY_MAXUTIL = 0,
  EB_POLICY_CUMUTIL = 1,
  EB_POLICY_DIFFPEAK = 2,
  EB_POLICY_ALL = 3
} eb_policy;

enum { EB_MAX_MB = 16, EB_MAX_D = 16, EB_MAX_E = 256, EB_MAX_K = 8, EB_MAX_S = 8 };

/* Length of the int32 `step_meta` array written by eb_permute:
 *   [0] R = rows of this step, [1] G = groups, [2] number of active layers,
 *   [3 .. 3+D] first group of every virtual device (D+1 entries),
 *   [EB_META_LEN-1] routing indices outside [0, E) met in topk_idx: each is skipped (its slot gets
 *   pos = -1 and no row, it is never used as an index) and counted here; always 0 for indices
 *   written by eb_route.  The entries in between are unused. */
enum { EB_META_LEN = 32 };

typedef struct {
  int32_t L, E, K, S, H, I, D; /* layers, routed experts, top-k, shared experts, hidden, intermediate, devices */
  int32_t renorm_topk;         /* 1: gate weights renormalised over the K chosen experts; 0: full softmax */
  int32_t max_tokens;          /* capacity: largest packed token count of any later call */
  const int32_t* expert_to_device; /* host [E], values in [0, D); copied by eb_create */
} eb_config;

typedef struct {
  int32_t n_mb;           /* micro-batches in this call */
  const int32_t* tok_off; /* host [n_mb + 1], ascending, tok_off[0] == 0; copied at call time */
  const int32_t* layer;   /* host [n_mb], current MoE layer l_j in [0, L); copied at call time */
  uint32_t pool_mask;     /* bit j set: micro-batch j is in the pool S of Algorithm 1 */
} eb_batch;

/* Result of Schedule(S, m).  Lives in device memory (and optionally in host memory). */
typedef struct {
  uint32_t run_mask;   /* RunSet */
  uint32_t defer_mask; /* pool minus RunSet */
  int32_t n_run;
  int32_t status;      /* EB_OK or a device-side error */
  int32_t joint_load[EB_MAX_D]; /* sum of the chosen micro-batches' per-device loads */
  int64_t util_num;    /* sum_d joint_load[d] */
  int64_t util_den;    /* D * max_d joint_load[d]  (Eq. 3 for this step; 0 means no work) */
} eb_sched_result;

/* Device buffers of one step, for eb_step / eb_step_host.  Sizes in elements:
 *   logits f32 [max_tokens, E]; x bf16 [max_tokens, H]; topk_idx i32 [max_tokens, K];
 *   topk_w f32 [max_tokens, K]; mb_load i32 [EB_MAX_MB, D]; mb_cnt i32 [EB_MAX_MB, E];
 *   sched: one eb_sched_result; group_off i32 [eb_groups_capacity + 1];
 *   group_w i32 [eb_groups_capacity]; row_src i32 [eb_rows_capacity];
 *   pos i32 [max_tokens, K + S]; xp, yp bf16 [eb_rows_capacity, H]; step_meta i32 [EB_META_LEN];
 *   out bf16 [max_tokens, H]. */
typedef struct {
  float* logits;
  void* x;
  int32_t* topk_idx;
  float* topk_w;
  int32_t* mb_load;
  int32_t* mb_cnt;
  eb_sched_result* sched;
  int32_t* group_off;
  int32_t* group_w;
  int32_t* row_src;
  int32_t* pos;
  void* xp;
  void* yp;
  int32_t* step_meta;
  void* out;
  const void* residual; /* NULL: out = MoE output (eb_combine); else bf16 [max_tokens, H] added as in eb_combine_residual; may equal out */
} eb_step_buffers;

/* ---- life cycle ------------------------------------------------------------------------- */

/* Creates a context on the current CUDA device.  Allocates a few KB of device tables with
 * cudaMalloc.  Returns EB_ERR_UNSUPPORTED for shapes outside the limits, EB_ERR_INVALID_ARG
 * for a bad table, EB_ERR_CUDA if the device is not sm_100 or a CUDA call fails.  Every later
 * call on the context must be made with that device current (EB_ERR_INVALID_ARG otherwise).  A
 * context is not thread safe: calls on one context are made by one thread at a time; different
 * contexts may be used from different threads. */
eb_status eb_create(const eb_config* cfg, eb_ctx** out);
eb_status eb_destroy(eb_ctx* ctx);

/* Expert weights, bf16, consumed in place: w_gate, w_up [L][E+S][I][H]; w_down [L][E+S][H][I];
 * slot e < E is routed expert e, slot E+s shared expert s.  Borrowed until rebind/destroy. */
eb_status eb_bind_weights(eb_ctx* ctx, const void* w_gate, const void* w_up, const void* w_down);

/* Scratch memory: the caller allocates eb_workspace_bytes(ctx) bytes of device memory
 * (256-byte aligned) and hands it over; it holds permutation tables, the tile lists and the
 * bf16 intermediate activations [rows, I] of the expert pass. */
size_t eb_workspace_bytes(const eb_ctx* ctx);
eb_status eb_set_workspace(eb_ctx* ctx, void* dev_ptr, size_t bytes);

int32_t eb_rows_capacity(const eb_ctx* ctx);   /* max_tokens * (K + S) */
int32_t eb_groups_capacity(const eb_ctx* ctx); /* EB_MAX_MB * (E + D * S) */

/* ---- the five calls of one step ----------------------------------------------------------- */

/* Top-k gating (Section 2.1): for every token of the micro-batches in `route_mask`, the K
 * experts with the largest logits (ties: lower index first), kept in that order, and their
 * softmax weights.  Also the per-micro-batch workload vectors of Section 2.3:
 * mb_load[j][d] = assignments of micro-batch j landing on device d, mb_cnt[j][e] likewise per
 * expert.  Rows / entries of micro-batches outside `route_mask` are left untouched (a deferred
 * micro-batch keeps its routing).  logits f32 [T_tot, E]; topk_idx i32 [T_tot, K];
 * topk_w f32 [T_tot, K]; mb_load i32 [n_mb, D]; mb_cnt i32 [n_mb, E].  Logits must be finite. */
eb_status eb_route(eb_ctx* ctx, void* stream, const eb_batch* batch, uint32_t route_mask,
                   const float* logits, int32_t* topk_idx, float* topk_w,
                   int32_t* mb_load, int32_t* mb_cnt);

/* Schedule(S, m) of Algorithm 1 on the routed loads.  If the pool has at most m members all
 * run.  MaxUtil scores every subset with at least m members by sum(W) / (D * max(W)), W the
 * summed load vector, compared exactly in integers; ties go to the larger subset, then to the
 * numerically smaller mask.  d_res: device.  h_res: host (pinned recommended) or NULL; when not
 * NULL the result is also copied there and the stream is synchronised before returning. */
eb_status eb_schedule(eb_ctx* ctx, void* stream, const eb_batch* batch, int32_t m, eb_policy policy,
                      const int32_t* mb_load, eb_sched_result* d_res, eb_sched_result* h_res);

/* Dispatch on one GPU (Section 2.2; stands in for the first all-to-all): histogram of the chosen micro-batches' assignments per
 * group, exclusive prefix sum, stable ranks, and a 16-byte-vector gather of the token rows into
 * group-contiguous order.  Reads the run mask from d_res on the device.
 * x bf16 [T_tot, H]; group_off i32 [G+1]; group_w i32 [G] = layer * (E+S) + slot, the weight
 * matrix of each group; row_src i32 [R] = source token of each row; pos i32 [T_tot, K+S] = row
 * of each (token, slot), -1 for tokens of micro-batches that do not run; xp bf16 [R, H];
 * step_meta i32 [EB_META_LEN].  Buffers must have the capacities given by
 * eb_groups_capacity / eb_rows_capacity; all are written by the call and owned by the caller.
 * Needs a workspace (EB_ERR_WORKSPACE otherwise). */
eb_status eb_permute(eb_ctx* ctx, void* stream, const eb_batch* batch, const eb_sched_result* d_res,
                     const void* x, const int32_t* topk_idx,
                     int32_t* group_off, int32_t* group_w, int32_t* row_src, int32_t* pos,
                     void* xp, int32_t* step_meta);

/* expert_i of Eq. 1 for every group in one pass (the joint execution of Section 4.1):
 * yp[r] = W_down (silu(W_gate xp[r]) * (W_up xp[r])) with the weight matrices of the row's group
 * (group_w); bf16 in, fp32 accumulation on the tensor cores, the intermediate rounded once to bf16.
 * group_off, group_w, step_meta are the tables eb_permute wrote (device, read only); xp bf16
 * [eb_rows_capacity, H] and yp bf16 [eb_rows_capacity, H] must be allocated to that capacity (tiles
 * are fetched in boxes of up to 128 rows; rows beyond the step's row count are read but never
 * written).  Needs bound weights (else EB_ERR_INVALID_ARG) and a workspace (else EB_ERR_WORKSPACE);
 * a tensor-map or launch failure gives EB_ERR_CUDA. */
eb_status eb_expert_ffn_grouped(eb_ctx* ctx, void* stream, const void* xp, const int32_t* group_off,
                                const int32_t* group_w, const int32_t* step_meta, void* yp);

/* Same pass restricted to the groups of one virtual device (a contiguous range of the group
 * table): used to time each device's share of a step.  Rows of other devices are not written. */
eb_status eb_expert_ffn_device(eb_ctx* ctx, void* stream, const void* xp, const int32_t* group_off,
                               const int32_t* group_w, const int32_t* step_meta, void* yp,
                               int32_t device);

/* Weighted aggregation, Eq. 1: out[t] = sum_k topk_w[t][k] * yp[pos[t][k]] + sum_s yp[pos[t][K+s]]
 * in fp32, k ascending then s, rounded to bf16.  Rows of tokens whose micro-batch did not run
 * are left untouched.  No residual is added. */
eb_status eb_combine(eb_ctx* ctx, void* stream, const eb_batch* batch, const eb_sched_result* d_res,
                     const void* yp, const int32_t* pos, const float* topk_w, void* out);

/* The same with the residual connection of the MoE block, Section 2.1: h_{l+1} = h'_l + MLP(h'_l).
 * out[t] = (the sum of Eq. 1 above) + residual[t], the residual row added last in fp32, one rounding to
 * bf16.  residual bf16 [T_tot, H] is the block's input h' (what eb_permute gathered from); it may be the
 * same buffer as `out` (the hidden states are then updated in place; rows of micro-batches that did
 * not run stay as they are).  residual == NULL is eb_combine. */
eb_status eb_combine_residual(eb_ctx* ctx, void* stream, const eb_batch* batch, const eb_sched_result* d_res,
                              const void* yp, const int32_t* pos, const float* topk_w, const void* residual,
                              void* out);

/* ---- whole step --------------------------------------------------------------------------- */

/* The five calls back to back on `stream` with device-resident inputs (buf->logits, buf->x); the
 * aggregation adds buf->residual when it is not NULL (Algorithm 1's step for a model that carries its
 * hidden states in buf->x: residual = out = x updates them in place). */
eb_status eb_step(eb_ctx* ctx, void* stream, const eb_batch* batch, uint32_t route_mask, int32_t m,
                  eb_policy policy, const eb_step_buffers* buf);

/* Same with HOST inputs and outputs: copies h_logits [T_tot, E] f32 and h_x [T_tot, H] bf16 to
 * the device buffers, runs the step, copies out [T_tot, H] bf16 and the schedule result back and
 * synchronises the stream.  Host buffers should be pinned for the copies to be asynchronous. */
eb_status eb_step_host(eb_ctx* ctx, void* stream, const eb_batch* batch, uint32_t route_mask, int32_t m,
                       eb_policy policy, const eb_step_buffers* buf,
                       const float* h_logits, const void* h_x, void* h_out, eb_sched_result* h_res);

/* Pipelined form of eb_step_host for independent steps: eb_step_host_submit enqueues the input copies
 * on a copy stream of the context, the step on `stream` (after the copies) and the output copies on a
 * second copy stream (after the step), and returns without waiting; eb_step_host_wait(slot) blocks until
 * the outputs of the submission made with that slot are in host memory.  With two or more slots in use
 * the copies of one step overlap the kernels of another; the kernels themselves still run one step
 * after the other on `stream` (they share the workspace).  Rules: slot in [0, EB_HOST_SLOTS); a slot is
 * reused only after its wait; buf->logits, buf->x, buf->sched and buf->out must be distinct buffers per
 * slot in flight (the other buffers of eb_step_buffers may be shared by all slots); host buffers must
 * stay valid, and should be pinned, until the wait returns.  The paper has no counterpart: it keeps the
 * hidden states on the device between layers. */
enum { EB_HOST_SLOTS = 4 };
eb_status eb_step_host_submit(eb_ctx* ctx, void* stream, const eb_batch* batch, uint32_t route_mask, int32_t m,
                              eb_policy policy, const eb_step_buffers* buf, const float* h_logits,
                              const void* h_x, void* h_out, eb_sched_result* h_res, int32_t slot);
eb_status eb_step_host_wait(eb_ctx* ctx, int32_t slot);

/* ---- allocation-free variant --------------------------------------------------------------- */

/* Largest packed token count eb_permute_noalloc accepts (its scratch is a fixed array). */
enum { EB_NOALLOC_MAX_TOKENS = 4096 };

/* The paper has no counterpart to this call; it exists for callers that are not allowed to
 * create device allocations where they invoke the library: a serving process that has handed all
 * free HBM to its cache and must not grow, a plug-in running inside a host framework's callback
 * while that framework owns the allocator, a latency-critical loop that cannot take cudaMalloc's
 * implicit synchronisation.  Such callers cannot use eb_create / eb_set_workspace.
 *
 * Computes exactly what eb_permute computes (same outputs, same layouts, same capacities of the
 * output buffers: group_off [EB_MAX_MB*(E+D*S)+1], group_w [EB_MAX_MB*(E+D*S)],
 * row_src [T_tot*(K+S)], pos [T_tot, K+S], xp [T_tot*(K+S), H], step_meta [EB_META_LEN]), but
 * needs no context and no workspace.  The model shape comes in `cfg` (host; max_tokens and I are
 * ignored) and the scratch (expert tables, per-chunk histograms, group sizes; about 316 KB) is a
 * static device array inside the library, resident on every GPU that loads the library until
 * the process exits.  It calls no cudaMalloc, cudaFree or other allocating routine.
 *
 * - At most EB_NOALLOC_MAX_TOKENS packed tokens; more returns EB_ERR_UNSUPPORTED and launches nothing.
 * - The first call on each device resolves the array's device address (cudaGetSymbolAddress, with
 *   that device current); make that first call outside any stream capture.
 * - All calls on a device share the one array, which keeps the previous call's contents; the call
 *   re-initialises what it reads on `stream` (a set-up kernel rewrites the expert tables, which it
 *   receives by value, and clears the counters; no host memory is read after the call returns).
 *   Two calls whose work overlaps on the GPU (different streams, or different threads) race on the
 *   array: serialise them.
 * - The call works on whichever device is current, each device with its own copy of the array.
 * - topk_idx and d_res are the caller's data here, not checked by a context: routing indices
 *   outside [0, E) are skipped and counted in step_meta[EB_META_LEN-1], never dereferenced.
 * - `err` (host, may be NULL) receives a description of a failure, truncated to err_cap bytes. */
eb_status eb_permute_noalloc(const eb_config* cfg, void* stream, const eb_batch* batch,
                             const eb_sched_result* d_res, const void* x, const int32_t* topk_idx,
                             int32_t* group_off, int32_t* group_w, int32_t* row_src, int32_t* pos,
                             void* xp, int32_t* step_meta, char* err, size_t err_cap);

/* ---- status and timing -------------------------------------------------------------------- */

/* Reads (and clears) the context's device status word; synchronises the device. */
eb_status eb_device_status(eb_ctx* ctx, int32_t* out_status);

/* Consistency check of a step's permutation tables on the device, for debugging without a memory
 * checker: offsets ascending and ending at the row count, weight ids in range, pos and row_src
 * mutually inverse on the chosen tokens and -1 elsewhere, every row in a group of its token's layer
 * and expert, token order kept inside groups.  Every index is range-checked before it is used.
 * Writes the number of violations to *out_errors (host) and synchronises the stream. */
eb_status eb_check_permutation(eb_ctx* ctx, void* stream, const eb_batch* batch, const eb_sched_result* d_res,
                               const int32_t* topk_idx, const int32_t* group_off, const int32_t* group_w,
                               const int32_t* row_src, const int32_t* pos, const int32_t* step_meta,
                               int32_t* out_errors);

/* The workspace regions (permutation tables, tile lists, intermediate activations) are separated by guard
 * areas of 256 bytes that eb_set_workspace fills with a pattern and no kernel ever writes.  This call counts
 * the guard bytes that no longer hold the pattern (*out_bad, host; 0 = intact) and synchronises the stream:
 * a kernel that wrote past the end of its region shows up here instead of silently corrupting its neighbour.
 * The paper has no counterpart: a debugging aid for boxes without a memory checker. */
eb_status eb_check_workspace_guards(eb_ctx* ctx, void* stream, int32_t* out_bad);

/* Exercises the bounded wait used by the expert kernels without any fault: one CTA waits on a
 * barrier that nothing arrives on, for at most `limit_cycles` SM cycles (1 .. 2e9), then gives up,
 * records EB_ERR_TIMEOUT in the context status word and returns normally.  *out_gave_up (host) is
 * set to 1 if the wait expired.  Synchronises the stream.  The context stays usable. */
eb_status eb_selftest_bounded_wait(eb_ctx* ctx, void* stream, int64_t limit_cycles, int32_t* out_gave_up);

/* Per-kernel timing: when enabled every internal launch is bracketed by CUDA events on its
 * stream.  eb_kernel_ms synchronises and writes the duration in ms of the most recent launch of
 * each kernel (negative if it has not run since timing was enabled); `ms` is host [eb_num_kernels()]. */
int32_t eb_num_kernels(void);
const char* eb_kernel_name(int32_t i);
eb_status eb_set_timing(eb_ctx* ctx, int32_t enabled);
eb_status eb_kernel_ms(eb_ctx* ctx, float* ms);

/* Kernels launched by the library in this process so far (all contexts; launches through the
 * allocation-free entry point and the self-test are not counted). */
uint64_t eb_launch_count(void);

const char* eb_status_string(eb_status s);
/* Text of the last failure on this context (host string, valid until the next call). */
const char* eb_last_error(const eb_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* EB_H_ */
