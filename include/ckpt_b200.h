/*
 * ckpt_b200 - checkpointed CNN training step for one B200 (sm_100a), C ABI.
 *
 * Two halves:
 *   - host planners: given the data sizes d_0..d_n of a layer chain, choose the checkpoint set that
 *     minimises peak activation memory under one of the paper's two memory models;
 *   - device executor: run one training step of a chain of layer units (forward keeping only the
 *     checkpoints, backward that recomputes each segment from its nearest checkpoint) inside a
 *     caller-provided activation arena, returning weight gradients and the arena's high-water mark.
 *
 * Conventions
 *   - every function returns CKPT_OK (0) or a negative CKPT_E_* code; nothing throws or aborts;
 *     ckpt_last_error() returns a thread-local, human-readable message for the last failure.
 *   - "host" / "device" is stated for every pointer.  The library never allocates device memory:
 *     arena, workspace, parameters and gradients are caller-owned (for example torch tensors).
 *   - activations are NHWC; convolution matrices are [C_out][k][k][C_in]; fully connected matrices
 *     are [out][in] with `in` enumerating the NHWC-flattened input.
 *   - d_i is the byte size of unit i's output for the whole batch, rounded up to 256 bytes so that
 *     every arena offset is aligned for vector and bulk-tensor access; d_0 is the input batch.
 *   - checkpoint sets are byte masks is_ckpt[0..n]; indices 0 and n are always checkpoints
 *     (Section 3.1 of the paper).
 */
#ifndef CKPT_B200_H
#define CKPT_B200_H

#include <stdint.h>

#if defined(__GNUC__)
#define CKPT_API __attribute__((visibility("default")))
#else
#define CKPT_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

/* ---------------------------------------------------------------- status codes */
#define CKPT_OK 0
#define CKPT_E_NULL (-1)           /* a required pointer is null                                  */
#define CKPT_E_BAD_N (-2)          /* n < 1                                                       */
#define CKPT_E_BAD_SIZE (-3)       /* some d_i < 1                                                */
#define CKPT_E_OVERFLOW (-4)       /* 2 * sum(d) does not fit in int64                            */
#define CKPT_E_BAD_PLAN (-5)       /* is_ckpt[0] or is_ckpt[n] is 0                               */
#define CKPT_E_BAD_ARG (-6)        /* unknown enum value, inconsistent shapes, ...                */
#define CKPT_E_ARENA_OOM (-7)      /* arena smaller than the plan's peak; nothing was launched    */
#define CKPT_E_WORKSPACE (-8)      /* workspace smaller than ckpt_chain_workspace_bytes()         */
#define CKPT_E_CUDA (-9)           /* a CUDA runtime/driver call failed (see ckpt_last_error)     */
#define CKPT_E_DEVICE_TIMEOUT (-10)/* a bounded device-side wait gave up; results are invalid     */
#define CKPT_E_UNSUPPORTED (-11)   /* shape/dtype combination has no kernel                       */
#define CKPT_E_NO_DEVICE (-12)     /* no CUDA device / driver available                           */

CKPT_API const char* ckpt_last_error(void);

/* ---------------------------------------------------------------- host planners
 *
 * Algorithms (numbered as in the paper):
 *   CKPT_ALGO_STATIC_N3  - Algorithm 3, "Checkpoint Selection" (Section 3.2): minimises Eq. (cost),
 *                          sum of checkpoints + largest segment sum, in O(n^3).
 *   CKPT_ALGO_DYNAMIC_N2 - Algorithm 5 (Section 4.1): minimises max_i m(i) of Eq. (memory) by the
 *                          O(n^2) recursion Eq. (T-rec).
 *   CKPT_ALGO_DYNAMIC_N  - Algorithm 6 (Section 4.2): same optimum by the monotone-queue /
 *                          two-pointer search.  Queue pushes, pops and pointer moves are O(n) in total as in
 *                          the paper; each U(i,j) is evaluated exactly from prefix sums and a range maximum found
 *                          by bisection (the paper's incremental update of a running maximum cannot be undone when
 *                          the pointer moves back), so the implementation is O(n log n).
 * Readings of the printed algorithms: data are d_0..d_n and the dynamic recursion runs down to
 * i = 0 (answer M(0)); j ranges up to n inclusive; M(n) = d_n is the base case; Algorithm 3 forces
 * d_n as a checkpoint (answer min_s s + d_n + M(n-1,s)) and inserts candidate i before reading the
 * queue head, as Eq. (T) requires.  Ties: dynamic - the smallest next checkpoint attaining the
 * minimum; static - the smallest segment cap, then the smallest previous checkpoint.
 */
#define CKPT_ALGO_STATIC_N3 0
#define CKPT_ALGO_DYNAMIC_N2 1
#define CKPT_ALGO_DYNAMIC_N 2
/* Comparison plan of Sections 2.1 and 5.3 (not optimal): a checkpoint every ceil(sqrt(n)) units plus
 * d_n; peak_bytes is its value under Eq. (memory). */
#define CKPT_ALGO_SQRT_N 3

/* d: host, n+1 sizes (>= 1).  is_ckpt: host, n+1 bytes, written (0/1).  peak_bytes: host, written:
 * the objective value of the returned set under the algorithm's own memory model. */
CKPT_API int ckpt_plan(int algo, int64_t n, const int64_t* d, uint8_t* is_ckpt, int64_t* peak_bytes);

/* Same as ckpt_plan, also reporting how many inner-loop steps the search took (queue pushes, pops
 * and pointer moves for the queue-based algorithms; (i,j) pairs for Algorithm 5). work: host. */
CKPT_API int ckpt_plan_counted(int algo, int64_t n, const int64_t* d, uint8_t* is_ckpt,
                      int64_t* peak_bytes, int64_t* work);

/* Objective of an arbitrary checkpoint set.
 *   CKPT_MODEL_STATIC  - Eq. (cost) (Section 3.1).
 *   CKPT_MODEL_DYNAMIC - Eq. (memory)/(memory-simple) with s(h,i) of Eq. (s) (Section 4).
 *   CKPT_MODEL_STORE_ALL - Algorithm 1: sum of d_0..d_n (is_ckpt ignored, may be null). */
#define CKPT_MODEL_STATIC 0
#define CKPT_MODEL_DYNAMIC 1
#define CKPT_MODEL_STORE_ALL 2
CKPT_API int ckpt_eval(int model, int64_t n, const int64_t* d, const uint8_t* is_ckpt, int64_t* peak_bytes);

/* Eq. (memory) with three sizes per tensor instead of one - the more faithful model of what a framework holds that
 * Section 6 leaves as future work, built on Observations (1)-(2) of Section 4.  Tensor t occupies kept[t] bytes while
 * it is a checkpoint, live[t] bytes while it is an interior tensor of the segment being processed (a unit's backward
 * may need more than its output: a pre-normalisation copy, the interior tensors of a residual block), and its
 * gradient r_t occupies grad[t] bytes.  Backward at checkpoint i with previous checkpoint h then holds
 *     sum of kept[c], c in C, c <= i  +  sum of live[t], h < t < i  +  max grad[t], h <= t < i
 *     (+ max grad[t], h < t <= i, when incoming != 0: the buffer of the gradient each step reads, which Eq. (memory)
 *     leaves out),
 * and the objective is the maximum over i.  kept = live = grad = d with incoming = 0 is Eq. (memory) itself.
 *   ckpt_plan_sizes: CKPT_ALGO_DYNAMIC_N2 (the recursion of Algorithm 5, any sizes) or CKPT_ALGO_DYNAMIC_N (the
 *     queue-based search of Algorithm 6; its Lemma 1, U(i,j) increasing in j, holds when live[t] >= kept[t] for
 *     0 < t < n, otherwise CKPT_E_BAD_ARG).  Same tie rule and outputs as ckpt_plan.
 *   ckpt_eval_sizes: the objective of a given set.
 * All arrays: host, n+1 entries, every entry >= 1. */
CKPT_API int ckpt_plan_sizes(int algo, int64_t n, const int64_t* kept, const int64_t* live, const int64_t* grad, int incoming,
                    uint8_t* is_ckpt, int64_t* peak_bytes);
CKPT_API int ckpt_eval_sizes(int64_t n, const int64_t* kept, const int64_t* live, const int64_t* grad, int incoming,
                    const uint8_t* is_ckpt, int64_t* peak_bytes);

/* Least recomputation under a memory budget (plan(layer sizes, layer costs) -> checkpoint set).  Section 3.1 asks for
 * the smallest peak only, and many sets reach the optimum of Eq. (memory); the backward pass of Algorithm 4 runs the
 * forward of every unit whose output is not a checkpoint a second time, so among the sets whose Eq. (memory) value is
 * at most budget_bytes this call returns one with the smallest sum of cost[i] over the non-checkpoint units
 * i = 1..n-1.  budget_bytes = 0 stands for the optimum of Algorithms 5/6 (same peak as ckpt_plan, fewer or cheaper
 * recomputed units); a larger budget buys less recomputation.  Exact: a search over suffix plans that keeps, per
 * checkpoint, the plans no other plan beats in both cost and tolerated prefix.
 * d, cost: host, n+1 entries (cost[0] and cost[n] are not read; entries >= 0, any unit: ckpt_chain_unit_costs gives
 * nanoseconds).  is_ckpt: host, n+1 entries written; *peak_bytes = Eq. (memory) of the returned set (<= budget);
 * *recompute_cost = its recomputation cost.  Errors: as ckpt_plan, CKPT_E_BAD_ARG when a cost is negative or no set
 * fits the budget. */
CKPT_API int ckpt_plan_min_recompute(int64_t n, const int64_t* d, const int64_t* cost, int64_t budget_bytes, uint8_t* is_ckpt,
                            int64_t* peak_bytes, int64_t* recompute_cost);

/* ---------------------------------------------------------------- launch log (host only)
 *
 * Which kernels ran.  ckpt_launch_log(1) clears the log and starts counting every kernel the library launches, by
 * kernel name; ckpt_launch_log(0) stops.  ckpt_launch_log_read writes the counts as text, one "count<TAB>name" line
 * per kernel, into text (host, capacity bytes, always terminated; may be null) and the size a complete copy needs
 * into *needed.  A step replayed from its recording (ckpt_chain_set_graph) launches nothing from the host and is
 * not counted. */
CKPT_API int ckpt_launch_log(int enable);
CKPT_API int ckpt_launch_log_read(char* text, int64_t capacity, int64_t* needed);

/* ---------------------------------------------------------------- arena schedule (host only)
 *
 * Execution policies = the paper's three memory schedules:
 *   CKPT_POLICY_STORE_ALL - Algorithm 1: every d_i allocated and kept.
 *   CKPT_POLICY_STATIC    - Algorithm 2: forward keeps checkpoints; backward frees the finished
 *                           segment and recomputes the previous one; checkpoints are never freed.
 *   CKPT_POLICY_DYNAMIC   - Algorithm 4: d_i released right after backward step i; one output-
 *                           gradient buffer of size max(d_h..d_{i-1}) per segment, the old buffer
 *                           being released before the next segment is recomputed, so that the
 *                           high-water mark is exactly Eq. (memory).
 *
 * ckpt_arena_dry_run replays the allocation events of one step without touching a device.
 * events (host, may be null): up to max_events records of 4 int64:
 *   {kind (1 = alloc, 0 = free), tensor id (0..n = d_i, n+1 = gradient buffer), offset, size}.
 * n_events / high_water_bytes / extent_bytes: host, written.  extent_bytes = highest arena offset
 * ever occupied; the placement rule guarantees extent_bytes == high_water_bytes == ckpt_eval(). */
#define CKPT_POLICY_STORE_ALL 0
#define CKPT_POLICY_STATIC 1
#define CKPT_POLICY_DYNAMIC 2
CKPT_API int ckpt_arena_dry_run(int policy, int64_t n, const int64_t* d, const uint8_t* is_ckpt,
                       int64_t* events, int64_t max_events, int64_t* n_events,
                       int64_t* high_water_bytes, int64_t* extent_bytes);

/* Memory at the end of every "training phase index" of Section 5.1.1: trace[0] = before the step
 * (d_0 only), trace[1..n] = end of the forward stage of unit i, trace[n+1..2n] = end of the backward
 * stage of unit n, n-1, .., 1, trace[2n+1] = after the step (everything but d_0 released; under
 * policies that keep tensors to the end, their release is counted here).  Bytes of the arena's
 * objects only (no weights, no workspace).  trace: host, 2n+2 entries written. */
CKPT_API int ckpt_arena_stage_trace(int policy, int64_t n, const int64_t* d, const uint8_t* is_ckpt, int64_t* trace);

/* ---------------------------------------------------------------- layer-chain description
 *
 * A chain is Eq. (1): d_i = f_i(d_{i-1}, w_i), i = 1..n, followed by a loss.  Unit kinds:
 *   CKPT_UNIT_CONV_BN_RELU - k x k cross-correlation (stride, zero padding, no bias), batch
 *       normalisation in training mode (biased variance, eps 1e-5), ReLU.
 *       parameters: w [c_out][k][k][c_in] (activation dtype), gamma [c_out] f32, beta [c_out] f32.
 *   CKPT_UNIT_MAXPOOL      - k x k max pooling (stride, padding); the first maximum in row-major
 *       window order receives the gradient.  No parameters.
 *   CKPT_UNIT_FC           - fully connected on the flattened input, bias, optional ReLU
 *       (flags & 1).  parameters: w [c_out][c_in] (activation dtype), b [c_out] f32.
 *   CKPT_UNIT_AVGPOOL      - global average over H and W.  No parameters.
 *   CKPT_UNIT_BOTTLENECK   - ResNet v1.5 bottleneck: 1x1 (c_in -> mid), 3x3 carrying the stride
 *       (mid -> mid), 1x1 (mid -> c_out), each with batch norm; projection shortcut when
 *       (flags & 2); ReLU after the residual add.  parameters: w1,g1,b1,w2,g2,b2,w3,g3,b3
 *       [,wp,gp,bp].
 *   CKPT_UNIT_CONV, CKPT_UNIT_BN, CKPT_UNIT_RELU - the three steps of a CONV_BN_RELU unit as chain
 *       units of their own (the finer layer granularity of Section 5.4: every step's output is a
 *       d_i the planner may keep or drop).  CONV: parameters w; BN: c_in = c_out = channels,
 *       parameters gamma, beta; RELU: no parameters.
 * Parameter tensors are numbered consecutively over the chain in the order listed above.
 * Gradients are always float32 with the parameter's shape.
 */
#define CKPT_UNIT_CONV_BN_RELU 0
#define CKPT_UNIT_MAXPOOL 1
#define CKPT_UNIT_FC 2
#define CKPT_UNIT_AVGPOOL 3
#define CKPT_UNIT_BOTTLENECK 4
#define CKPT_UNIT_CONV 5
#define CKPT_UNIT_BN 6
#define CKPT_UNIT_RELU 7

#define CKPT_DTYPE_F32 0   /* float32 storage and arithmetic (no tensor cores)                    */
#define CKPT_DTYPE_BF16 1  /* bfloat16 storage, float32 accumulation                              */

#define CKPT_LOSS_SUM 0        /* L = sum of every element of d_n                                 */
#define CKPT_LOSS_SOFTMAX_CE 1 /* softmax cross-entropy over d_n's channels, mean over the batch  */

typedef struct ckpt_unit_desc {
    int32_t kind;
    int32_t c_in;    /* FC: input features (must equal H*W*C of the incoming tensor)              */
    int32_t c_out;
    int32_t k;       /* filter / window size                                                      */
    int32_t stride;
    int32_t pad;
    int32_t mid;     /* bottleneck width                                                          */
    int32_t flags;   /* FC: bit 0 = ReLU; bottleneck: bit 1 = projection shortcut                 */
} ckpt_unit_desc;

typedef struct ckpt_chain ckpt_chain;  /* opaque, host memory owned by the library */

/* units: host array of n descriptors (copied).  Shapes are checked unit by unit. */
CKPT_API int ckpt_chain_create(const ckpt_unit_desc* units, int64_t n, int64_t batch, int32_t in_h,
                      int32_t in_w, int32_t in_c, int dtype, int loss, ckpt_chain** out);
CKPT_API void ckpt_chain_destroy(ckpt_chain* chain);

/* d: host, n+1 entries written (bytes, 256-aligned).  shapes (host, may be null): 3*(n+1) int32
 * {H, W, C} of d_0..d_n. */
CKPT_API int ckpt_chain_sizes(const ckpt_chain* chain, int64_t* d, int32_t* shapes);
/* cost_ns: host, n+1 entries written: a model of the time of each unit's forward pass (nanoseconds, from its
 * arithmetic and memory traffic at nominal rates; entry 0 is 0), the layer costs ckpt_plan_min_recompute takes. */
CKPT_API int ckpt_chain_unit_costs(const ckpt_chain* chain, int64_t* cost_ns);
CKPT_API int ckpt_chain_num_params(const ckpt_chain* chain, int64_t* count);
/* unit (1-based index of the owning unit), elems (element count), dtype (CKPT_DTYPE_* of the
 * parameter's storage; its gradient is always f32): host, written. */
CKPT_API int ckpt_chain_param_info(const ckpt_chain* chain, int64_t p, int64_t* unit, int64_t* elems,
                          int32_t* dtype);
/* Plan-independent scratch the executor needs besides the arena: gradient carry buffers, the
 * pre-normalisation buffer that each unit's backward re-derives, split-K partial sums, saved
 * batch statistics.  bytes: host, written. */
CKPT_API int ckpt_chain_workspace_bytes(const ckpt_chain* chain, int64_t* bytes);
/* The same for one schedule (policy as in ckpt_train_step).  Algorithm 4's schedule (CKPT_POLICY_DYNAMIC) places the
 * activated copy of a unit's input, and the last pre-normalisation tensor of a residual block, in whichever of its
 * gradient buffers is idle at that moment and needs no buffer of its own for them: its workspace is a prefix of the
 * full one.  ckpt_train_step
 * accepts a workspace of this size for that policy.  Errors: CKPT_E_NULL, CKPT_E_BAD_ARG (policy). */
CKPT_API int ckpt_chain_workspace_bytes_for(const ckpt_chain* chain, int policy, int64_t* bytes);
/* Algorithm 1 taken literally for residual blocks (off by default).  A block's output is the only chain tensor of the
 * block, and by default every schedule re-derives the block's interior tensors from its input at the start of the
 * block's backward - store-all included, which therefore already pays one extra forward of every block.  With
 * enable = 1 a CKPT_POLICY_STORE_ALL step gives every block a region of its own in the workspace, keeps the interiors
 * from the forward pass and re-derives nothing: the step time of a schedule that stores everything, against which the
 * recomputation overhead of the checkpointed schedules is measured.  The other policies are unaffected.  The
 * workspace of the store-all policy grows by the sum of all blocks' regions (ckpt_chain_workspace_bytes and
 * ckpt_chain_workspace_bytes_for report it); gradients are bit-identical either way.  Drops recorded graphs. */
CKPT_API int ckpt_chain_set_keep_interiors(ckpt_chain* chain, int enable);
/* Kernel selection for dense contractions: 0 = automatic (tensor cores where a kernel exists),
 * 1 = plain CUDA-core kernels only. */
CKPT_API int ckpt_chain_set_impl(ckpt_chain* chain, int impl);
/* Graph replay of the training step (off by default).  The launch sequence of a step (Algorithms 1, 2
 * and 4 as executed here) is a function of the chain, the plan, the policy and the pointers passed to
 * ckpt_train_step.  With enable = 1 the first step with a given set of those arguments runs launch by
 * launch, the second is recorded as a CUDA graph while it runs, and later ones replay the recording:
 * one submission per step, which matters for chains whose kernels are shorter than a launch (hundreds
 * of units on small tensors).  Results are bit-identical to the launch-by-launch step.  Up to four
 * recordings are kept per chain (least recently used dropped).  The caller keeps every buffer of a
 * recorded step alive and unchanged in place (contents may change, addresses may not); a batch or
 * label pointer in pageable host memory disables recording for that call.  enable = 0 drops the
 * recordings.  The library holds 64 bytes of pinned host memory per chain while enabled. */
CKPT_API int ckpt_chain_set_graph(ckpt_chain* chain, int enable);
/* Input staging: overlaps the host-to-device copy of the next step's batch with the current step (the training loop
 * of Algorithms 1, 2 and 4 reads one batch per step; ckpt_train_step itself copies a host batch at its start, on the
 * step's stream).  ckpt_chain_stage_batch starts an asynchronous copy of batch (host; pinned memory for a copy that
 * really overlaps) and labels (host, or null for the sum loss) into slot 0 or 1 of staging (device, caller-owned,
 * ckpt_chain_staging_bytes bytes, 256-byte aligned) on a stream the chain owns, and returns the device addresses of the
 * staged batch and labels.  Passing that batch address to ckpt_train_step makes the step wait, on its own stream, for
 * the copy before it reads the batch.  A slot may be staged again once the step that was given it has returned
 * (ckpt_train_step returns after its step has finished).  Typical loop: stage(slot 0, batch 0); for k: stage(slot
 * (k+1) % 2, batch k+1); train_step(staged slot k % 2).
 * Errors: CKPT_E_NULL, CKPT_E_BAD_ARG (slot), CKPT_E_WORKSPACE (staging too small), CKPT_E_NO_DEVICE, CKPT_E_CUDA. */
CKPT_API int ckpt_chain_staging_bytes(const ckpt_chain* chain, int64_t* bytes);
CKPT_API int ckpt_chain_stage_batch(ckpt_chain* chain, int slot, const void* batch, const int32_t* labels, void* staging,
                           int64_t staging_bytes, const void** batch_dev, const int32_t** labels_dev);

/* Verification aid (off by default): the backward recursion of Eq. (3) made visible.  With a tap set, every
 * ckpt_train_step also copies r_i = dL/dd_i, as it enters the backward step of unit i, to
 * tap + (d_1 + .. + d_{i-1}) for i = n .. 1 (d_i bytes each, chain dtype; for a conv+BN+ReLU unit d_i is the stored
 * convolution output, so r_i is the gradient with respect to that).  tap: device, at least d_1 + .. + d_n bytes,
 * or null to switch the copies off.  Together with CKPT_POLICY_STORE_ALL - after which the arena holds d_0 .. d_n at
 * consecutive offsets, Algorithm 1 freeing nothing - this lets a test check every unit's forward and backward
 * against a reference on the unit's own inputs.  Costs one device copy per unit. */
CKPT_API int ckpt_chain_set_gradient_tap(ckpt_chain* chain, void* tap, int64_t tap_bytes);

/* "Update w_i with g_i" - the last line of the backward loop of Algorithms 1, 2 and 4 - as plain gradient descent
 * (the paper names no rule): with learning_rate > 0 every following ckpt_train_step also overwrites each parameter
 * tensor with w - learning_rate * g, in the parameter's storage type (bf16 filters: float32 arithmetic, rounded to
 * nearest even), as soon as its gradient g is complete and nothing in the step reads the parameter any more; the
 * gradients are still written to `grads`.  For convolution filters on the tensor-core path the update happens in
 * the pass that sums the slices of the split weight gradient (no extra pass over the filter), and the input gradient
 * of the unit, which reads the filter, is computed before it.  params then point to memory the step writes.
 * learning_rate = 0 (default) leaves the parameters untouched.  NaN or negative values: CKPT_E_BAD_ARG. */
CKPT_API int ckpt_chain_set_sgd(ckpt_chain* chain, double learning_rate);

/* Failure-path self-test (off by default).  With wait_runs_out = 1 every following step launches, after its loss,
 * one extra single-warp kernel whose only wait has no producer and a limit of 2e5 clock cycles: the wait gives up,
 * writes its code into the step's status word and the kernel returns, as every bounded wait of the tensor-core
 * kernels does when its producer never arrives.  The step then finishes normally on the device and returns
 * CKPT_E_DEVICE_TIMEOUT with report->device_status = 1; the context stays usable.  Nothing faults or spins without
 * a limit. */
CKPT_API int ckpt_chain_set_selftest(ckpt_chain* chain, int wait_runs_out);

/* ---------------------------------------------------------------- the training step
 *
 * One pass of Algorithm 1, 2 or 4 (policy) over one batch.  Follows the paper's "Require: weights
 * w_1..w_n, input x (d_0), ground truth G", except that the weight update is left to the caller:
 * the step *returns* g_i (Eq. (5)) for every parameter.
 *
 * batch:   host or device, d_0 payload (batch*H*W*C elements of the chain dtype); copied into the
 *          arena at the start of the step, on `stream`.
 * labels:  host or device int32[batch] (ignored for CKPT_LOSS_SUM, may be null).
 * params:  host array of device pointers, one per parameter tensor.
 * grads:   host array of device pointers (float32), written.
 * arena:   device, arena_bytes >= ckpt_eval(model of policy) or CKPT_E_ARENA_OOM is returned before
 *          anything is launched.  Contents on return are unspecified.
 * workspace: device, ws_bytes >= ckpt_chain_workspace_bytes_for(policy) (ckpt_chain_workspace_bytes() fits every policy).
 * stream:  a cudaStream_t (null = default stream).  The call returns after the stream has drained.
 * report:  host, written.
 * Determinism: every reduction has a fixed order, so gradients are bit-identical across policies
 * and checkpoint sets for the same inputs.
 */
typedef struct ckpt_step_report {
    int64_t peak_bytes;      /* arena high-water mark: max over time of live bytes               */
    int64_t extent_bytes;    /* highest arena offset occupied                                    */
    int64_t predicted_bytes; /* ckpt_eval() of (policy's model, is_ckpt)                         */
    int64_t workspace_bytes; /* workspace actually required                                      */
    int64_t launches;        /* kernels launched by this step                                    */
    int64_t recomputed_units;/* unit forwards re-run during the backward phase                   */
    double loss;
    int32_t device_status;   /* 0, or the code written by a kernel whose bounded wait gave up    */
    int32_t replayed;        /* 1 when the step ran as a replay of its captured launch sequence  */
} ckpt_step_report;

CKPT_API int ckpt_train_step(ckpt_chain* chain, const uint8_t* is_ckpt, int policy, const void* batch,
                    const int32_t* labels, void* const* params, void* const* grads, void* arena,
                    int64_t arena_bytes, void* workspace, int64_t ws_bytes, void* stream,
                    ckpt_step_report* report);

/* ---------------------------------------------------------------- single operations
 *
 * The kernels the step is made of, callable one at a time (used by the parity tests and for
 * profiling).  All tensor pointers are device pointers; scratch is device memory of at least the
 * size returned by the matching *_scratch_bytes call (may be null when that size is 0).
 * impl: 0 = automatic, 1 = CUDA-core kernel, 2 = tensor-core kernel (CKPT_E_UNSUPPORTED if the
 * shape has none).  Calls are asynchronous on `stream`.
 *
 * ckpt_conv2d_forward : z[n,ho,wo,co] = sum_{r,s,ci} x[n, ho*stride-pad+r, wo*stride-pad+s, ci] *
 *                       w[co,r,s,ci]                                    (Eq. (1) for a conv unit)
 * ckpt_conv2d_dgrad   : dx = (d z / d x)^T dz                           (Eq. (3))
 * ckpt_conv2d_wgrad   : dw[co,r,s,ci] (f32) = sum_{n,ho,wo} dz * x      (Eq. (5))
 */
typedef struct ckpt_conv_shape {
    int32_t n, h, w, c_in, c_out, k, stride, pad;
} ckpt_conv_shape;

/* Status of the single operations below.  Their tensor-core kernels bound every device-side wait; a wait that
 * gives up records a code in a status word owned by the library and the kernel returns early, leaving its output
 * incomplete.  ckpt_op_status waits for the device to go idle, writes that word to *status (host; 0 = every wait was
 * satisfied), clears it, and returns CKPT_E_DEVICE_TIMEOUT when it was not 0.  Call it after a batch of single
 * operations whose results matter.  (ckpt_train_step has its own status word and checks it itself.) */
CKPT_API int ckpt_op_status(int32_t* status);
/* Launches one single-warp kernel whose only wait has no producer and gives up after limit_cycles (1 .. 2e9) clock
 * cycles, recording its code (9001) in the status word that ckpt_op_status reads: the failure path of the bounded
 * waits, exercised without a fault.  Asynchronous on `stream`. */
CKPT_API int ckpt_selftest_bounded_wait(int64_t limit_cycles, void* stream);

CKPT_API int ckpt_conv2d_scratch_bytes(const ckpt_conv_shape* s, int dtype, int64_t* bytes);
CKPT_API int ckpt_conv2d_forward(const ckpt_conv_shape* s, int dtype, int impl, const void* x, const void* w,
                        void* z, void* scratch, int64_t scratch_bytes, void* stream);
CKPT_API int ckpt_conv2d_dgrad(const ckpt_conv_shape* s, int dtype, int impl, const void* dz, const void* w,
                      void* dx, void* scratch, int64_t scratch_bytes, void* stream);
CKPT_API int ckpt_conv2d_wgrad(const ckpt_conv_shape* s, int dtype, int impl, const void* dz, const void* x,
                      float* dw, void* scratch, int64_t scratch_bytes, void* stream);

/* Convolution forward followed by the batch statistics of its output, as the conv+BN+ReLU unit of the
 * chain runs them (the forward step d_i = f_i(d_{i-1}, w_i) of Eq. (1) up to the point where d_i is
 * stored): z = conv(x, w) and stats[0..4c) as for ckpt_bn_relu_forward, computed over the stored
 * (rounded) z.  Where the tensor-core kernel for the shape is a persistent one, the per-channel sums
 * are gathered in its epilogue and z is not read again; otherwise two kernels run.
 * scratch: max(ckpt_conv2d_scratch_bytes, ckpt_bn_scratch_bytes(n*h_out*w_out, c_out)) bytes.
 * fused (host, optional): set to 1 when the sums came from the convolution's epilogue, else 0. */
CKPT_API int ckpt_conv2d_bn_statistics(const ckpt_conv_shape* s, int dtype, const void* x, const void* w, void* z,
                              const float* gamma, const float* beta, float* stats, void* scratch,
                              int64_t scratch_bytes, int32_t* fused, void* stream);

/* Batch normalisation (training mode) + ReLU over rows x channels (rows = N*H*W).
 * forward : stats[0..c) = mean, [c..2c) = 1/sqrt(var+eps), [2c..3c) = scale, [3c..4c) = shift
 *           (y = max(z*scale + shift, 0) when relu != 0, else z*scale+shift).
 * backward: given dy and the same z/stats, writes dz (may alias dy), dgamma, dbeta.
 * scratch: ckpt_bn_scratch_bytes(). */
CKPT_API int ckpt_bn_scratch_bytes(int64_t rows, int32_t c, int64_t* bytes);
CKPT_API int ckpt_bn_relu_forward(int dtype, int64_t rows, int32_t c, const void* z, const float* gamma,
                         const float* beta, int relu, void* y, float* stats, void* scratch,
                         void* stream);
CKPT_API int ckpt_bn_relu_backward(int dtype, int64_t rows, int32_t c, const void* dy, const void* z,
                          const float* gamma, const float* stats, int relu, void* dz, float* dgamma,
                          float* dbeta, void* scratch, void* stream);

/* Same result as ckpt_bn_relu_forward, for callers that cannot allocate device memory and therefore
 * have no scratch buffer to pass: code embedded in a framework that owns the whole memory budget,
 * latency-critical loops that must avoid the device-wide synchronisation of cudaMalloc/cudaFree,
 * or callers that were themselves only given input and output buffers.  (The paper has no
 * counterpart to this call; it exists for deployment only.)
 *   - The partial sums live in an array built into the library image (4,857,856 bytes, resident on
 *     every GPU that loads the library until the process exits), enough for
 *     c <= CKPT_BN_STATIC_MAX_CHANNELS and any row count; a larger c returns CKPT_E_UNSUPPORTED.
 *   - The call performs no cudaMalloc/cudaFree and calls no allocating routine.
 *   - The first call on each device looks up the array's device address; make that first call
 *     before starting any stream capture on that device.
 *   - All calls share the one array, which keeps whatever the previous call left in it (nothing in
 *     it needs clearing: each call overwrites what it reads).  Two calls that may run on the GPU at
 *     the same time - different streams, or different host threads - race on it: serialise them.
 * Pointers as for ckpt_bn_relu_forward (all device); asynchronous on `stream`. */
#define CKPT_BN_STATIC_MAX_CHANNELS 512
CKPT_API int ckpt_bn_relu_forward_noalloc(int dtype, int64_t rows, int32_t c, const void* z, const float* gamma,
                                 const float* beta, int relu, void* y, float* stats, void* stream);

/* Max pooling, NHWC.  backward recomputes the arg-max from x (first maximum in row-major window order).
 * scratch (device, may be null): with ckpt_maxpool_backward_scratch_bytes bytes (8-byte aligned) the general
 * (not 2x2 stride 2) backward records one arg-max byte per output element and gathers from that. */
CKPT_API int ckpt_maxpool_forward(int dtype, int32_t n, int32_t h, int32_t w, int32_t c, int32_t k,
                         int32_t stride, int32_t pad, const void* x, void* y, void* stream);
CKPT_API int ckpt_maxpool_backward_scratch_bytes(int dtype, int32_t n, int32_t h, int32_t w, int32_t c, int32_t k,
                                        int32_t stride, int32_t pad, int64_t* bytes);
CKPT_API int ckpt_maxpool_backward(int dtype, int32_t n, int32_t h, int32_t w, int32_t c, int32_t k,
                          int32_t stride, int32_t pad, const void* x, const void* dy, void* dx,
                          void* scratch, int64_t scratch_bytes, void* stream);

/* Softmax cross-entropy, mean over the batch: loss (device float, written), dlogits (chain dtype).
 * labels: device int32. */
CKPT_API int ckpt_softmax_ce(int dtype, int32_t batch, int32_t classes, const void* logits,
                    const int32_t* labels, float* loss, void* dlogits, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CKPT_B200_H */
