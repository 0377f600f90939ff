/*
 * ftpipe.h -- C ABI of the per-stage training library (single B200, sm_100a).
 *
 * The calls follow the problem statement of FTPipeHD (Chen et al., arXiv 2110.02781):
 * a DNN is cut into contiguous ranges of layers ("stages", Sec. III-B); every stage runs
 * the forward pass, the backward pass and the SGD update of its range (Sec. III-C, IV-B);
 * a per-layer time profile (Sec. III-B "model profiling") feeds the capacity estimate
 * (Eq. 1-3) and the partition optimiser (Eq. 4-7); after a new partition the weights are
 * re-homed (Sec. III-D, Algorithm 1) and on a schedule they are replicated to the next
 * stage and to the central node (Sec. III-E).
 *
 * Conventions
 *   - A "unit" is the paper's layer: what the profile, the optimiser and run_stage index.
 *     Units are 0-indexed; a partition is N+1 boundaries 0 = p_0 < ... < p_N = L and stage i
 *     owns units [p_i, p_{i+1}).
 *   - Activations are channels-last (N, H, W, C); a 1-D signal has H == 1.  Element type is
 *     float (precision 0) or bfloat16 (precision 1; master weights, gradients, statistics and
 *     the loss stay float).
 *   - Canonical parameter order of a unit: its ops in order; per op
 *       CONV1D/CONV2D/FC : W[kh][kw][cin][cout] then bias[cout] if has_bias
 *       DWCONV3x3        : W[3][3][c]
 *       BN               : gamma[c], beta[c]      (state: running_mean[c], running_var[c])
 *   - Ownership: the CALLER allocates every device and pinned-host buffer, including the
 *     workspace the model lives in, and supplies the stream (a cudaStream_t passed as void*).
 *     The library owns only the small host-side ftp_model object.  No call allocates device
 *     memory.  Pointers marked "device" must be device addresses, "host" host addresses.
 *   - All GPU work is asynchronous on the given stream unless stated otherwise.
 *   - Errors: every call returns an ftp_status; arguments are validated before any launch
 *     and a failed call launches nothing.  ftp_last_error() gives the text for this thread.
 *     Kernels never trap or assert.  Every wait inside a tensor-core kernel is bounded; one that
 *     runs out makes the kernel skip its stores, return, and leave a code in a device status
 *     word.  Calls that synchronise (ftp_train_step with loss_host, ftp_profile_layers,
 *     ftp_get_tensor / ftp_get_logits to a host buffer, ftp_check_device_status) read that word,
 *     return FTP_ETIMEOUT when it is set and clear it; asynchronous calls queue a copy of it
 *     behind their launches and the next call of the model that launches or reports
 *     (run_stage, sgd_step, train_step, stage_times) returns FTP_ETIMEOUT before doing anything
 *     once that copy shows a code, until ftp_check_device_status has cleared it.  Tensors
 *     written between the failed wait and the report are invalid.
 */
#ifndef FTPIPE_H
#define FTPIPE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ftp_model ftp_model; /* opaque, library-owned */

typedef enum {
    FTP_OK = 0,
    FTP_EINVAL = 1,   /* bad argument (null pointer, bad kind, a >= b, N > L, ...) */
    FTP_ERANGE = 2,   /* index or size out of range, buffer too small or misaligned */
    FTP_ENOMEM = 3,   /* host allocation failed or workspace too small */
    FTP_ECUDA = 4,    /* a CUDA runtime call or a launch failed */
    FTP_ESTATE = 5,   /* call order violated (backward without forward, ...) */
    FTP_ETIMEOUT = 6, /* a bounded device-side wait ran out */
    FTP_EUNSUPPORTED = 7
} ftp_status;

enum { FTP_CONV1D = 0, FTP_CONV2D = 1, FTP_DWCONV3x3 = 2, FTP_BN = 3, FTP_ACT = 4, FTP_ADD_RESIDUAL = 5,
       FTP_MAXPOOL2 = 6, FTP_GAP = 7, FTP_FC = 8, FTP_SOFTMAX_CE = 9 };
enum { FTP_ACT_NONE = 0, FTP_ACT_RELU = 1, FTP_ACT_RELU6 = 2 };
enum { FTP_FP32 = 0, FTP_BF16 = 1 };
/* selector of ftp_get_tensor / ftp_set_tensor */
enum { FTP_T_WEIGHTS = 0, FTP_T_GRADS = 1, FTP_T_MOMENTUM = 2, FTP_T_STATE = 3 };

typedef struct {
    int32_t unit;         /* partition unit of this op; non-decreasing along the list */
    int32_t kind;         /* FTP_CONV1D ... FTP_SOFTMAX_CE */
    int32_t cin, cout;    /* channels in / out (BN, pools, ADD: cin == cout) */
    int32_t k;            /* kernel size (CONV1D: 1 x k; CONV2D: k x k; DW: 3; FC: 1) */
    int32_t stride, pad;
    int32_t act;          /* activation applied to this op's output (CONV*, FC, BN, ACT) */
    int32_t has_bias;
    int32_t residual_src; /* ADD_RESIDUAL: index of the op whose output is added; -1 otherwise */
} ftp_layer_desc;

typedef struct {
    int32_t batch, in_c, in_h, in_w, n_classes;
    int32_t precision;    /* FTP_FP32 or FTP_BF16 */
    int32_t max_stages;   /* upper bound on the number of stages (each gets a weight arena) */
    float lr, momentum, weight_decay, bn_eps, bn_momentum;
} ftp_model_cfg;

/* One record of the kernel trace (see ftp_trace_enable). */
typedef struct {
    int32_t kernel;       /* kernel class id, see ftp_kernel_name */
    int32_t unit;         /* unit the launch belongs to, -1 if none */
    int32_t op;           /* op index, -1 if none */
    int32_t backward;     /* 0 forward, 1 backward, 2 optimiser / copies */
    float ms;             /* device time of the launch (CUDA events on the launching stream) */
    double bytes;         /* algorithmic bytes: each input read once, each output written once */
    double flops;         /* algorithmic floating-point operations */
} ftp_trace_rec;

/* ---- build_model(layers): Sec. III-B (the central node loads the whole model; a worker
 * holds the sub-model of its range).  ------------------------------------------------------ */

/* Sizes of the device workspace and of the pinned-host workspace the model needs.
 * layers: host array of n descriptors.  Pure host arithmetic. */
ftp_status ftp_workspace_bytes(const ftp_layer_desc* layers, int32_t n, const ftp_model_cfg* cfg,
                               size_t* dev_bytes, size_t* pinned_bytes);

/* Build the unit table, the per-stage weight arenas (float master weights, momentum, BN
 * running statistics, bf16 shadow), the gradient arena, the activation stash and the
 * scratch space inside dev_ws (device, 256-byte aligned, >= dev_bytes) and pinned_ws
 * (pinned host memory registered for device access, >= pinned_bytes).  The initial partition
 * is one stage owning every unit.  Arena contents are undefined until ftp_set_tensor.
 * The workspaces must outlive the model.  Validates the layer list (shapes must chain). */
ftp_status ftp_build_model(const ftp_layer_desc* layers, int32_t n, const ftp_model_cfg* cfg, void* dev_ws,
                           size_t dev_bytes, void* pinned_ws, size_t pinned_bytes, ftp_model** out);
void ftp_destroy_model(ftp_model* m);

ftp_status ftp_num_units(const ftp_model* m, int32_t* L);
/* Offset and count (in floats) of a unit's trainable parameters / BN running statistics in
 * the canonical whole-model order. */
ftp_status ftp_unit_param_span(const ftp_model* m, int32_t unit, int64_t* offset, int64_t* count);
ftp_status ftp_unit_state_span(const ftp_model* m, int32_t unit, int64_t* offset, int64_t* count);
/* Shape (N, H, W, C) and byte size of the boundary activation leaving a unit: the D_j of
 * Eq. 5 (Sec. III-B "size of the output data of each layer"). */
ftp_status ftp_unit_output_shape(const ftp_model* m, int32_t unit, int32_t shape[4], int64_t* bytes);

/* Copy `count` floats of one unit's tensor (which = FTP_T_*) from / to a host or device
 * buffer.  Setting the weights also refreshes the bf16 shadow and marks the momentum buffer
 * of the unit as not yet initialised.  Host copies use pageable-safe synchronous semantics:
 * when the other side is a host pointer the call returns after the copy has completed. */
ftp_status ftp_set_tensor(ftp_model* m, int32_t which, int32_t unit, const float* src, int64_t count,
                          int32_t src_is_device, void* stream);
ftp_status ftp_get_tensor(const ftp_model* m, int32_t which, int32_t unit, float* dst, int64_t count,
                          int32_t dst_is_device, void* stream);

/* ---- run_stage(a, b, micro_batch): Sec. III-B / III-C.  -------------------------------- */

/* Forward of units [a, b) on one micro-batch.
 *   act_in  : device; the input batch (a == 0) or the boundary activation leaving unit a-1.
 *   act_out : device; receives the boundary activation leaving unit b-1; must be NULL when
 *             b == L (the last unit ends in the loss).
 *   labels  : device int32[batch], required iff b == L.  Device-resident labels are not validated:
 *             a label outside [0, n_classes) is treated as the nearest valid class.
 *   loss_out: device float[1], required iff b == L; mean softmax cross-entropy.
 * act_in and act_out must stay valid and unmodified until the backward pass of the same
 * range has completed (they are read again there; nothing is copied).  Updates the BN
 * running statistics of the range. */
ftp_status ftp_run_stage_forward(ftp_model* m, int32_t a, int32_t b, const void* act_in, void* act_out,
                                 const int32_t* labels, float* loss_out, void* stream);

/* Backward of units [a, b) using the values stashed by the last forward of the same range.
 *   grad_out: device; gradient of the loss w.r.t. the boundary activation leaving unit b-1
 *             (same shape and type); must be NULL when b == L.
 *   grad_in : device; receives the gradient w.r.t. act_in; may be NULL when a == 0.
 * Leaves the weight gradients of the range in the gradient arena (float).  Every reduction
 * has a fixed order: results do not depend on how the units are grouped into stages. */
ftp_status ftp_run_stage_backward(ftp_model* m, int32_t a, int32_t b, const void* grad_out, void* grad_in,
                                  void* stream);

/* Device copy of the logits (float[batch * n_classes]) of the last forward that reached L. */
ftp_status ftp_get_logits(const ftp_model* m, float* dst, int32_t dst_is_device, void* stream);

/* SGD with momentum and weight decay on units [a, b) (Sec. IV-B):
 *   g <- g + wd*w ;  m <- g on a unit's first update, else mu*m + g ;  w <- w - lr*m
 * for every trainable parameter, refreshing the bf16 shadow.  When snap_dev / snap_host are
 * non-NULL the same kernel also stores the updated weights there (device buffer / pinned
 * host buffer mapped into the device address space), laid out as the trainable spans of
 * units a..b-1 back to back (the fused half of a replication tick, Sec. III-E). */
ftp_status ftp_sgd_step(ftp_model* m, int32_t a, int32_t b, float lr, float* snap_dev, float* snap_host,
                        void* stream);

/* One synchronous training step over the current partition: forward through every stage,
 * backward through every stage, SGD on every stage; internal boundary buffers.
 *   x, labels   : the input batch and int32 labels; host (pinned or pageable) when
 *                 inputs_on_host != 0 -- they are then copied to the device inside the call, and a
 *                 label outside [0, n_classes) is refused with FTP_ERANGE before anything is
 *                 launched -- else device (labels then clamp as in ftp_run_stage_forward).
 *   loss_host   : if non-NULL (host float[1]) the loss is copied back and the call returns
 *                 after the step has completed; if NULL the call is fully asynchronous.
 * Under stream capture (the caller records the step into a CUDA graph): host inputs must be
 * pinned -- their copies become nodes of the graph and read the same buffers at every replay, and
 * the labels are checked at capture time only (at replay they clamp) -- and loss_host, if
 * non-NULL, must be pinned too: the copy of the loss into it becomes the last node, nothing is
 * synchronised, and the value is valid once a replay has completed.  Record after the model's
 * first update: whether a unit's momentum buffer is initialised or accumulated is decided when
 * the step is recorded, and so are lr and the partition. */
ftp_status ftp_train_step(ftp_model* m, const void* x, const int32_t* labels, int32_t inputs_on_host, float lr,
                          float* loss_host, void* stream);

/* Waits for the stream, reads the device status word (see "Errors" above) and clears it:
 * FTP_OK, or FTP_ETIMEOUT if a bounded device-side wait ran out since the last check. */
ftp_status ftp_check_device_status(ftp_model* m, void* stream);
/* Memory-safety check (the workspace's stand-in for a memory checker): every buffer the model carves out of dev_ws is
 * followed by a 256-byte guard zone holding a fixed pattern since ftp_build_model.  Waits for the stream, reads all
 * zones back and returns FTP_ESTATE (text: which zone, at which workspace offset) if a kernel has written past the end
 * of a buffer; *first_bad_offset (nullable) = that offset or -1, *n_guards (nullable) = zones checked. */
ftp_status ftp_check_guards(ftp_model* m, int32_t* n_guards, int64_t* first_bad_offset, void* stream);
/* Test hook: writes `code` into the device status word from the host, as a kernel whose wait ran
 * out would (0 clears it).  No kernel is launched.  Synchronises the stream. */
ftp_status ftp_debug_set_device_status(ftp_model* m, int32_t code, void* stream);

/* ---- profile_layers(): Sec. III-B "model profiling" and Sec. III-D "execution profiling". */

/* Runs `reps` forward+backward passes of the whole model on the sample batch (device
 * pointers) and returns, per unit, the mean forward and backward device time in seconds and
 * the size in bytes of its output (host arrays of L entries).  Weight values are left
 * unchanged (no optimiser step) but BN running statistics are restored afterwards.
 * Synchronises the stream. */
ftp_status ftp_profile_layers(ftp_model* m, int32_t reps, const void* sample_in, const int32_t* labels,
                              double* fwd_s, double* bwd_s, int64_t* out_bytes, void* stream);

/* Sec. III-B / III-D: every worker reports the execution time of its batches, from which the central
 * node estimates capacities (Eq. 1).  With stage timing on, ftp_train_step brackets every stage's
 * forward and backward with events (issued eagerly: not for steps replayed from a CUDA graph);
 * ftp_stage_times waits for the last such step and returns forward + backward device seconds per
 * stage of the partition it ran under (seconds: max_stages doubles; *n_stages: how many are set).
 * The optimiser step is not included, as in ftp_profile_layers.  FTP_ESTATE if no step was timed. */
ftp_status ftp_stage_timing_enable(ftp_model* m, int32_t on);
ftp_status ftp_stage_times(ftp_model* m, double* seconds, int32_t* n_stages);

/* Sec. III-B "the i-th worker measures the bandwidth between itself and its next worker": the B_{i,i+1} of
 * Eq. 5, as this machine has them.  Times `reps` copies of min(bytes, the model's scratch size) bytes with CUDA
 * events: between two device buffers of the workspace (what a boundary activation or a chain replica crosses
 * when stages share one GPU) and, if pinned_host is non-NULL (pinned host memory of at least `bytes` bytes),
 * from the device to it (the path of the global replica to the central node).  Results in bytes per second;
 * *d2h_bytes_per_s = 0 without a host buffer.  Synchronises the stream; call it between steps. */
ftp_status ftp_measure_bandwidth(ftp_model* m, void* pinned_host, size_t bytes, int32_t reps, double* d2d_bytes_per_s,
                                 double* d2h_bytes_per_s, void* stream);

/* Eq. 1-3: capacities[i] = stage_times[i] / sum of layer_times over stage i; [0] = 1.0. */
ftp_status ftp_estimate_capacity(const double* layer_times, int32_t L, const int32_t* points, int32_t N,
                                 const double* stage_times, double* capacities);

/* ---- choose_partition(layer_times, capacities): Eq. 4-7.  Pure host function.
 *   layer_times[L] : T^0_{e,j}; capacities[N] : C_i (a slowdown multiplier).
 *   out_bytes[L], bandwidth[N-1] : D_j and B_{i,i+1}; both NULL drops the 2*T_c term.
 *   points_out[N+1], bottleneck_out : the optimal boundaries and A(L-1, N).
 * Every stage is non-empty (N > L is FTP_EINVAL).  Among optimal partitions the one returned
 * takes, from the last cut backwards, the smallest cut index reaching the optimum. */
ftp_status ftp_choose_partition(const double* layer_times, int32_t L, const double* capacities, int32_t N,
                                const double* out_bytes, const double* bandwidth, int32_t* points_out,
                                double* bottleneck_out);

/* Algorithm 1 for one worker.  p_cur has n_cur+1 entries (old worker list), p_new n_new+1.
 * i_cur: the worker's old index (-1 if it held nothing), i_new: its new index, i_fail: the
 * failed old index or -1.  owner_of_needed[k] (k over the new range p_new[i_new] ..) is the
 * index, in the NEW worker list, to fetch unit p_new[i_new]+k from, or -1 if it is held
 * locally; *n_local counts the local ones. */
ftp_status ftp_redistribution_plan(const int32_t* p_new, int32_t n_new, const int32_t* p_cur, int32_t n_cur,
                                   int32_t i_fail, int32_t i_cur, int32_t i_new, int32_t* owner_of_needed,
                                   int32_t* n_local);

/* Install a new partition (Sec. III-D "weight redistribution"): every stage computes its
 * Algorithm-1 plan, the spans of the units that change owner (weights, momentum, running
 * statistics, shadow) are copied between stage arenas on the stream, and only after all
 * copies are enqueued does the owner table switch (the commit).  moved_units (nullable)
 * receives how many units changed owner. */
ftp_status ftp_set_partition(ftp_model* m, const int32_t* points, int32_t n_stages, int32_t* moved_units,
                             void* stream);
ftp_status ftp_get_partition(const ftp_model* m, int32_t* points /* max_stages+1 */, int32_t* n_stages);

/* ---- recovery from worker failures: Sec. III-F.  --------------------------------------------
 * A failure is a host-side event here (all stages share one GPU): the caller names the stages
 * whose memory is to be treated as lost; nothing on the device is faulted. */

/* Where a unit's weights come from after failures (pure host function).  failed[n_failed]:
 * distinct old indices in 1 .. n_cur-1 (worker 0 is the central node and does not fail); the
 * survivors keep their order and become 0 .. n_new-1, n_new = n_cur - n_failed.  For every unit u
 * of the model: kind[u] is FTP_SRC_LOCAL (its new owner holds it already), FTP_SRC_STAGE (the live
 * weights of surviving worker index[u], new numbering), FTP_SRC_REPLICA (the chain replica of the
 * failed worker that held u, kept by the worker after it, index[u] in the new numbering, 0 = the
 * central node for the last worker) or FTP_SRC_CENTRAL (the global replica on the central node:
 * the keeper of the chain replica failed too).  With one failure this is Algorithm 1. */
enum { FTP_SRC_LOCAL = 0, FTP_SRC_STAGE = 1, FTP_SRC_REPLICA = 2, FTP_SRC_CENTRAL = 3 };
ftp_status ftp_recovery_plan(const int32_t* p_cur, int32_t n_cur, const int32_t* failed, int32_t n_failed,
                             const int32_t* p_new, int32_t n_new, int32_t* kind /* L */, int32_t* index /* L */);

/* One failed stage and its chain replica: the bytes ftp_snapshot_weights(stage) wrote under the
 * partition that is current now (device memory, or host memory for the last stage, whose replica
 * the central node keeps).  replica may be NULL when none exists. */
typedef struct {
    int32_t stage;
    int32_t replica_is_host;
    const void* replica;
    size_t replica_bytes;
} ftp_failed_stage;

/* Recover and re-partition (Sec. III-F): the failed stages' arenas are abandoned, the survivors
 * are renumbered in order, and the model is spread over them at p_new (n_new = stages - n_failed
 * boundaries + 1, normally from ftp_choose_partition).  Per unit, following ftp_recovery_plan:
 * local units stay where they are, units of other survivors are copied between arenas with their
 * momentum, units of a failed stage are loaded from its chain replica (weights and BN running
 * statistics as of that replica; their momentum restarts from the next gradient) or, when the
 * replica's keeper failed too or no replica was given, from `central`: the global replica, all
 * units in canonical order, host memory, nullable.  A unit with no source left is FTP_ESTATE and
 * nothing is changed.  The owner table switches only after every copy is enqueued (the commit);
 * forward state of all units is discarded, as the paper discards the batches in flight.
 * counts (nullable): units taken from other stages, from chain replicas, from the global replica.
 * A replica must have been taken under the current partition (its size is checked). */
ftp_status ftp_recover(ftp_model* m, const ftp_failed_stage* failed, int32_t n_failed, const void* central,
                       size_t central_bytes, const int32_t* p_new, int32_t n_new, int32_t* counts /* 3 */,
                       void* stream);

/* ---- training state of a node and the fault handler of the central node: Sec. III-B (Table I), Sec. III-F.
 * Pure host functions; nothing on the device is involved.
 *
 * Table I: every node holds the committed forward id and the committed backward id (the latest batch
 * that has completed forwarding / backwarding; both start at -1), the learning rate, the epoch and batch
 * numbers, and `status` (0 normal, 1 fault recovery). */
typedef struct {
    int64_t committed_forward_id, committed_backward_id;
    int32_t status;
    float learning_rate;
    int64_t epoch_number, batch_number;
} ftp_train_state;
ftp_status ftp_state_init(ftp_train_state* st, float learning_rate, int64_t epoch_number, int64_t batch_number);
ftp_status ftp_state_forward_done(ftp_train_state* st, int64_t batch_id);
ftp_status ftp_state_backward_done(ftp_train_state* st, int64_t batch_id);
/* The central node's timer for batch_id ran out before its gradients came back.  *triggered = 1 and
 * status becomes 1 if the handler was not running yet; 0 if it was (later timers do not start it again). */
ftp_status ftp_state_timer_expired(ftp_train_state* st, int64_t batch_id, int32_t* triggered);
/* *allowed = 0 while status is 1 for batches beyond the committed forward id: they were sent before the
 * sub-models were rebuilt and are discarded. */
ftp_status ftp_state_may_forward(const ftp_train_state* st, int64_t batch_id, int32_t* allowed);
/* Last phase of the handler: both committed ids become batch_id (the batch whose gradients were not
 * received), status returns to 0; *resume_from (nullable) = the batch to forward first, batch_id. */
ftp_status ftp_state_reset(ftp_train_state* st, int64_t batch_id, int64_t* resume_from);

/* The three outcomes of the handler's probe.  responses[n_workers]: how each worker of the list answered
 * (worker 0 is the central node and answers normally).  All normal -> FTP_ACTION_RESTART_BATCH.  All answer
 * and exactly one has restarted -> FTP_ACTION_RESEND_STATE, *restarted_worker = its index (it is sent the
 * state variables and reloads its weights from the replica its neighbour keeps).  Otherwise ->
 * FTP_ACTION_REDISTRIBUTE with failed[0 .. *n_failed) = the workers that were silent or, beside other
 * faults, restarted (their weights are lost either way), ascending: the input of ftp_recovery_plan. */
enum { FTP_PROBE_NORMAL = 0, FTP_PROBE_RESTARTED = 1, FTP_PROBE_SILENT = 2 };
enum { FTP_ACTION_RESTART_BATCH = 0, FTP_ACTION_RESEND_STATE = 1, FTP_ACTION_REDISTRIBUTE = 2 };
ftp_status ftp_classify_probe(const int32_t* responses, int32_t n_workers, int32_t* action, int32_t* failed /* n_workers */,
                              int32_t* n_failed, int32_t* restarted_worker);

/* Schedules (Sec. III-D, IV-B): 1 if, after the 0-indexed batch `it` has finished, the dynamic partition
 * runs (after `first` batches, then whenever the count is a multiple of `period`; the paper uses 10 and
 * 100) / a replication with the given period runs (chain 50, global 100 in the paper's runs). */
int32_t ftp_is_repartition_iter(int64_t it, int64_t first, int64_t period);
int32_t ftp_is_replication_iter(int64_t it, int64_t period);

/* ---- asynchronous pipeline training: Sec. III-C (1F1B, weight stashing, vertical sync, weight aggregation).
 *
 * The order of passes and the version numbers are pure host functions.  On the device a weight version of a
 * stage is the set of parameter spans of its units inside one model object; several models built from the same
 * layer list (each with a workspace of its own) hold the versions and the activations of the batches in flight,
 * and the three calls below move and combine versions between them.  A driver (paper_2110_02781_b200/async_pipeline.py)
 * strings them together with ftp_run_stage_forward / ftp_run_stage_backward. */

/* 1F1B on `stage` of n_stages: the stage forwards min(n_stages - stage, n_batches) batches, then a backward and a
 * forward pass alternate, then the remaining backward passes.  is_backward[e], batch[e] for e < 2 * n_batches. */
ftp_status ftp_async_stage_order(int32_t n_stages, int32_t stage, int32_t n_batches, int32_t* is_backward, int32_t* batch);
/* Version counter of a stage taken by itself (as on stage 0): starts at 0, every backward pass adds one; after the
 * forward pass that follows every (k_interval * (n_stages - stage))-th update the n_stages - stage stashed versions
 * are aggregated, which adds one more (no aggregation on the last stage, which has a single version).
 * forward_version[b]: version batch b is forwarded (and, weight stashing, backwarded) with;
 * version_after_backward[b]; aggregate_after_forward[b] = 1 where an aggregation follows F_b.  n_batches entries each. */
ftp_status ftp_async_version_trace(int32_t n_stages, int32_t stage, int32_t n_batches, int32_t k_interval, int64_t* forward_version,
                                   int64_t* version_after_backward, int32_t* aggregate_after_forward);

/* Copy, for units [a, b), what `what` selects (a mask) from src to dst: float master weights (the copies the kernels
 * read are rebuilt), momentum buffers, BN running statistics.  Both models must come from the same layer list.
 * Device-to-device, asynchronous on the stream. */
enum { FTP_SYNC_WEIGHTS = 1, FTP_SYNC_MOMENTUM = 2, FTP_SYNC_STATE = 4 };
ftp_status ftp_sync_units(ftp_model* dst, const ftp_model* src, int32_t a, int32_t b, int32_t what, void* stream);
/* ftp_sgd_step on dst's weights and momentum of units [a, b) with the gradients that the last backward pass of
 * `grads` left in ITS gradient arena: the update of the latest weights by a gradient taken at stashed ones. */
ftp_status ftp_sgd_step_from(ftp_model* dst, const ftp_model* grads, int32_t a, int32_t b, float lr, void* stream);
/* Weight aggregation: for units [a, b), dst's master weights and BN running statistics become the arithmetic mean of
 * those of srcs[0 .. n_src) (1..8 models, added in that order; dst may be one of them); momentum is left alone. */
ftp_status ftp_aggregate_weights(ftp_model* dst, const ftp_model* const* srcs, int32_t n_src, int32_t a, int32_t b, void* stream);

/* ---- snapshot_weights(stage, dst): Sec. III-E chain / global replication. ----------------- */

/* Copy stage's replica -- per unit of the stage, in order: trainable weights then BN running
 * statistics, float -- to dst (device, or host when dst_is_host).  *written = bytes copied.
 * Asynchronous for device and pinned-host destinations. */
ftp_status ftp_snapshot_weights(const ftp_model* m, int32_t stage, void* dst, size_t dst_bytes,
                                int32_t dst_is_host, size_t* written, void* stream);

/* ---- measurement aids ---------------------------------------------------------------------- */

/* While enabled, every kernel launch is bracketed by CUDA events on its stream and recorded.
 * ftp_trace_read synchronises, copies up to max records (in launch order) and clears the
 * log; *total is the number that were logged. */
ftp_status ftp_trace_enable(ftp_model* m, int32_t on);
ftp_status ftp_trace_read(ftp_model* m, ftp_trace_rec* out, int32_t max, int32_t* total);
const char* ftp_kernel_name(int32_t kernel);
/* Number of kernel launches issued by this model since it was built. */
ftp_status ftp_launch_count(const ftp_model* m, int64_t* launches);

/* ---- for callers that cannot allocate ------------------------------------------------------------
 * (The paper has no counterpart: this is a packaging variant of the weight-gradient step of
 * run_stage's backward pass.)
 *
 * dw[k][k][cin][cout] = sum over output pixels of x (shifted by the tap) times dy, for a dense
 * k x k convolution with the given stride and padding on float tensors x (n, h, w, cin) and
 * dy (n, ho, wo, cout), all device pointers, 16-byte alignment recommended.
 *
 * Unlike every other call, this one takes no workspace: the partial sums of its split reduction go
 * to an 8 MiB array that is part of the library's device image (each GPU that loads the library
 * holds it until the process exits).  It is meant for callers that get input and output buffers
 * and may not call cudaMalloc themselves: a stage running inside a stream-ordered region where an
 * allocation would stall the device, or a host framework that owns all device memory.  The call
 * itself allocates nothing, on the host or on the device.
 *   - Shapes whose partials exceed the array are refused with FTP_ERANGE (use the model API).
 *   - The first call on a device looks the array's address up (the device must be current).  With
 *     CUDA's lazy module loading that look-up is also what places the array on the device: an
 *     implicit allocation that may synchronise the device.  So make that first call during set-up
 *     -- any small shape will do -- before entering the region that must not allocate, and outside
 *     any stream capture.  Later calls on that device only read a cached pointer (published
 *     atomically, so concurrent first calls from several host threads are safe).
 *   - All calls on a device share the array: calls whose kernels may overlap on the GPU (different
 *     streams) race on it.  Nothing needs clearing between calls.
 * Asynchronous on the stream. */
ftp_status ftp_conv_wgrad_static(const float* x, const float* dy, float* dw, int32_t n, int32_t h, int32_t w,
                                 int32_t cin, int32_t cout, int32_t k, int32_t stride, int32_t pad, void* stream);

const char* ftp_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FTPIPE_H */
