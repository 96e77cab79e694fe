/*
 * hpf.h -- C ABI of the B200 (sm_100a) library for the partitioned, micro-batch
 * pipelined training step of HyPar-Flow (arXiv 1911.05146).
 *
 * A network is a list of ops (Section 5.1: the model as a list of layers).  The
 * list is cut into consecutive partitions (Section 5.1); each partition becomes
 * one pipeline stage bound to one CUDA stream.  A batch is split into
 * micro-batches that flow through the stages (Section 5.3, "pipeline stages
 * within each minibatch").  Activations cross a cut forward and partial errors
 * cross it backward (Section 5.2, Eq. 5-7; Section 5.3 send/recv); on one GPU
 * the hand-off is an event on a shared device buffer.  Per-micro-batch weight
 * gradients land in their own slot and are averaged at the end (the arithmetic
 * of the gradient allreduce of Section 5.3).
 *
 * Conventions
 *   - Every function returns HPF_OK (0) or a negative hpf_status.  Nothing
 *     aborts, nothing throws across this boundary.
 *   - "d_" arguments are DEVICE pointers, "h_" arguments are HOST pointers,
 *     everything else is host memory owned by the caller for the duration of
 *     the call only.
 *   - The library allocates no device memory (the one exception is stated at
 *     its declaration): parameters, gradient buffers and the workspace belong
 *     to the caller, as do the streams.
 *   - Tensors are fp32, channels innermost: activations [n][h][w][c], conv
 *     weights [c_out][r][s][c_in].
 *   - The step calls (forward, backward, grad_average) only enqueue work.
 *     hpf_loss and hpf_synchronize wait for it.
 *   - There is no CPU fallback: without a CUDA device the step calls fail with
 *     HPF_ERR_CUDA.
 */
#ifndef HPF_H_
#define HPF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hpf_model hpf_model; /* opaque, host side */

typedef enum {
    HPF_OK = 0,
    HPF_ERR_INVALID = -1,     /* null pointer, bad cut list, B % M != 0, malformed op list, shape mismatch */
    HPF_ERR_UNSUPPORTED = -2, /* a shape no kernel covers (e.g. BN channels not a multiple of 4) */
    HPF_ERR_STATE = -3,       /* call order: backward before forward, average before backward, not bound */
    HPF_ERR_WORKSPACE = -4,   /* workspace too small or misaligned */
    HPF_ERR_CUDA = -5,        /* a CUDA call failed; text via hpf_last_error */
    HPF_ERR_TIMEOUT = -6      /* hpf_synchronize deadline passed, or a bounded device-side wait gave up */
} hpf_status;

typedef enum { HPF_OP_CONV = 1, HPF_OP_BNRELU = 2, HPF_OP_ADD = 3, HPF_OP_MAXPOOL = 4, HPF_OP_HEAD = 5, HPF_OP_BN = 6,
               HPF_OP_RELU = 7 } hpf_op_kind;

/* One entry of the layer list.
 *   CONV    cross-correlation, zero padding, no bias: ksize x ksize, stride, pad; c_in -> c_out
 *   BNRELU  training-mode batch norm over the micro-batch (biased variance) followed by ReLU; c_in == c_out
 *   BN      the same batch norm without the activation, RELU the activation alone (max(x, 0), derivative 0 at 0): the
 *           post-activation residual block is CONV BNRELU CONV BN, ADD with the shortcut, RELU; c_in == c_out
 *   ADD     src0 + src1 (residual join)
 *   MAXPOOL ksize x ksize window, stride, pad (padding never wins)
 *   HEAD    mean over (h,w), fully connected to c_out classes, softmax cross-entropy, mean over the
 *           micro-batch (Eq. 2 with the cross-entropy loss).  Must be the last op and only the last. */
typedef struct {
    int32_t kind;        /* hpf_op_kind */
    int32_t src0, src1;  /* index of the producing op, -1 = the network input; src1 only for ADD, else -1 */
    int32_t c_in, c_out;
    int32_t ksize, stride, pad;
    float eps;           /* BNRELU */
} hpf_op;

/* ---- model (host only; no CUDA call) -------------------------------------------------------------
 * Section 5.1.  in_shape = {B, H, W, C}.  cuts = P-1 strictly increasing op indices in [1, n_ops-1];
 * partition p owns ops [cuts[p-1], cuts[p]).  A cut may fall anywhere, also inside a residual block.
 * n_microbatches = M must divide B (Section 5.3: between 1 and the batch size).
 * Errors: HPF_ERR_INVALID for a malformed list / cuts / M; HPF_ERR_UNSUPPORTED for a shape outside
 * the kernels' reach.  *out is set only on success; release it with hpf_model_destroy. */
int hpf_model_create(const hpf_op *ops, int32_t n_ops, const int32_t in_shape[4], const int32_t *cuts,
                     int32_t n_cuts, int32_t n_microbatches, hpf_model **out);
int hpf_model_destroy(hpf_model *model);

/* Options, to be set before hpf_workspace_bytes / hpf_bind.
 *   HPF_OPT_GRAPH          1 (default): each phase is captured once into a CUDA graph and replayed;
 *                          0: kernels are enqueued directly on the streams every call.
 *   HPF_OPT_CONV_PATH      0 (default): tensor-core (tcgen05) convolution kernels wherever the shape
 *                          allows, error-compensated three-pass TF32 (fp32-class accuracy), CUDA-core
 *                          kernels for the rest (3-channel stem, odd channel counts);
 *                          1: CUDA-core kernels everywhere (fp32 FMA; a cross-check, not a fallback);
 *                          2: as 0 with a single TF32 pass (11-bit operands; error grows with depth).
 *   HPF_OPT_SINGLE_STREAM  1: all stages on stream 0 (hazard check: results must equal the multi-stream run).
 *   HPF_OPT_KEEP_MESSAGES  1: every partition copies what it receives across a cut (activations forward,
 *                          partial errors backward) into message buffers readable with hpf_message_ptr.
 *   HPF_OPT_FUSE_ADD       1 (default): a residual ADD is computed in the epilogue of the later of its two
 *                          producers when that is a convolution nothing else reads, in the same partition;
 *                          that convolution's own output is then not stored (hpf_tensor_ptr answers
 *                          HPF_ERR_STATE for it).  0: every op's output is stored.
 *   HPF_OPT_PDL            1 (default): hot kernels use programmatic dependent launch (a kernel is scheduled and runs
 *                          its set-up while its predecessor in the stream drains).  0: plain stream-ordered launches.
 *   HPF_OPT_WGRAD_PASSES   1 (default) or 3: TF32 passes of the tensor-core weight gradient.  A weight gradient feeds
 *                          nothing but the average, so its rounding error (about 8e-4 relative with one pass) does not
 *                          compound with depth the way forward and data-gradient errors do; those always follow
 *                          HPF_OPT_CONV_PATH.
 *   HPF_OPT_FUSE_BN        bit 0: the per-channel sums of a BN's forward statistics are formed in the write-out of the
 *                          tensor-core convolution kernel that produces the BN's input, when both run back to back on
 *                          one stream; the BN forward is then one kernel.  bit 1 (needs bit 0): a BN+ReLU whose output
 *                          only the next op reads, a stride-1 tensor-core convolution of the same partition, has no
 *                          kernel of its own: that convolution derives the statistics from the per-tile sums, applies
 *                          the BN+ReLU to its input tile on the way to the tensor core and stores the BN's output and
 *                          statistics as a by-product.  0: every BN runs its own kernels.  Default 3.
 *   HPF_OPT_CELL_TIMES     1: a one-thread kernel stores the device's nanosecond timer at the start and at the end of
 *                          every (partition, micro-batch) cell of the forward and backward schedules (Section 5.3's
 *                          pipeline, as it really ran); read them with hpf_cell_times.  Default 0.
 *   HPF_OPT_BN_CLUSTER     1 (default): the backward of a BN whose micro-batch tensor is small enough to sit in the
 *                          registers of a few thread-block clusters is one launch (the CTAs of a cluster exchange their
 *                          per-channel sums through distributed shared memory); 0: always the reduce + apply pair.
 *   HPF_OPT_PDL_LATE_FROM  N (default 8): with programmatic dependent launch, the forward convolutions of a cell that runs while at
 *                          least N cells of the one-graph schedule are under way let their successor be scheduled only when
 *                          their accumulator is complete, not at their first instruction: a successor scheduled early sits in
 *                          its SM slots for the whole life of its predecessor, which shortens a lone stage's chain of kernels
 *                          but costs throughput once every stage is busy.  0: always late; a large N: always early.
 *   HPF_OPT_STAGE_LANES    L (default 1): a stage keeps up to L of its micro-batches under way at once, micro-batch m on lane
 *                          m mod L, every lane with its own streams and scratch memory.  L = 1 is the schedule of Section 5.3
 *                          as the paper's one-process-per-partition runs it: a stage works through its micro-batches one
 *                          after the other, and P + M - 1 ticks pass before the last cell ends.  On one GPU the stages share
 *                          the same SMs, so nothing forces that order: with L > 1 the cells (p, m) and (p, m + 1) may run side
 *                          by side, the hand-offs between stages are unchanged, and the idle slots of the pipeline's fill and
 *                          drain get used.  Every cell computes on the same data with the same kernels: results are
 *                          bit-identical for every L.  hpf_bind then wants its streams per (partition, lane).
 *   HPF_OPT_WGRAD_DIRECT   1 (default): the tensor-core weight gradient hands its TMA tiles (pixels x channels, channels
 *                          innermost) to the tensor core as MN-major operands, as they land in shared memory; 0: the earlier
 *                          kernel, which transposes every tile in shared memory first (kept as a cross-check; also used for
 *                          channel counts that are neither 16 nor a multiple of 32).
 *   HPF_OPT_CELL_CTAS      N > 0: the forward tensor-core convolutions of a (partition, micro-batch) cell that follow each
 *                          other with no other kernel between them run as ONE persistent kernel of N CTAs that stays
 *                          resident for the cell, walks the list of convolutions and meets at a grid-wide barrier between
 *                          them (Section 5.3's stage as one resident grid instead of a chain of launches).  The cells of
 *                          all partitions must fit the GPU together (hpf_bind: HPF_ERR_UNSUPPORTED otherwise).  Results
 *                          are bit-identical to N = 0 when the tile assignment is the same.  0: one launch per convolution. */
typedef enum { HPF_OPT_GRAPH = 1, HPF_OPT_CONV_PATH = 2, HPF_OPT_SINGLE_STREAM = 3, HPF_OPT_KEEP_MESSAGES = 4,
               HPF_OPT_FUSE_ADD = 5, HPF_OPT_PDL = 6, HPF_OPT_WGRAD_PASSES = 7, HPF_OPT_FUSE_BN = 8, HPF_OPT_CELL_TIMES = 9,
               HPF_OPT_BN_CLUSTER = 10, HPF_OPT_CELL_CTAS = 11, HPF_OPT_PDL_LATE_FROM = 12,
               HPF_OPT_STAGE_LANES = 13, HPF_OPT_WGRAD_DIRECT = 14 } hpf_option;
int hpf_set_option(hpf_model *model, int32_t option, int32_t value);

/* ---- integer bookkeeping (Section 5.1 lists, Section 5.3 pipelining) ----------------------------- */
int hpf_num_ops(const hpf_model *model, int32_t *n_ops);
int hpf_num_partitions(const hpf_model *model, int32_t *P);
/* S = P * min(HPF_OPT_STAGE_LANES, M): hpf_bind takes S, 2S or 3S streams */
int hpf_num_stream_slots(const hpf_model *model, int32_t *S);
int hpf_num_params(const hpf_model *model, int64_t *G);
/* Offsets (in floats) into the flat parameter / gradient vectors: ops in list order; CONV weights
 * [c_out][r][s][c_in]; BNRELU gamma[C] then beta[C]; HEAD W[classes][C] then bias[classes]. */
int hpf_param_layout(const hpf_model *model, int32_t op, int64_t *w_off, int64_t *w_cnt, int64_t *b_off, int64_t *b_cnt);
int hpf_op_shape(const hpf_model *model, int32_t op, int32_t hwc[3]);
int hpf_partition_of_op(const hpf_model *model, int32_t op, int32_t *p);
int hpf_partition_range(const hpf_model *model, int32_t p, int32_t *first_op, int32_t *end_op);
int hpf_microbatch_range(const hpf_model *model, int32_t m, int32_t *first, int32_t *end);
/* The tensors crossing cut `cut` (0-based): produced before it, read at or after it (Section 5.3,
 * Forward/Backward lists), ascending producer index. */
int hpf_boundary_count(const hpf_model *model, int32_t cut, int32_t *n);
int hpf_boundary_desc(const hpf_model *model, int32_t cut, int32_t i, int32_t *producer_op, int32_t shape[4] /* b,H,W,C */);
/* Fill/drain pipeline: forward (p,m) runs at tick p+m, backward (p,m) at tick (P-1-p)+m. */
int hpf_schedule_tick(const hpf_model *model, int32_t p, int32_t m, int32_t *fwd_tick, int32_t *bwd_tick);

/* ---- load balancer (Section 5.4 names the component and leaves it to future work) -----------------
 * hpf_estimate_op_costs: modelled time (microseconds, forward + backward on the pipeline's critical chain) of every op
 * for one micro-batch of b samples: a fixed latency per kernel, a term per tensor-core K step and a term per byte
 * moved, with constants calibrated on B200 at micro-batch 16 (weight gradients run beside the chain and are not
 * counted).  Host only.  cost_us: n_ops doubles.
 * hpf_balance_cuts: P-1 cut points that minimise the largest partition cost (contiguous partitions, every
 * partition non-empty).  Any non-negative costs may be passed (measured ones, too).  Host only. */
int hpf_estimate_op_costs(const hpf_op *ops, int32_t n_ops, const int32_t in_shape[4] /* b,H,W,C */, double *cost_us);
int hpf_balance_cuts(const double *cost, int32_t n_ops, int32_t n_partitions, int32_t *cuts /* P-1 */);

/* ---- device resources ---------------------------------------------------------------------------- */
int hpf_workspace_bytes(const hpf_model *model, size_t *bytes);
/* d_params [G], d_grad_slots [M][G] (slot m = dL_m/dtheta), d_grad_avg [G], d_workspace (256-byte
 * aligned, >= hpf_workspace_bytes): all caller-owned device memory that must outlive the model.
 * cuda_streams: n_streams >= P cudaStream_t handles (stage p runs on stream p; stream 0 is the one
 * the phases fork from and join to).  With n_streams >= 2P, stream P+p carries stage p's weight-gradient
 * kernels, which feed only the final average and so leave the chain of dependent kernels; with n_streams >= 3P,
 * stream 2P+p carries stage p's backward cells in hpf_forward_backward.  With HPF_OPT_STAGE_LANES = L > 1 read
 * S = P * min(L, M) for P throughout: lane l of stage p is stream slot p * min(L, M) + l.  Creates
 * events and tensor-map descriptors; allocates nothing on the device.  Errors: HPF_ERR_WORKSPACE, HPF_ERR_INVALID, HPF_ERR_CUDA. */
int hpf_bind(hpf_model *model, float *d_params, float *d_grad_slots, float *d_grad_avg, void *d_workspace,
             size_t ws_bytes, void *const *cuda_streams, int32_t n_streams);

/* ---- the step ------------------------------------------------------------------------------------ */
/* Section 5.3 forward pass: every (partition p, micro-batch m) in pipeline order.  d_x [B][H][W][C]
 * fp32, d_labels [B] int32 in [0, classes); both must already be valid for work ordered after
 * stream 0's current tail, and stay valid until the backward work has finished. */
int hpf_forward(hpf_model *model, const float *d_x, const int32_t *d_labels);
/* Section 5.2 Eq. 5-7: reverse sweep, last partition first; writes slot m of d_grad_slots. */
int hpf_backward(hpf_model *model);
/* hpf_forward and hpf_backward as ONE set of dependencies (Section 5.3: a stage works as soon as what it needs has
 * arrived): the backward cell (p, m) starts when the cell that feeds it has finished - backward (p+1, m), or forward
 * (P-1, m) for the last partition - instead of after the whole forward pass, so the backward pipeline fills while the
 * forward pipeline drains.  The same kernels run on the same data: every result is bit-identical to hpf_forward followed
 * by hpf_backward.  With n_streams >= 3P at hpf_bind, stream 2P+p carries partition p's backward cells, beside its
 * forward cells on stream p; with fewer streams the call is hpf_forward followed by hpf_backward in one graph.
 * Leaves the model where hpf_backward does (hpf_grad_average / hpf_sgd_momentum_step next; hpf_loss any time after). */
int hpf_forward_backward(hpf_model *model, const float *d_x, const int32_t *d_labels);
/* ---- one cell at a time (Section 5.3: one process per model-partition) ---------------------------------------------
 * The calls a stage-per-GPU run is made of: every GPU binds the same model (same op list, cuts, micro-batch count, hence
 * the same memory plan) and runs only the cells of the partition it owns; what crosses a cut is copied between the GPUs'
 * workspaces, where it lives at the same offset on both sides (hpf_tensor_ptr), by the caller (a peer copy or an NCCL
 * send / recv into the consumer's own memory).  All calls enqueue on partition p's stream (weight gradients on its side
 * stream) without a CUDA graph and without waiting for any other partition: the caller orders the cells.
 *   hpf_prepare_partition  once per step before the partition's first cell: the split / rearranged weights.
 *   hpf_forward_cell       ops of partition p on micro-batch m.  d_x [B][H][W][C]: needed by partition 0 (NULL otherwise);
 *                          d_labels [B]: needed by the last partition.  Reads the activations of the live set of cut p-1
 *                          for micro-batch m (hpf_boundary_desc), which must be in place.
 *   hpf_backward_cell      reverse sweep of partition p on micro-batch m; for p < P-1 the gradient buffers listed by
 *                          hpf_backward_message_desc(cut p) must hold what the partition above computed (Eq. 7).
 *   hpf_join_partition     orders partition p's weight-gradient side stream before what follows on its stream.
 *   hpf_partition_param_range   partition p's contiguous slice of the flat parameter / gradient vectors: the message
 *                          of the per-partition allreduce across replicas (Section 5.3, one communicator per partition).
 *   hpf_backward_message_count / _desc   the gradient buffers (by op: hpf_tensor_ptr(op, m, 1)) that partition p+1 hands
 *                          down across cut p: for every tensor of the live set the buffer that holds the sum over its
 *                          consumers at or above the cut, plus the gradient of a residual add that a kernel below the cut
 *                          folds in on the fly. */
int hpf_prepare_partition(hpf_model *model, int32_t p);
int hpf_forward_cell(hpf_model *model, int32_t p, int32_t m, const float *d_x, const int32_t *d_labels);
int hpf_backward_cell(hpf_model *model, int32_t p, int32_t m);
int hpf_join_partition(hpf_model *model, int32_t p);
int hpf_partition_param_range(const hpf_model *model, int32_t p, int64_t *first, int64_t *count);
int hpf_backward_message_count(const hpf_model *model, int32_t cut, int32_t *n);
int hpf_backward_message_desc(const hpf_model *model, int32_t cut, int32_t j, int32_t *op, int32_t shape[4] /* b,H,W,C */);
/* d_grad_avg = (sum over m ascending of slot m) / M  (Section 5.3: gradients accumulated/averaged). */
int hpf_grad_average(hpf_model *model);
/* The gradient average fused with the parameter update that closes the training step (Section 5.3: the averaged
 * gradients are applied, optimizer.apply_gradients()).  SGD with momentum in the Keras form:
 *     gbar = (sum_m g_m)/M;  g' = gbar + weight_decay*theta;  v <- momentum*v - lr*g';  theta <- theta + v.
 * Reads the bound gradient slots, writes gbar to the bound d_grad_avg and updates the bound d_params and d_velocity
 * (device, G floats, caller-owned, zero before the first step) in place, in one kernel enqueued behind the backward
 * phase.  Needs hpf_backward (HPF_ERR_STATE otherwise); use it INSTEAD of hpf_grad_average.  Hyper-parameters must
 * be >= 0 (HPF_ERR_INVALID). */
int hpf_sgd_momentum_step(hpf_model *model, float *d_velocity, float lr, float momentum, float weight_decay);
/* Waits for the forward work; *h_loss = (1/M) sum_m L_m. */
int hpf_loss(hpf_model *model, float *h_loss);
/* The whole step from HOST buffers (pinned memory recommended): copies h_x / h_labels to the device,
 * runs forward, backward and the average, copies the loss back and waits. */
int hpf_step_host(hpf_model *model, const float *h_x, const int32_t *h_labels, float *h_loss);
/* Waits (polling, timeout_ms <= 0: no limit) for all enqueued work; reports a sticky device-side
 * error flag (bounded waits inside kernels) as HPF_ERR_TIMEOUT. */
int hpf_synchronize(hpf_model *model, int32_t timeout_ms);

/* ---- inspection for parity tests ----------------------------------------------------------------- */
/* Output of op `op` for micro-batch m (want_grad = 0) or dL_m/d(output) (want_grad = 1) as left by the
 * last step.  shape = {b, H, W, C}; the head's output is its logits {b,1,1,classes}. */
int hpf_tensor_ptr(const hpf_model *model, int32_t op, int32_t m, int32_t want_grad, const float **d_ptr, int32_t shape[4]);
/* With HPF_OPT_KEEP_MESSAGES: the i-th tensor received across `cut` for micro-batch m, forward
 * (want_grad = 0: the activation) or backward (want_grad = 1: the partial error, i.e. the sum over
 * the consumers at or after the cut, Eq. 7). */
int hpf_message_ptr(const hpf_model *model, int32_t cut, int32_t i, int32_t m, int32_t want_grad, const float **d_ptr);
/* Per-micro-batch losses L_m (device, M floats). */
int hpf_loss_slots_ptr(const hpf_model *model, const float **d_ptr);
/* Pipeline timeline (needs HPF_OPT_CELL_TIMES=1 and the phase to have run): h_ns[(p*M + m)*2 + {0,1}] = device
 * timer in nanoseconds at the start / end of cell (partition p, micro-batch m) of the last forward (phase 0) or
 * backward (phase 1).  h_ns: host, 2*P*M values.  Synchronises.  HPF_ERR_STATE if the option is off. */
int hpf_cell_times(hpf_model *model, int32_t phase, int64_t *h_ns);

/* Bytes one step (forward + backward + average) has to move between the kernels under the fusions the model's options
 * select: per op what its kernels read and write once (a BN+ReLU applied by the reading convolution and a residual add
 * computed in a convolution's write-out move nothing of their own; the by-products those convolutions store are
 * counted with them), times M, plus the once-per-step weight preparation and the gradient average.  Host only. */
int hpf_step_bytes(const hpf_model *model, double *fused_bytes);
/* Kernel launches (graph kernel nodes count as launches) issued by the step calls since bind. */
int hpf_launch_count(const hpf_model *model, int64_t *n);
/* How many convolution launch sites per phase use the tensor-core path / the CUDA-core path. */
int hpf_conv_path_counts(const hpf_model *model, int64_t *n_tensor, int64_t *n_cuda_core);

/* ---- single kernels on caller buffers (convolution sweep, memory-bound kernel benchmarks) --------
 * All pointers are device pointers, `stream` is a cudaStream_t.  x [N][H][W][C], w [K][R][R][C],
 * y/dy [N][P][Q][K] with P = (H+2*pad-R)/stride+1.  path: 0 = tensor cores, three-pass TF32;
 * 2 = tensor cores, one TF32 pass (both HPF_ERR_UNSUPPORTED when the shape is outside their reach);
 * 1 = CUDA cores; hpf_conv_wgrad also takes 3 and 4: as 0 and 2 with the kernel that transposes its tiles in shared
 * memory instead of handing them to the tensor core as MN-major operands (a cross-check).  d_scratch: caller-owned scratch of at least hpf_conv_scratch_bytes(), zeroed ONCE by the caller (e.g.
 * allocated zeroed) and used by one stream at a time.  Its last 256 bytes are the device status of the tensor-core
 * kernels: a kernel whose bounded wait gives up stores a non-zero code there (first failure wins) and nothing ever
 * clears it.  Launches that split a long K loop over several CTAs keep their tickets in it and leave them at zero.
 * Everything else is written by the call and holds nothing afterwards.
 * d_wprep: the weights as the tensor-core kernels read them, 4*K*R*R*C floats written by
 * hpf_conv_prepare_weights ([hi | lo | rearranged-for-dgrad hi | lo]); ignored (may be NULL) for path 1
 * and by hpf_conv_wgrad. */
int hpf_conv_scratch_bytes(int32_t N, int32_t H, int32_t W, int32_t C, int32_t K, int32_t R, int32_t stride,
                           int32_t pad, size_t *bytes);
int hpf_conv_prepare_weights(const float *d_w, float *d_wprep, int32_t C, int32_t K, int32_t R, void *stream);
int hpf_conv_fwd(const float *d_x, const float *d_w, const float *d_wprep, float *d_y, int32_t N, int32_t H, int32_t W,
                 int32_t C, int32_t K, int32_t R, int32_t stride, int32_t pad, int32_t path, void *d_scratch, void *stream);
int hpf_conv_dgrad(const float *d_dy, const float *d_w, const float *d_wprep, float *d_dx, int32_t N, int32_t H,
                   int32_t W, int32_t C, int32_t K, int32_t R, int32_t stride, int32_t pad, int32_t path,
                   void *d_scratch, void *stream);
int hpf_conv_wgrad(const float *d_x, const float *d_dy, float *d_dw, int32_t N, int32_t H, int32_t W, int32_t C,
                   int32_t K, int32_t R, int32_t stride, int32_t pad, int32_t path, void *d_scratch, void *stream);
/* Fused BN(training)+ReLU over x [rows][C]: d_stats receives mean[C] then 1/sqrt(var+eps)[C].
 * d_scratch: at least hpf_bnrelu_scratch_bytes(rows, C); the caller zeroes its first 256 bytes once (word 0 is a ticket
 * the kernels count on and leave at zero), the calls enqueue kernels only.
 * Tensors of 16 MB and more that fit the registers and shared memory of the whole GPU (16...512 channels, a power of two)
 * are processed by ONE cooperative launch that keeps the tensor on chip between the statistics and the apply step; it
 * occupies every SM while it runs.  That launch synchronises its CTAs through words 0-1 of the scratch; the wait is
 * bounded (2 s): if it ever gives up, word 2 of the scratch becomes 1, d_stats (forward) or d_dgamma / d_dbeta
 * (backward) are NaN and the output is not written; the CTAs that arrived are still counted in word 0, so the caller
 * must zero the first 256 bytes of the scratch again before its next use.  hpf_bnrelu_status copies that flag to the
 * host (it waits for the device).  HPF_BN_RESIDENT=0 in the environment keeps all sizes on the two-kernel path. */
int hpf_bnrelu_scratch_bytes(int64_t rows, int32_t C, size_t *bytes);
int hpf_bnrelu_status(const void *d_scratch, int32_t *h_gave_up);
int hpf_bnrelu_fwd(const float *d_x, const float *d_gamma, const float *d_beta, float eps, float *d_y,
                   float *d_stats, int64_t rows, int32_t C, void *d_scratch, void *stream);
/* dx (+= if accumulate) = BN+ReLU backward of dy; d_addend (may be NULL) is added to dx as well
 * (the shortcut's gradient at a residual fan-out).  d_dgamma / d_dbeta [C] are overwritten. */
int hpf_bnrelu_bwd(const float *d_x, const float *d_dy, const float *d_gamma, const float *d_beta,
                   const float *d_stats, float *d_dx, const float *d_addend, int32_t accumulate,
                   float *d_dgamma, float *d_dbeta, int64_t rows, int32_t C, void *d_scratch, void *stream);
/* The same BN+ReLU forward for callers that cannot allocate device memory or be handed scratch at the
 * time of the call (code inside a no-allocation region: a real-time loop, a stream callback, a plug-in
 * given only its input and output buffers).  The paper has no counterpart; this is a convenience of the
 * library.  The scratch is a fixed array of hpf_static_scratch_bytes() (2 MiB) inside the library's
 * device image: every GPU that loads the library holds it until the process exits.  The call allocates
 * nothing (no cudaMalloc, no cudaFree, no allocating library routine).
 *   - Sizes whose partial sums exceed the array (hpf_bnrelu_scratch_bytes(rows, C) > 2 MiB) are refused
 *     with HPF_ERR_WORKSPACE; nothing is launched.
 *   - The first call on a device looks up the array's device address (that device must be current).
 *     Make that first call outside any stream capture.  Two host threads may make it at the same time.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the call
 *     clears the part that must start at zero.  Two calls whose kernels overlap on the GPU (different
 *     streams, no ordering between them) race on it: order them.
 * Inputs and outputs are the caller's, exactly as for hpf_bnrelu_fwd.  The call always runs the reduce + apply
 * kernel pair and never the one-launch on-chip path, so for tensors of 16 MB and more, where hpf_bnrelu_fwd takes
 * that path, the two agree to rounding (a different summation order), not bit for bit, unless HPF_BN_RESIDENT=0. */
int hpf_bnrelu_fwd_static(const float *d_x, const float *d_gamma, const float *d_beta, float eps, float *d_y,
                          float *d_stats, int64_t rows, int32_t C, void *stream);
int hpf_static_scratch_bytes(size_t *bytes);
/* out[j] = (sum_{m ascending} slots[m][j]) / M */
int hpf_grad_average_flat(const float *d_slots, float *d_out, int32_t M, int64_t G, void *stream);
/* The same update on caller buffers: d_slots [M][G]; d_grad_avg [G] or NULL; d_params, d_velocity [G] updated in place. */
int hpf_sgd_momentum_flat(const float *d_slots, float *d_grad_avg, float *d_params, float *d_velocity, int32_t M, int64_t G,
                          float lr, float momentum, float weight_decay, void *stream);

const char *hpf_strerror(int status);
/* Text of the most recent failure on the calling thread (CUDA error string and call site). */
const char *hpf_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* HPF_H_ */
