/*
 * splitbrain.h - C ABI of the B200 (sm_100a) hot path of SplitBrain hybrid data/model-parallel
 * CNN training: one synchronous SGD iteration in which the 3x3 convolution stack runs
 * data-parallel over R logical replicas of the minibatch and every fully-connected layer is
 * split by output column into K logical model shards whose input is the gathered activations of
 * all replicas.
 *
 * General conventions
 *  - Memory: the caller owns every byte.  The library never allocates device memory; it carves
 *    parameters, momentum, gradients, activations, scratch and status words out of one caller
 *    supplied device arena (size from sb_model_bytes, 256-byte aligned).  Pointers returned by
 *    sb_tensor are borrowed views into that arena and die with it.
 *  - "device" / "host" is stated per pointer argument.  No torch types cross this boundary.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All calls
 *    except sb_model_bytes/create/destroy, sb_loss, sb_tensor_read/write and sb_train_step_host
 *    only enqueue work and return immediately.
 *  - Errors: every call returns an sb_status; nothing throws, aborts or traps.  Argument and shape
 *    errors are detected before any launch.  sb_last_error() gives a thread-local message.
 *  - Layouts: images and conv activations NHWC; conv weights [Cout][3][3][Cin]; FC weights
 *    [out][in] (shard j is the contiguous row block [c_j, c_{j+1}), c_j = floor(j*out/K)); the
 *    flatten order at the conv -> FC boundary is (h, w, c).
 *  - Precision modes: SB_FP32 keeps everything in float.  SB_BF16 stores activations,
 *    activation gradients and the weight copies used by the contractions in bfloat16
 *    (round-to-nearest-even), accumulates in float, and keeps master weights, momentum, weight
 *    gradients, logits and the loss in float.
 *
 * Paper references are to "SplitBrain: Hybrid Data and Model Parallel Deep Learning"
 * (arXiv 2112.15317) by section / paragraph / listing.
 */
#ifndef SPLITBRAIN_H
#define SPLITBRAIN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sb_model sb_model; /* opaque; host object owned by the library */

typedef enum {
    SB_OK = 0,
    SB_ERR_INVALID_ARG = 1,     /* null pointer, bad enum, misaligned pointer */
    SB_ERR_SHAPE = 2,           /* layer list / sizes that do not form a valid network */
    SB_ERR_UNSUPPORTED = 3,
    SB_ERR_ARENA_TOO_SMALL = 4,
    SB_ERR_CUDA = 5,            /* a CUDA runtime/driver call failed; see sb_last_error() */
    SB_ERR_STATE = 6,           /* call order (e.g. backward before forward) */
    SB_ERR_TIMEOUT = 7          /* a bounded device-side wait expired (status word set by a kernel) */
} sb_status;

typedef enum {
    SB_CONV3X3_RELU = 1, /* 3x3 cross-correlation, stride 1, zero pad 1, + bias, ReLU */
    SB_MAXPOOL2 = 2,     /* 2x2 max, stride 2 */
    SB_FC_RELU = 3,      /* fully connected + bias + ReLU, column-sharded K ways */
    SB_FC = 4,           /* fully connected + bias (the logits layer) */
    SB_SOFTMAX_XENT = 5, /* log-softmax + negative log-likelihood, mean over the batch */
    SB_FC_RELU_WHOLE = 6, /* SB_FC_RELU kept whole on every worker: the "do not partition" outcome of the paper's
                             computation-to-communication test for this layer [Layer Partitioning] */
    SB_FC_WHOLE = 7,      /* SB_FC (logits layer) kept whole */
    SB_DROPOUT = 8        /* dropout on the output of the SB_FC_RELU / SB_FC_RELU_WHOLE layer directly below it: a one-to-one
                             functional layer that follows the partitioned width, no modulo or shard node in between [Listing 1,
                             case DROPOUT | RELU].  `out` = drop probability p in units of 1/65536 (1..65535).  Element (batch row
                             g, column c) of the layer's [B, width] input is kept iff the first output word of the
                             Philox-4x32-10 counter-based generator at counter (e mod 2^32, e div 2^32, layer index, iteration),
                             e = g*width + c, key = the seed of sb_dropout_seed, is >= p * 2^32; kept elements are multiplied by
                             1/(1 - p) (float 65536 / (65536 - out)), dropped ones are zero.  The mask depends on the logical
                             element only, never on R or K.  The iteration counter lives on the device and goes up by one each
                             time a forward pass has run the network's last dropout layer (graph replays included); in
                             sb_modulo_step the K sub-iterations are one iteration and every example meets the mask of its
                             batch row. */
} sb_layer_kind;

typedef struct {
    int32_t kind; /* sb_layer_kind */
    int32_t out;  /* Cout / out-features / number of classes; ignored for SB_MAXPOOL2; SB_DROPOUT: p * 65536 */
} sb_layer;

enum { SB_FP32 = 0, SB_BF16 = 1 };

/* sb_config.flags */
enum {
    SB_FLAG_INPUT_GRAD = 1,  /* also compute the gradient w.r.t. the network input (layer 0 dgrad) */
    SB_FLAG_FORCE_SIMT = 2,  /* use the CUDA-core kernels for every layer (cross-check / debugging) */
    SB_FLAG_PROFILE_LAYERS = 4, /* sb_profile_end reports one entry per (kernel class, layer): "name#layer" */
    SB_FLAG_FORCE_PAIR = 8,  /* run every forward / data-gradient GEMM whose N tile is 128 or 256 wide, and every conv weight
                                gradient with 256+ output channels, on CTA pairs (tcgen05 cta_group::2), whatever the size;
                                by default the planner uses pairs only where they pay (256-wide tiles and at least one wave
                                of CTAs; weight gradients with long reductions) */
    SB_FLAG_MODULO_SCHEDULE = 16, /* reserve the buffers and plan the sub-batch kernels sb_modulo_step needs
                                (batch_per_replica must be a multiple of K; the first layer must not be an FC layer) */
    SB_FLAG_NO_HALO = 32,    /* 3x3 forward / data-gradient GEMMs on the kernel that fetches an activation box per filter tap
                                instead of the default one that shares a fetch of bh + 2 image rows between the three taps of
                                a filter column (for tests: both kernels must give the same results) */
    SB_FLAG_FORCE_PERSIST = 64 /* 3x3 forward / data-gradient GEMMs of layers up to 128 channels wide on the persistent kernel
                                (a few CTAs walk all output tiles, two accumulators in turn), whatever the layer's size; by
                                default only layers with several tiles per SM use it (for tests at small sizes) */
};

typedef struct {
    int32_t H, W, C;            /* input image geometry */
    int32_t batch_per_replica;  /* b: images per replica; the step's batch is B = R*b */
    int32_t R;                  /* data-parallel replicas of the conv stack (1..64) */
    int32_t K;                  /* model shards per FC layer (1..64, K <= every FC width) */
    int32_t precision;          /* SB_FP32 or SB_BF16 */
    int32_t flags;
} sb_config;

/* Tensor selectors for sb_tensor. */
enum {
    SB_T_WEIGHT = 0,   /* master weights, float.  conv: [Cout,3,3,Cin]; FC shard: [out_j,in] */
    SB_T_BIAS = 1,     /* float [Cout] / [out_j] */
    SB_T_GRAD_W = 2,   /* float, same shape as the weight */
    SB_T_GRAD_B = 3,
    SB_T_MOM_W = 4,    /* momentum, float */
    SB_T_MOM_B = 5,
    SB_T_ACT = 6,      /* layer output.  conv/pool: replica `part`'s [b,H,W,C]; FC: [B,out] (part
                          ignored); activation dtype, except the logits layer which is float */
    SB_T_DACT = 7,     /* gradient w.r.t. the layer's pre-activation output (conv, FC) or w.r.t. its
                          output (pool, dropout: zero wherever the dropout output is zero); same shape/partitioning as SB_T_ACT;
                          activation dtype */
    SB_T_POOL_IDX = 8, /* uint8 argmax position (dh*2+dw) per pooled element, replica `part` */
    SB_T_ROW_LOSS = 9, /* float [B]: per-row negative log-likelihood (layer = the loss layer) */
    SB_T_INPUT_GRAD = 10, /* gradient w.r.t. replica `part`'s input (needs SB_FLAG_INPUT_GRAD) */
    SB_T_SHADOW_W = 11 /* bf16 copy of the weight used by the contractions (SB_BF16 only) */
};
enum { SB_DT_F32 = 0, SB_DT_BF16 = 1, SB_DT_U8 = 2, SB_DT_I32 = 3 };

/*
 * Size of the device arena a model needs.  [Design: the model builder supplies a sequential
 * layer list, the batch size and the MP group size.]
 *   layers, cfg : host pointers.  arena_bytes : host pointer, receives the size.
 * Validation (SB_ERR_SHAPE): conv/pool layers first, then FC layers, then exactly one loss
 * whose class count equals the last FC width; H and W even at every pool; 1 <= R,K <= 64;
 * K <= every FC width.
 */
sb_status sb_model_bytes(const sb_layer* layers, int32_t n_layers, const sb_config* cfg,
                         size_t* arena_bytes);

/*
 * Build the partitioned network [Design, Layer Partitioning / Listing 1]: conv, pool and ReLU
 * layers are replicated over the R replicas (one parameter copy, since the replicas are kept
 * in sync every step); every FC layer is split into K column shards of 1/K size; the modulo
 * layer (gather of the replicas' features) and the shard layers (concatenation of the column
 * slices) exist only as the addressing of the FC kernels.
 *   arena : DEVICE pointer, 256-byte aligned, arena_bytes long, zero-filled by this call.
 *   out   : host pointer, receives the model handle.
 * All parameters start at zero: load them with sb_tensor_write (then sb_refresh_shadow).
 * Synchronises the device once (arena clear).
 */
sb_status sb_model_create(const sb_layer* layers, int32_t n_layers, const sb_config* cfg,
                          void* arena, size_t arena_bytes, sb_model** out);

sb_status sb_model_destroy(sb_model* m);

/*
 * Forward pass of one training iteration [Implementation: DP through the conv layers, MP
 * through the FC layers; Modulo Layer and Shard Layer, fprop].
 *   x      : HOST array of R DEVICE pointers; x[r] = replica r's images [b,H,W,C] in the
 *            activation dtype (float or bfloat16), 16-byte aligned.
 *   labels : HOST array of R DEVICE pointers; labels[r] = int32 [b], values in [0, classes).
 * Row g = r*b + i of every FC-side tensor belongs to replica r (the owner rule of the modulo layer:
 * a batch row's index divided by the rows per worker) [Modulo Layer].  Computes the per-row and mean loss and the gradient
 * of the loss w.r.t. the logits.  The input buffers must stay valid until sb_backward has run.
 */
sb_status sb_forward(sb_model* m, const void* const* x, const int32_t* const* labels, void* stream);

/*
 * Backward pass [Shard Layer and Modulo Layer, bprop; DP reduce]: FC weight/bias gradients per
 * shard; input gradients summed over the K shards and routed back to the owning replica's rows;
 * pooling and conv backward per replica; conv weight gradients summed over the R replicas.
 * Requires a preceding sb_forward (SB_ERR_STATE otherwise).
 */
sb_status sb_backward(sb_model* m, void* stream);

/*
 * SGD with momentum on every parameter [Implementation]:
 * v <- momentum*v + g ; w <- w - lr*v ; in SB_BF16 mode also refreshes the bf16 weight copies.
 */
sb_status sb_sgd_step(sb_model* m, float lr, float momentum, void* stream);

/*
 * One iteration in the modulo layer's own schedule [Modulo Layer]:
 * the conv-side layers run forward once on all R*b rows; the FC stack then runs K sub-iterations, sub-iteration k
 * on the k-th slice of b/K examples of every replica (inside a sub-batch the row at position p belongs to replica
 * p / (b/K)); every row's loss gradient is (softmax - onehot)/(R*b), which for the FC parameters is the mean over
 * the sub-batch divided by K, and the FC parameters take an SGD-momentum update after every sub-iteration, so K
 * per iteration; after the K-th the conv-side layers back-propagate once over all rows and take their update.
 * With K = 1 the result is that of sb_forward + sb_backward + sb_sgd_step; with K > 1 it is a different
 * algorithm (the FC weights move between sub-iterations).  sb_loss afterwards returns the mean of the R*b row
 * losses.  Needs SB_FLAG_MODULO_SCHEDULE at creation (SB_ERR_STATE otherwise).  Arguments as for sb_forward /
 * sb_sgd_step; runs on `stream`, asynchronous; like sb_graph_step the second call captures the iteration as a CUDA
 * graph and later calls with the same pointers and hyper-parameters replay it.  Afterwards SB_T_ROW_LOSS and the FC activation tensors hold their
 * rows in sub-iteration order (position k*(R*b/K) + r*(b/K) + i = example k*(b/K) + i of replica r), the FC
 * activations as left by the sub-iteration that wrote them; sb_backward needs a new sb_forward.
 */
sb_status sb_modulo_step(sb_model* m, const void* const* x, const int32_t* const* labels, float lr, float momentum,
                         void* stream);

/*
 * One whole iteration (sb_forward + sb_backward + sb_sgd_step on device-resident inputs) replayed as a CUDA
 * graph: the first call runs the three passes directly, the second captures them on `stream` (thread-local
 * capture mode) and every later call with the same input pointers, lr and momentum is one graph launch, which
 * removes the per-kernel launch cost that dominates at small batch sizes.  Different pointers or
 * hyper-parameters re-capture.  `stream` must not be the legacy default stream (NULL runs the passes directly).
 * Arguments as for sb_forward / sb_sgd_step.  Parameters, momentum, activations and loss are identical to the
 * three separate calls.  SB_T_GRAD_W / SB_T_GRAD_B are unspecified afterwards (here and after
 * sb_modulo_step / sb_train_step_host): where a weight gradient is summed from split partial copies, the ordered
 * sum feeds the update directly and is not stored, and the weight-gradient kernel of a large FC layer applies the
 * update to its tile itself; use sb_backward to read gradients.
 */
sb_status sb_graph_step(sb_model* m, const void* const* x, const int32_t* const* labels, float lr, float momentum,
                        void* stream);

/*
 * Mean loss of the last sb_forward.  Synchronises `stream`, copies 4 bytes to host_loss (HOST),
 * and checks the device status word: returns SB_ERR_TIMEOUT if any kernel gave up on a bounded
 * wait since the last call.
 */
sb_status sb_loss(sb_model* m, void* stream, float* host_loss);

/*
 * One whole iteration from HOST buffers (forward, backward, SGD step, loss read-back): the
 * end-to-end call.  host_x: [B,H,W,C] in the activation dtype, rows r*b..(r+1)*b-1 = replica r;
 * host_labels: int32 [B].  Both are copied host->device on `stream` into staging space inside
 * the arena (pinned host memory makes the copies asynchronous).  Synchronises `stream`.  From the second call on,
 * the copies, the iteration and the read-back of the loss are replayed as one CUDA graph keyed by the two host
 * pointers, lr and momentum (the host buffers must then stay at the same addresses; new addresses re-capture).
 */
sb_status sb_train_step_host(sb_model* m, const void* host_x, const int32_t* host_labels,
                             float lr, float momentum, void* stream, float* host_loss);

/*
 * Input prefetch for sb_train_step_host: starts the host->device copy of a LATER iteration's inputs into the second of
 * two staging areas inside the arena, on a copy stream of the library's own, and returns at once, so that the copy runs
 * while the current iteration computes.  Staged batches (two at most) are consumed in order: the next
 * sb_train_step_host / sb_train_step_host_async call must name the same host_x / host_labels, waits for the staged copy on the device instead of
 * copying, and is otherwise the same call (same result bits).  The host buffers must stay unchanged until that call
 * returns; pinned host memory makes the copy asynchronous.
 *   host_x, host_labels : HOST, as for sb_train_step_host.
 * Errors: SB_ERR_STATE with two batches already staged; sb_train_step_host returns SB_ERR_STATE when a batch is
 * staged and it is called with other host buffers.
 */
sb_status sb_prefetch_host(sb_model* m, const void* host_x, const int32_t* host_labels);

/*
 * sb_train_step_host without the wait: launches the iteration on `stream` and returns; sb_train_step_host_wait
 * blocks until the OLDEST launched iteration has finished and returns its loss (and SB_ERR_TIMEOUT if one of its kernels
 * gave up on a bounded wait).  Two iterations may be in flight, so that the host's launch and wake-up latency and the
 * read-back of one iteration hide behind the next one.  The iteration must have been staged by sb_prefetch_host (one
 * staging area and one pair of pinned result words per iteration in flight); without a staged batch, on the first
 * call of a model and in the diagnostic modes the call runs the iteration to completion itself and the wait returns
 * its result at once.  Iterations run in launch order on `stream`; results equal those of sb_train_step_host bit
 * for bit.
 * Errors: SB_ERR_STATE with two iterations in flight, with none to wait for, when a staged batch's host buffers are
 * not the ones named, and when sb_train_step_host is called while iterations are in flight.
 */
sb_status sb_train_step_host_async(sb_model* m, const void* host_x, const int32_t* host_labels, float lr, float momentum, void* stream);
sb_status sb_train_step_host_wait(sb_model* m, void* stream, float* host_loss);

/*
 * Introspection for parity tests and checkpointing: a borrowed DEVICE pointer to one tensor.
 *   what  : SB_T_*;  layer : index into the layer list;
 *   part  : replica r for conv-side activations, shard j for FC parameters.
 *   dev_ptr, shape (4 entries, unused = 1), dtype (SB_DT_*) : host pointers, any may be NULL.
 */
sb_status sb_tensor(sb_model* m, int32_t what, int32_t layer, int32_t part, void** dev_ptr,
                    int64_t shape[4], int32_t* dtype);

/* Blocking copies between a HOST buffer (dense, the tensor's dtype) and a tensor selected as in
 * sb_tensor.  `bytes` must equal the tensor's size. */
sb_status sb_tensor_read(sb_model* m, int32_t what, int32_t layer, int32_t part, void* host_dst, size_t bytes);
sb_status sb_tensor_write(sb_model* m, int32_t what, int32_t layer, int32_t part, const void* host_src, size_t bytes);

/* Rebuild the bf16 weight copies from the float master weights (after sb_tensor_write). */
sb_status sb_refresh_shadow(sb_model* m, void* stream);

/*
 * Dropout masks [Listing 1, case DROPOUT | RELU; see SB_DROPOUT]: sets the 64-bit key of the mask generator and the
 * iteration number (taken modulo 2^32) the next forward pass draws its masks for.  Enqueues one tiny kernel on `stream`
 * (asynchronous; a model is created with seed 0, iteration 0).  SB_ERR_INVALID_ARG for a null model.
 */
sb_status sb_dropout_seed(sb_model* m, uint64_t seed, uint64_t iteration, void* stream);

/*
 * Run a sub-range of layers only, on whatever the arena buffers currently hold ("teacher
 * forcing" for per-layer parity tests and micro-benchmarks).  sb_forward_layers runs layers
 * first..last in order; x/labels may be NULL unless layer 0 / the loss layer is in range.
 * sb_backward_layers runs the backward of layers last..first (last >= first) in reverse order.
 */
sb_status sb_forward_layers(sb_model* m, int32_t first, int32_t last, const void* const* x,
                            const int32_t* const* labels, void* stream);
sb_status sb_backward_layers(sb_model* m, int32_t last, int32_t first, void* stream);

/*
 * Layer partitioning as a table [Listing 1 "Layer Partitioning"; Layer Partitioning paragraph].  Walks the sequential
 * layer list and returns the transformed network: every input layer in order (SB_NODE_LAYER, with the number of
 * column shards it is split into: K for SB_FC_RELU / SB_FC when K > 1, else 1), a SB_NODE_MODULO node in front of the
 * first split layer (its input is whole: the MP group gathers the replicas' rows there), and a SB_NODE_SHARD node in
 * front of every layer, the loss included, whose input arrives as column slices.  dim / dimF are the widths, per
 * example, of the node's OUTPUT as one worker holds it and in full (dim = ceil(out / K) for a split layer).
 * Convolution / pooling layers are never split and refuse a partitioned input (SB_ERR_UNSUPPORTED).
 * Host-only: no CUDA call, usable without a GPU.  sb_model_create consumes the same table (per-layer shard counts).
 *   layers, cfg : HOST, as for sb_model_create (H, W, C, K are read).
 *   out         : HOST array of max_nodes entries, or NULL to query the count;  n_nodes : HOST, receives the count.
 * Errors: as sb_model_bytes for the layer list; SB_ERR_INVALID_ARG if max_nodes is too small.  Message: sb_partition_last_error().
 */
typedef enum { SB_NODE_LAYER = 0, SB_NODE_MODULO = 1, SB_NODE_SHARD = 2 } sb_node_kind;
typedef struct {
    int32_t node;   /* sb_node_kind */
    int32_t layer;  /* SB_NODE_LAYER: index into the input list; MODULO / SHARD: the layer it is inserted in front of */
    int32_t shards; /* SB_NODE_LAYER: 1 = whole on every worker, K = split by output column; inserted nodes: K */
    int32_t reserved;
    int64_t dim;    /* output width one worker holds */
    int64_t dimF;   /* full output width */
} sb_plan_node;
sb_status sb_partition(const sb_layer* layers, int32_t n, const sb_config* cfg, sb_plan_node* out, int32_t max_nodes, int32_t* n_nodes);
const char* sb_partition_last_error(void);

/*
 * Exchange schedule of N = R workers in R / K MP groups of K = mp workers each [Modulo Layer, Shard Layer, Group MP
 * Extension; Distributed Machine Learning: reduce].  Worker p is data replica p (rows [p*b, (p+1)*b) of the N*b-row
 * batch), belongs to group gid = p / K and holds model shard off = p % K of that group; R must be a multiple of K
 * (R = K: a single group; K = 1: pure data parallelism).  Lists every block that travels between two workers in one
 * synchronous iteration, forward pass first, then the backward pass in execution order; src and dst are worker ids,
 * rows are rows of the whole batch:
 *   SB_X_GATHER_ROWS : modulo layer, forward.  src sends its b feature rows [row0,row1) x all D columns to dst (same group).
 *   SB_X_GATHER_COLS : shard layer, forward.  src sends its column slice [col0,col1) of layer `layer`'s output for the
 *                      group's rows [row0,row1).
 *   SB_X_REDUCE_COLS : shard layer, backward.  src sends columns [col0,col1) (dst's slice) of its full-width partial
 *                      gradient w.r.t. layer `layer`'s output; dst adds the K partial results in worker order.
 *   SB_X_REDUCE_ROWS : modulo layer, backward.  src sends rows [row0,row1) (dst's examples) of its full-width partial
 *                      gradient w.r.t. the features; dst adds the K partial results in worker order.
 *   SB_X_ALLREDUCE   : the parameters of layer `layer` are held by every worker and trained on its own rows (conv stack):
 *                      their gradients are summed over all N workers (src = dst = -1).
 *   SB_X_ALLREDUCE_GROUPS : more than one group only.  Shard src (= offset inside a group; -1: a layer kept whole, every
 *                      offset) of FC layer `layer`, output columns [col0,col1), was trained by each group on that group's
 *                      rows: its gradients are summed over the workers gid*K + src of all groups, in group order.
 * On one GPU every one of these is addressing inside one device buffer (the arithmetic of N workers in groups of mp is
 * sb_config's R = N, K = mp); this table is the contract a multi-GPU runtime has to carry out (it has been executed
 * by CPU worker processes in the tests, not on several GPUs).
 * Host-only.  out may be NULL to query the count.
 */
typedef enum { SB_X_GATHER_ROWS = 1, SB_X_GATHER_COLS = 2, SB_X_REDUCE_COLS = 3, SB_X_REDUCE_ROWS = 4, SB_X_ALLREDUCE = 5,
               SB_X_ALLREDUCE_GROUPS = 6 } sb_exchange_kind;
typedef struct {
    int32_t kind;   /* sb_exchange_kind */
    int32_t layer;  /* layer whose output (or parameters) the block belongs to; for the modulo layer: the first split FC layer */
    int32_t pass;   /* 0 forward, 1 backward */
    int32_t src, dst;
    int32_t reserved;
    int64_t row0, row1, col0, col1; /* block of the [B, width] matrix */
    int64_t width;
} sb_exchange_msg;
sb_status sb_exchange_plan(const sb_layer* layers, int32_t n, const sb_config* cfg, sb_exchange_msg* out, int32_t max_msgs, int32_t* n_msgs);

/*
 * Parameter bytes (float master copies) one worker of an MP group of size K holds: all conv
 * parameters plus shard `shard` of every FC layer [Evaluation: parameter-memory saving].
 */
sb_status sb_param_bytes(const sb_model* m, int32_t shard, size_t* bytes);

/*
 * Per-kernel timing with CUDA events on the launching stream.  sb_profile_begin switches event
 * recording on: every kernel the library enqueues afterwards is bracketed by two events (this
 * serialises nothing but adds launch overhead, so whole-step timings should be taken with
 * profiling off).  sb_profile_end synchronises the stream, switches recording off and returns one
 * entry per kernel class with its launch count, total device time, and the ALGORITHMIC work of
 * those launches: flops = 2*M*N*K of the contractions; bytes = every operand read once and every
 * result written once (no im2col expansion, no padding, no re-reads).
 *   out : HOST array of max_entries entries;  n : HOST, receives the number written.
 */
typedef struct {
    char name[32];      /* kernel class, e.g. "conv_fwd_umma", "sgd", "pool_bwd" */
    int32_t launches;
    float ms_total;
    double flops;
    double bytes;
} sb_profile_entry;
sb_status sb_profile_begin(sb_model* m, void* stream);
sb_status sb_profile_end(sb_model* m, void* stream, sb_profile_entry* out, int32_t max_entries, int32_t* n);

/*
 * Self-test of the hang-safety path.  Every wait inside the library's kernels is bounded; a wait that runs out makes
 * the kernel record a code in the model's device status word and return normally, and the next sb_loss (or
 * sb_train_step_host) returns SB_ERR_TIMEOUT and clears the word.  This call enqueues one CTA that waits limit_ms
 * (1..1000) on a barrier that nothing completes and then reports in that way, so that a caller (or a test) can see
 * the whole path work without a stalled pipeline.  The GPU context stays usable.  No counterpart in the paper.
 */
sb_status sb_debug_wait_probe(sb_model* m, int32_t limit_ms, void* stream);

/*
 * Debug aids that stand in for a memory checker (no counterpart in the paper).
 * sb_debug_poison fills every buffer a training step rewrites -- activations, activation gradients, pooling argmax bytes,
 * split partial sums and the other scratch regions; not the parameters, momentum or gradients of parameters -- with 0xFF
 * bytes (NaN in float and bfloat16), on `stream`.  A kernel that reads an element nothing wrote in the same step then
 * produces NaN instead of silently re-using the previous step's value.  The next call must be sb_forward / a whole step.
 * sb_debug_check_guards synchronises `stream` and checks the guard bytes the library keeps behind every region of the
 * arena (256 bytes or more of a fixed pattern, written at creation): n_bad (HOST) receives the number of regions whose
 * guard was overwritten, first_bad_offset (HOST, may be NULL) the arena offset of the first damaged byte or -1.
 */
sb_status sb_debug_poison(sb_model* m, void* stream);
sb_status sb_debug_check_guards(sb_model* m, void* stream, int32_t* n_bad, int64_t* first_bad_offset);

/* Number of kernels the last sb_forward + sb_backward + sb_sgd_step enqueued (host counter). */
sb_status sb_launch_count(const sb_model* m, int64_t* launches);

const char* sb_last_error(void);

/*
 * (No counterpart in the paper: this entry point exists for callers that cannot allocate.)
 *
 * Weight and bias gradient of an input-layer 3x3 convolution (zero pad 1, stride 1), computed without
 * any device allocation: dw[k,r,s,c] = sum_{n,h,w} dy[n,h,w,k] * x[n,h+r-1,w+s-1,c], db[k] = sum dy[n,h,w,k].
 * It is the model path's input-layer weight-gradient kernel with its split partial sums kept in a
 * fixed 2 MiB array that is part of the library image instead of the caller's arena.
 *
 * Who needs it: code that wants this gradient but may not create device memory at that moment, for
 * example a monitoring or validation hook that runs beside a training job whose memory pool already
 * owns the whole GPU (a cudaMalloc there can fail, and it would also stall the running job because
 * device allocation synchronises the device), or a host program that forbids allocation after start-up.
 * Such a caller passes its existing input and output buffers and nothing else.
 *
 *   x  : DEVICE, [B,H,W,Cin], float (SB_FP32) or bfloat16 (SB_BF16), one contiguous buffer
 *   dy : DEVICE, [B,H,W,Cout], same dtype as x
 *   dw : DEVICE, float [Cout,3,3,Cin], overwritten        db : DEVICE, float [Cout], overwritten
 *   stream : cudaStream_t as void*; the call only enqueues two kernels.
 * Limits (SB_ERR_UNSUPPORTED otherwise): Cin in {1,3,4} and Cout*(9*Cin+1) <= 4096, e.g. Cout <= 146
 * for RGB inputs.  B, H, W are unlimited (at most 128 partial buffers are used whatever the size).
 * The first call on each device looks up the scratch array's device address (with that device
 * current); make that first call before any stream capture begins.  The library calls no cudaMalloc,
 * cudaFree or other allocating routine here.
 * The scratch array is shared by every call in the process and holds the previous call's partial
 * sums; the kernels rewrite every value they later read, so no clearing is needed, but two calls
 * that run concurrently on one GPU race on it: serialise them (same stream, or an event).
 * Every GPU that loads the library holds the 2 MiB until the process exits.
 * Errors are reported through the return code and sb_static_last_error().
 */
sb_status sb_conv_in_wgrad_static(const void* x, const void* dy, float* dw, float* db, int32_t B, int32_t H,
                                  int32_t W, int32_t Cin, int32_t Cout, int32_t precision, void* stream);
const char* sb_static_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SPLITBRAIN_H */
