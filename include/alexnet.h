/*
 * C ABI of the B200 AlexNet training-step library.
 *
 * The calls follow the paper's statement of the problem: model replicas that
 * start from the same parameters ("Data parallelism", first paragraph), a
 * loader that brings the next minibatch to the GPU and preprocesses it while
 * the current one trains ("Parallel Data Loading" and its figure), one update
 * per replica on its own minibatch, and the exchange and average of weights,
 * biases and momentum between replicas ("Data parallelism" and its figure):
 * with both replicas in one GPU's memory (alexnet_replica_average,
 * alexnet_update_and_average) or with one replica per GPU and process
 * (alexnet_param_regions + the caller's all-reduce + alexnet_scale_and_refresh,
 * or the gradient form alexnet_forward_backward + all-reduce +
 * alexnet_apply_update).
 *
 * Conventions
 *   - every function returns ALEXNET_OK (0) or a negative error code; nothing
 *     aborts or throws.  alexnet_last_error() gives a message for the last failure.
 *   - "host" pointers are ordinary CPU pointers (pinned where stated);
 *     "device" pointers are CUDA device pointers of the current device.
 *   - streams are cudaStream_t handles passed as void*.
 *   - the caller owns the device arena, the host buffers and the streams; the
 *     library owns only its handle, events and tensor maps.
 *   - canonical parameter vector (get/set): fp32, concatenated conv1.W
 *     [96][3][11][11], conv1.b, conv2.W [256][48][5][5], conv2.b, conv3.W
 *     [384][256][3][3], conv3.b, conv4.W [384][192][3][3], conv4.b, conv5.W
 *     [256][192][3][3], conv5.b, fc6.W [4096][9216] (input index c*36+h*6+w),
 *     fc6.b, fc7.W [4096][4096], fc7.b, fc8.W [1000][4096], fc8.b;
 *     60,965,224 floats.  Grouped filters are [Cout][Cin/groups][kh][kw]; output
 *     channel co belongs to group co / (Cout/groups).  Convolution is
 *     cross-correlation (no kernel flip).
 */
#ifndef ALEXNET_H
#define ALEXNET_H
#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct alexnet alexnet_t; /* opaque */

enum {
    ALEXNET_OK = 0,
    ALEXNET_ERR_ARG = -1,            /* NULL / out-of-range / inconsistent argument */
    ALEXNET_ERR_CUDA = -2,           /* a CUDA runtime or driver call failed */
    ALEXNET_ERR_STATE = -3,          /* call out of order (no batch loaded, both slots busy) */
    ALEXNET_ERR_DEVICE_TIMEOUT = -4, /* a bounded device-side wait expired (latched) */
    ALEXNET_ERR_NOMEM = -5           /* arena too small */
};

enum {                                /* alexnet_config_t.flags */
    ALEXNET_FLAG_LRN_ALPHA_DIV_N = 1, /* s = k + (alpha/n) * sum a^2 instead of alpha * sum a^2 */
    ALEXNET_FLAG_WD_ON_BIASES = 2,    /* weight decay also on biases */
    ALEXNET_FLAG_INVERTED_DROPOUT = 4, /* kept units scaled by 1/(1-p) */
    ALEXNET_FLAG_FUSED_FC_UPDATE = 8,  /* the FC weight-gradient kernel applies the momentum update to the FC weights in its
                                        * epilogue (same arithmetic, bit-identical parameters) and never stores those
                                        * gradients: get_params(which = 2) is then meaningless for fc6.W / fc7.W / fc8.W,
                                        * and alexnet_run_op of an FC weight-gradient operation updates the weights */
    ALEXNET_FLAG_NO_CTA_PAIRS = 16,    /* convolution forward / backward-data never run as clusters of two CTAs */
    ALEXNET_FLAG_ALL_CTA_PAIRS = 32,   /* ... always do (default: per layer, where the cost model expects a gain);
                                        * results do not depend on either flag beyond fp32 summation order */
    ALEXNET_FLAG_SHARED_REPLICA_WEIGHTS = 64,/* replicas == 2: both replicas use ONE copy of parameters, momentum and their bf16
                                        * forms.  Valid for the paper's scheme because the replicas are equal at the start of
                                        * every iteration (same initialisation; every exchange makes them equal again).  An
                                        * iteration is then alexnet_forward_backward on both replicas followed by
                                        * alexnet_update_and_average, which applies each replica's update to the shared state
                                        * and stores the average: the same arithmetic and bits as with two copies, 26 bytes of
                                        * parameter traffic per index instead of 44, and 14 bytes per parameter less memory.
                                        * alexnet_train_step and alexnet_apply_update return STATE (they would let one replica
                                        * run ahead of the other); alexnet_replica_average is a no-op; get/set_params address
                                        * the one copy through either replica index */
    ALEXNET_FLAG_FC_CHAIN = 128        /* the three FC forward passes run as ONE cooperative launch (fc_chain_kernel) whose weight
                                        * stream never stops at a layer boundary, where that is possible: batch <= 128 and a
                                        * device that can hold the whole grid at once; elsewhere the flag changes nothing.
                                        * Same units, arithmetic and summation order as the three launches: bit-identical
                                        * activations, masks and logits.  Off by default: measured, the step is no faster
                                        * (a layer boundary inside the launch costs what a launch boundary costs) */
};

typedef struct {
    int32_t batch;      /* images per replica per step, >= 1 */
    int32_t replicas;   /* 1 or 2 */
    uint64_t seed;      /* seeds crop/flip and dropout streams (and the optional init) */
    float lr, momentum, weight_decay;   /* Krizhevsky et al. 2012: 0.01, 0.9, 5e-4 */
    int32_t lrn_size;   /* must be 5 */
    float lrn_alpha, lrn_beta, lrn_k;   /* 1e-4, 0.75, 2 */
    float dropout_p;    /* 0.5; 0 disables */
    float init_std;     /* > 0: weights ~ N(0, init_std^2) from the seed, same in all replicas; 0: zeros */
    uint32_t flags;
} alexnet_config_t;

/* Number of parameters (60,965,224). */
size_t alexnet_param_count(void);

/* Bytes of device memory alexnet_create needs for this configuration
 * (parameters, momentum, gradients, bf16 copies, activations, batch slots,
 * split-K scratch).  Returns 0 for an invalid configuration. */
size_t alexnet_workspace_bytes(const alexnet_config_t* cfg);

/* Build `replicas` identically initialised models inside the caller's device
 * arena (paper: "Data parallelism", first sentences).
 *   dev_arena        device, >= alexnet_workspace_bytes(cfg), 1024-byte aligned; owned by the caller,
 *                    must outlive the handle
 *   host_mean_image  host fp32 [256][256][3] (HWC), or NULL for zeros; copied
 *   compute_stream   stream of train_step / replica_average
 *   copy_stream      side stream of load_batch_async (may equal compute_stream: no overlap then)
 * Errors: ARG (bad cfg / NULL), NOMEM (arena_bytes too small), CUDA. */
int alexnet_create(const alexnet_config_t* cfg, void* dev_arena, size_t arena_bytes,
                   const float* host_mean_image, void* compute_stream, void* copy_stream, alexnet_t** out);
int alexnet_destroy(alexnet_t* h);

/* Loader half of the paper's "Parallel Data Loading": on the copy stream,
 * copy one uint8 minibatch [B][256][256][3] (HWC) and its int32 labels [B]
 * (each in [0,1000)) to the device and run the preprocessing gather
 * (subtract mean image, random 227 crop, random flip; offsets and flip bits
 * from (seed, replica, step)).  Asynchronous; returns at once.  The source
 * buffers may be pinned host memory or device memory and must stay unchanged
 * until the copy has run (alexnet_sync, or the next load into the same slot).
 * Each replica has two batch slots filled in turn; a third load with none
 * consumed returns STATE. */
int alexnet_load_batch_async(alexnet_t* h, int replica, const uint8_t* images, const int32_t* labels, uint64_t step);

/* The intensity augmentation of Krizhevsky et al. 2012 (section 4.1), which the
 * paper's experiments leave out ("Experiments", the sentence on the reported
 * error rates): off by default; with sigma > 0 every later training load adds,
 * to all pixels of image n, the RGB offset eigvec * (alpha_n .* eigval) with
 * alpha_n ~ N(0, sigma^2) in R^3 drawn per image from (seed, replica, step).
 *   host_eigvec  host fp32 [3][3], row = colour, column i = i-th principal component of the RGB values of the training set
 *   host_eigval  host fp32 [3]
 *   sigma        0.1 in that paper; 0 switches the augmentation off (the arrays may then be NULL)
 * Evaluation batches are never augmented.  Takes effect for loads issued after the call.  Errors: ARG. */
int alexnet_set_color_augmentation(alexnet_t* h, const float* host_eigvec, const float* host_eigval, float sigma);

/* One SGD step of `replica` on its oldest loaded batch (paper, "Data
 * parallelism": every replica is updated on a minibatch of its own): forward,
 * softmax cross-entropy, backward, momentum update
 *   v <- momentum*v - lr*weight_decay*w - lr*g ; w <- w + v   (decay on weights only unless flagged).
 * Runs on the compute stream after the batch's load has finished; the
 * independent branches of the backward pass (weight gradients) run on
 * streams the handle owns, forked from and joined into the compute stream
 * inside the call, so work queued on the compute stream afterwards is
 * ordered after the whole step.  If host_loss is non-NULL the mean loss is written there and the call
 * synchronises the compute stream; otherwise it is asynchronous.
 * Errors: STATE (no loaded batch), DEVICE_TIMEOUT (latched), CUDA. */
int alexnet_train_step(alexnet_t* h, int replica, float* host_loss);

/* Queue, on the compute stream, a copy of the mean loss of the replica's most
 * recent train_step to *loss_out (pinned host memory or device memory, one
 * float) and return without waiting: the host can read step i's loss while
 * step i+1 runs.  The value is there once the compute stream has reached this
 * point (alexnet_sync, or an event the caller records on that stream after
 * the call); loss_out must stay valid until then.  Errors: ARG, CUDA. */
int alexnet_loss_async(alexnet_t* h, int replica, float* loss_out);

/* Evaluation of one minibatch, the measurement behind the paper's reported
 * validation errors ("Experiments": top-1 and top-5 error): forward pass only,
 * on the centre 227 x 227 crop without flip, with the dropout masks replaced by
 * their expectation (outputs of fc6 / fc7 times 1 - p, unless training uses
 * inverted dropout).  Copies images [B][256][256][3] uint8 and labels [B] int32
 * (pinned host or device memory) like load_batch_async, runs on both streams
 * and waits for the result.  A sample counts for top-k when fewer than k classes
 * rank before its label (greater logit, or equal logit and smaller index).
 *   host_top1, host_top5  number of samples of the batch in the top 1 / top 5 (may be NULL)
 *   host_loss             mean cross-entropy of the batch (may be NULL)
 * Parameters are not changed.  Errors: ARG, STATE (a loaded training batch is
 * still waiting for its train_step), DEVICE_TIMEOUT, CUDA. */
int alexnet_eval_batch(alexnet_t* h, int replica, const uint8_t* images, const int32_t* labels, int32_t* host_top1,
                       int32_t* host_top5, float* host_loss);

/* Steps 2 and 3 of the paper's data-parallel figure for two replicas held in
 * one GPU memory: w_a = w_b = (w_a+w_b)/2 and the same for momentum, over all
 * weights and biases.  No-op returning OK when replicas == 1. */
int alexnet_replica_average(alexnet_t* h);

/* The step in two halves, for callers that combine the gradients or the
 * parameters of several replicas before or after the update.
 *
 * alexnet_forward_backward is alexnet_train_step without the momentum update:
 * forward, loss, backward on the replica's oldest loaded batch; the gradient of
 * the mean loss stays in the replica's gradient array (get_params which = 2,
 * alexnet_param_regions) and is marked pending.  The FC weight gradients are
 * always stored here, whatever ALEXNET_FLAG_FUSED_FC_UPDATE says.
 *
 * alexnet_apply_update applies the update rule of alexnet_train_step to the
 * pending gradient multiplied by grad_scale (1 for a single replica; 1/R after
 * the caller has summed the gradients of R replicas into the array): by the
 * paper's remark that averaging the updated parameters and momenta of
 * identically starting replicas equals one update on the joint minibatch
 * ("Data parallelism", last paragraph), this is the gradient form of its
 * exchange.  Errors: STATE (no pending gradient), ARG, DEVICE_TIMEOUT, CUDA.
 *
 * alexnet_update_and_average is steps 1 to 3 of the paper's data-parallel
 * figure for two replicas in one GPU memory in ONE pass over the parameters:
 * both pending gradients are applied (each replica's own w, v, g; the same
 * arithmetic as alexnet_train_step) and w, v of both replicas are replaced by
 * the averages, 44 bytes of traffic per parameter index instead of 22 + 22 for
 * two updates and 36 for alexnet_replica_average.  The result is bit-identical
 * to alexnet_apply_update on both replicas followed by alexnet_replica_average.
 * Errors: STATE (replicas != 2 or a replica without pending gradient). */
int alexnet_forward_backward(alexnet_t* h, int replica, float* host_loss);
int alexnet_apply_update(alexnet_t* h, int replica, float grad_scale);
int alexnet_update_and_average(alexnet_t* h);

/* One replica per GPU and process: the exchange between GPUs is the caller's
 * (an all-reduce over NVLink by NCCL, or peer copies); the library exposes what
 * has to travel and finishes the average.
 *
 * alexnet_param_regions returns device pointers to the replica's parameters,
 * momentum and gradient: three arrays of *n_floats fp32 values each, in the
 * library's internal order (a fixed permutation of the canonical vector with
 * zero padding, identical in every process of the same build), owned by the
 * handle's arena and valid until alexnet_destroy.  Any of the four output
 * pointers may be NULL.  Work the caller queues on these arrays must be
 * ordered against the compute stream.
 *
 * alexnet_scale_and_refresh multiplies parameters and momentum by `scale`
 * (1/R after an all-reduce(sum) over R replicas: steps 2 and 3 of the paper's
 * data-parallel figure) and rebuilds the bf16 copies the tensor-core kernels
 * read (including the transposed convolution filters); with scale == 1 it only
 * rebuilds the copies, which is what a caller needs after writing averaged
 * parameters into the arrays itself.  Asynchronous, on the compute stream. */
int alexnet_param_regions(alexnet_t* h, int replica, float** dev_w, float** dev_v, float** dev_g, size_t* n_floats);

/* Overlapping the exchange of gradients with the backward pass.  In the arrays
 * of alexnet_param_regions the weights of the three FC layers (96% of all
 * parameters) are the contiguous range [*fc_weights_begin, *fc_weights_end)
 * (in floats; the convolution filters lie before it, all biases after it), and
 * their gradients are complete early in the backward pass, while the
 * convolution layers' backward pass is still to run.
 * alexnet_stream_wait_fc_gradients makes `stream` (a cudaStream_t of the
 * caller, e.g. the one it issues its all-reduce from) wait, on the device,
 * until the FC weight gradients of the backward pass issued last by
 * alexnet_forward_backward are written; work queued on `stream` afterwards
 * then runs beside the rest of that backward pass.  (When that pass kept
 * everything on the compute stream, i.e. with per-kernel timing on, the wait
 * is for the whole pass.)  The caller orders its stream back before
 * alexnet_apply_update.  Errors: ARG, DEVICE_TIMEOUT, CUDA. */
int alexnet_param_layout(const alexnet_t* h, size_t* fc_weights_begin, size_t* fc_weights_end, size_t* n_floats);
int alexnet_stream_wait_fc_gradients(alexnet_t* h, void* stream);

/* The paper's own form of the exchange (the data-parallel figure: step 2, each
 * GPU copies the other's weights, biases and momentum into receive buffers of
 * its own; step 3, it averages them with its own): the caller has brought the
 * other replicas' parameter and momentum arrays (alexnet_param_regions of the
 * peers: peer copies, or an all-gather) into buffers on THIS GPU; this call
 * replaces the replica's parameters and momentum by the mean over all `count`
 * replicas and rebuilds the bf16 copies.  One pass: (count - 1) x 8 + 8 bytes
 * read and 10 written per parameter index.
 *   dev_w, dev_v  host arrays of `count` device pointers, entry r = the arrays received from the replica of rank r
 *                 (n_floats fp32 each, 16-byte aligned, in this GPU's memory); entry `self` is ignored: the replica's
 *                 own arrays take its place, so that every rank adds the replicas in the same (rank) order and all
 *                 ranks end with bit-identical parameters
 *   count         number of replicas, 1..8;  self: this replica's rank, 0 <= self < count
 * Asynchronous, on the compute stream; the buffers must stay unchanged until it has run.  Errors: ARG, DEVICE_TIMEOUT, CUDA. */
int alexnet_average_received(alexnet_t* h, int replica, const float* const* dev_w, const float* const* dev_v, int count, int self);
int alexnet_scale_and_refresh(alexnet_t* h, int replica, float scale);

/* Read / write a replica's parameters in the canonical order above.
 *   which: 0 = parameters, 1 = momentum, 2 = gradient of the last step (read only)
 *   host buffer of n = alexnet_param_count() floats.  Synchronous. */
int alexnet_get_params(alexnet_t* h, int replica, int which, float* host_out, size_t n);
int alexnet_set_params(alexnet_t* h, int replica, int which, const float* host_in, size_t n);

/* Debug / parity access to intermediate tensors of the last step of a replica,
 * converted to fp32 in canonical NCHW (or [B][N]) order.  alexnet_tensor_size
 * gives the element count.  set_tensor writes a tensor (rounded to its device
 * type) so that one operation can be run in isolation by alexnet_run_op.  The
 * training step fuses LRN with pooling and does not store the normalised
 * tensors N1/N2 nor their gradients DN1/DN2; get_tensor recomputes them on
 * demand with the single-operation kernels (same arithmetic). */
enum {
    ALEXNET_T_CROPFLIP = 0, /* [B][3]: ox, oy, flip */
    ALEXNET_T_X0, ALEXNET_T_A1, ALEXNET_T_N1, ALEXNET_T_P1, ALEXNET_T_ARG1,
    ALEXNET_T_A2, ALEXNET_T_N2, ALEXNET_T_P2, ALEXNET_T_ARG2,
    ALEXNET_T_A3, ALEXNET_T_A4, ALEXNET_T_A5, ALEXNET_T_P5, ALEXNET_T_ARG5,
    ALEXNET_T_F6, ALEXNET_T_F7, ALEXNET_T_Z, ALEXNET_T_M6, ALEXNET_T_M7,
    ALEXNET_T_DZ, ALEXNET_T_DF7, ALEXNET_T_DF6, ALEXNET_T_DP5, ALEXNET_T_DA5, ALEXNET_T_DA4, ALEXNET_T_DA3,
    ALEXNET_T_DP2, ALEXNET_T_DN2, ALEXNET_T_DA2, ALEXNET_T_DP1, ALEXNET_T_DN1, ALEXNET_T_DA1,
    ALEXNET_T_LOSS, /* [B] per-sample loss */
    ALEXNET_T_DX0,  /* gradient with respect to the preprocessed image, [B][3][227][227]: written only by
                     * ALEXNET_OP_CONV1_BWD_DATA (the training step never needs it) */
    ALEXNET_T_COUNT
};
size_t alexnet_tensor_size(const alexnet_t* h, int tensor_id);
int alexnet_get_tensor(alexnet_t* h, int replica, int tensor_id, float* host_out, size_t n);
int alexnet_set_tensor(alexnet_t* h, int replica, int tensor_id, const float* host_in, size_t n);

/* Run one operation of the step `iters` times on the replica's current
 * tensors (compute stream, asynchronous), for per-layer parity and timing.
 * Operation ids: ALEXNET_OP_*.  Operations that read a batch slot (conv1,
 * softmax labels, preprocess) and get/set_tensor of X0 and CROPFLIP use the slot
 * touched by the most recent load_batch_async or train_step of that replica. */
enum {
    ALEXNET_OP_CONV1_FWD = 0, ALEXNET_OP_CONV2_FWD, ALEXNET_OP_CONV3_FWD, ALEXNET_OP_CONV4_FWD, ALEXNET_OP_CONV5_FWD,
    ALEXNET_OP_CONV2_BWD_DATA, ALEXNET_OP_CONV3_BWD_DATA, ALEXNET_OP_CONV4_BWD_DATA, ALEXNET_OP_CONV5_BWD_DATA,
    ALEXNET_OP_CONV1_BWD_WEIGHT, ALEXNET_OP_CONV2_BWD_WEIGHT, ALEXNET_OP_CONV3_BWD_WEIGHT,
    ALEXNET_OP_CONV4_BWD_WEIGHT, ALEXNET_OP_CONV5_BWD_WEIGHT,
    ALEXNET_OP_FC6_FWD, ALEXNET_OP_FC7_FWD, ALEXNET_OP_FC8_FWD,
    ALEXNET_OP_FC6_BWD_DATA, ALEXNET_OP_FC7_BWD_DATA, ALEXNET_OP_FC8_BWD_DATA,
    ALEXNET_OP_FC6_BWD_WEIGHT, ALEXNET_OP_FC7_BWD_WEIGHT, ALEXNET_OP_FC8_BWD_WEIGHT,
    ALEXNET_OP_LRN1_FWD, ALEXNET_OP_LRN2_FWD, ALEXNET_OP_LRN1_BWD, ALEXNET_OP_LRN2_BWD,
    ALEXNET_OP_POOL1_FWD, ALEXNET_OP_POOL2_FWD, ALEXNET_OP_POOL5_FWD,
    ALEXNET_OP_POOL1_BWD, ALEXNET_OP_POOL2_BWD, ALEXNET_OP_POOL5_BWD,
    ALEXNET_OP_SOFTMAX, ALEXNET_OP_UPDATE, ALEXNET_OP_AVERAGE, ALEXNET_OP_PREPROCESS,
    ALEXNET_OP_CONV1_BWD_DATA,   /* DA1 -> DX0; not part of the training step (per-layer sweep only) */
    /* the fused kernels the training step runs for the two LRN layers: A -> P, ARG (normalisation + pooling) and
     * A, DP, ARG -> DA (pooling gradient + normalisation gradient + ReLU mask) */
    ALEXNET_OP_LRN1_POOL1_FWD, ALEXNET_OP_LRN2_POOL2_FWD, ALEXNET_OP_POOL1_LRN1_BWD, ALEXNET_OP_POOL2_LRN2_BWD,
    ALEXNET_OP_UPDATE_AVERAGE,   /* the one-pass update + average of alexnet_update_and_average on whatever the gradient
                                  * arrays of the two replicas hold */
    ALEXNET_OP_SCALE_REFRESH,    /* alexnet_scale_and_refresh with scale 1 */
    ALEXNET_OP_FC_CHAIN_FWD,     /* P5 -> F6, M6, F7, M7 and fc8's split partials in one launch (what the step runs under
                                  * ALEXNET_FLAG_FC_CHAIN); ALEXNET_ERR_STATE where it is not available */
    ALEXNET_OP_COUNT
};
int alexnet_run_op(alexnet_t* h, int replica, int op, int iters);

/* Number of kernels launched by this handle since creation (for accounting). */
uint64_t alexnet_launch_count(const alexnet_t* h);

/* Optional timing of the tensor-core kernels: while enabled, every launch of
 * one is bracketed by a CUDA event pair on its stream (and the whole step stays
 * on the compute stream).  profile_read waits for both streams, returns per
 * kernel class the summed device time (ms) and the number of launches recorded
 * since the last read, and clears the record.  Index 0 = conv_kernel on
 * convolutions (forward and backward-data), 1 = wgrad_kernel (convolution
 * weight gradients), 2 = gemm_kernel (FC backward-data and weight gradients),
 * 3 = the FC forward passes (fc_chain_kernel: one launch for the three layers;
 * or conv_kernel's 1 x 1 case, one launch per layer; HBM-bound at batch 128).
 * Both arrays have four entries. */
int alexnet_profile(alexnet_t* h, int enable);
int alexnet_profile_read(alexnet_t* h, double* ms4, uint64_t* launches4);

/* Per-role timeline of the convolution kernel, for the timeline tool.  Only a
 * library built with -DALEXNET_TIMELINE records it (python -m
 * paper_1412_2302_b200.build --timeline builds that variant next to the normal
 * one); the normal build returns ALEXNET_ERR_STATE.  Waits for the device, then
 * copies the record of the most recent conv_kernel launch to host_out (may be
 * NULL): 160 CTA slots x 16 values (slot = blockIdx % 160):
 *   [0] start, [12] set-up done, [1] predecessor complete, [13] / [14] issuer enters / leaves its main loop,
 *   [15] last store of the first epilogue warp complete, [2] exit           (all in ns of the global timer)
 *   [3] [4] [5] cycles the first issuer waited for activations / weights / a free accumulator, [6] cycles of its main
 *   loop, [7] instructions it issued, [8] cycles the first epilogue warp waited for accumulators,
 *   [10] [11] cycles the producers waited for free activation / weight stages.
 * clear != 0 zeroes the record afterwards. */
int alexnet_timeline_read(long long* host_out, int clear);

/* Bias gradient db[c] = sum over rows of dy[row][c], for callers that cannot
 * allocate device memory when they need it.  (The paper has no counterpart of
 * this call; it is the bias-gradient reduction of the step offered on its own.)
 * Such callers are, for example, a loop in the middle of overlapped steps,
 * where cudaMalloc / cudaFree would synchronise the device and serialise the
 * loader stream with the compute stream, or a process that has handed all free
 * HBM to the arena of alexnet_create.  The scratch of the two-stage reduction
 * lives in a fixed 1 MiB array inside the library image, held by every GPU that
 * loads the library until the process exits; nothing is allocated or freed.
 *   dev_dy    device, bf16 [rows][channels], row-major, 16-byte aligned; read only
 *   rows      >= 1
 *   channels  multiple of 8, at most 4096 (the fixed scratch); larger values are
 *             rejected with ALEXNET_ERR_ARG and a message
 *   dev_db    device, fp32 [channels]; written
 *   stream    cudaStream_t the two kernels are launched on (asynchronous)
 *   err       optional host buffer for an error message (may be NULL)
 * The first call on a device looks up the scratch address for that device;
 * make that call before any stream capture begins there.  All calls share the
 * scratch, which keeps the last call's contents (nothing in it needs clearing:
 * each call overwrites what it later reads), so calls whose kernels could run
 * at the same time on one GPU race: order them on one stream or with events. */
int alexnet_bias_grad_noalloc(const void* dev_dy, int64_t rows, int32_t channels, float* dev_db, void* stream,
                              char* err, size_t err_len);

/* Host half of the paper's loading process ("Parallel Data Loading": a second
 * process loads the next minibatch while the current one trains): a worker
 * pool of `threads` threads (every batch is cut into `threads` chunks of
 * consecutive images, handed out in order) gathers
 * minibatches from a dataset in host memory (for instance a
 * memory-mapped file of uint8 [n][256][256][3] images and int32 labels) into a
 * ring of `depth` staging slots.  Sample j of the stream is dataset entry
 * perm_e[j mod n_epoch] with e = j / n_epoch and n_epoch = floor(n / batch) *
 * batch (an epoch drops the incomplete last batch); perm_e is the identity, or
 * with `shuffle` a Fisher-Yates shuffle (i from n_epoch-1 down to 1, swap with
 * hash(key_e, i) mod (i+1), key_e = mix(seed ^ 9<<56 ^ e), same counter hash as
 * crop / flip).  No CUDA calls are made: `ring` is caller memory of
 * alexnet_loader_ring_bytes(batch, depth) bytes, pinned if
 * alexnet_load_batch_async is to copy from it asynchronously.
 *   next     waits up to timeout_ms for the next batch in order and returns pointers to its images [batch][256][256][3]
 *            and labels [batch] inside the ring (STATE on time-out or when all `depth` slots are held)
 *   release  returns the oldest held slot to the worker; call it once the copy out of that slot has finished
 *            (for example after the train_step consuming it returned its loss, or after alexnet_sync)
 * Errors: ARG, NOMEM (ring too small), STATE. */
typedef struct alexnet_loader alexnet_loader_t;
size_t alexnet_loader_ring_bytes(int32_t batch, int32_t depth);
int alexnet_loader_create(const uint8_t* host_images, const int32_t* host_labels, uint64_t n_images, int32_t batch,
                          uint8_t* ring, size_t ring_bytes, int32_t depth, int32_t threads, uint64_t seed, int32_t shuffle,
                          alexnet_loader_t** out);
int alexnet_loader_next(alexnet_loader_t* l, int32_t timeout_ms, const uint8_t** images, const int32_t** labels, uint64_t* batch_index);
int alexnet_loader_release(alexnet_loader_t* l);
int alexnet_loader_destroy(alexnet_loader_t* l);

/* Message of the most recent alexnet_create that failed in the calling thread
 * (there is no handle to ask then); an empty string when none has failed. */
const char* alexnet_create_error(void);

/* Failure-detection self-test.  Every wait inside the tensor-core kernels is
 * bounded: when its cycle budget runs out the kernel sets the handle's device
 * status word, drains and returns, and the host reports DEVICE_TIMEOUT from
 * then on.  This call launches, on the compute stream, one warp that waits
 * through the same bounded-wait routine on a barrier that nothing ever arrives
 * on, with a budget of `budget_cycles` SM clock cycles (clamped to
 * [1e4, 2e8], i.e. at most about a tenth of a second), so the wait expires by
 * construction; the GPU context stays usable.  After the next synchronising
 * call (alexnet_sync, get_params, a train_step that returns its loss) the
 * handle is latched: every later call returns ALEXNET_ERR_DEVICE_TIMEOUT until
 * alexnet_destroy, which still succeeds. */
int alexnet_debug_expire_wait(alexnet_t* h, long long budget_cycles);

/* Wait for both streams; returns a latched DEVICE_TIMEOUT or CUDA error if any. */
int alexnet_sync(alexnet_t* h);
const char* alexnet_last_error(const alexnet_t* h);

#ifdef __cplusplus
}
#endif
#endif
