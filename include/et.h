/*
 * et.h -- C ABI of the elastic (masked) backward pass of a stack of dense layers.
 *
 * The operation is the one ElasticTrainer's tensor selection speeds up (arXiv
 * 2312.14227): given a binary selection mask over the trainable tensors, listed in
 * forward execution order (Section 5), the backward pass
 *   - passes the error gradient  dX_l = dZ_l * W_l^T  only through layers AFTER the
 *     deepest selected one (Section 2.2: an unselected layer still passes gradients,
 *     nothing at or below the deepest selected layer does),
 *   - forms the weight gradient  dW_l = X_l^T * dZ_l  and the bias gradient
 *     db_l = column sums of dZ_l  only for selected tensors (Section 5.1: the three
 *     backward operations of a dense layer),
 *   - reduces the first-order tensor importance  S_k = sum_i g_i * dw_i  (Eq. 2),
 *   - and updates the selected tensors only.
 *
 * Conventions
 *   Layers l = 0..L-1 in forward order, 0 nearest the input.  Tensor 2l is the kernel
 *   W_l [in_features x out_features], row-major (out_features contiguous); tensor
 *   2l+1 is the bias b_l [out_features].  Activations are [M x features], row-major.
 *       Z_l     = a_l * W_l + b_l
 *       H_l     = act_l(Z_l)
 *       a_{l+1} = sum of the `fold` equal column slices of H_l  (+ a_j if residual_src = j)
 *   a_0 is the stack input; the width of a_{l+1} is out_features / fold.
 *
 *   A layer of kind ET_LAYER_ATTENTION is the softmax attention core (the paper counts attention
 *   operations among the non-trainable layers, Sections 5.3 and 5.4): a_l = [q | k | v], per sequence
 *   and head  P = softmax(q k^T / 8),  a_{l+1} = [P v] with the heads side by side.  It has no
 *   trainable tensors: its W and b pointers may be NULL, its two mask bits must be 0 and its two
 *   slots in gradient / importance / state arrays are ignored.  Its backward (above the deepest
 *   selected layer only) recomputes P from the saved per-row log-sum-exp.
 *
 *   A layer of kind ET_LAYER_BATCHNORM is a batch normalisation in training mode, the layer Section 5.2
 *   is written about: like ET_LAYER_NORM with the mean and the biased variance of each feature taken
 *   over all M rows instead of over each row's features, no running averages, followed by act_l:
 *       a_{l+1} = act_l( (a_l - mean_c) / sqrt(var_c + eps) * gamma_l + beta_l )
 *   in_features == out_features (a multiple of 8), fold = 1, residual_src = -1; gamma and beta are
 *   tensors 2l and 2l+1 and are costed by the same black-box rule.
 *
 *   A layer of kind ET_LAYER_IM2COL gathers the k x k patches of a convolution (stride 1, zero
 *   padding k / 2) from NHWC rows:  a_{l+1}[(n,h,w), (kh*k + kw)*C + c] = a_l[(n, h+kh-k/2, w+kw-k/2), c].
 *   Followed by a dense layer with in_features = k*k*C it is the convolutional layer of Section 5.1
 *   (that layer's kernel is the convolution kernel in (kh, kw, c_in) x c_out layout).  Like the
 *   attention core it has no tensors: NULL pointers, mask bits 0.  On ET_BF16 stacks, when C is a
 *   multiple of 128, the layer is not the first one and the dense layer follows it directly (fold = 1,
 *   out_features a multiple of 64), the gathered matrix a_{l+1} is never formed: the dense layer's three
 *   GEMMs fetch the patches themselves, and the gather's forward and backward launch nothing.
 *
 *   A layer of kind ET_LAYER_NORM is a layer normalisation over the features of each row
 *   (Section 5.2 treats normalisation layers as two trainable tensors, Gamma and Beta;
 *   Section 5.4 says LayerNorm behaves like batch normalisation in this respect):
 *       xhat    = (a_l - mean) / sqrt(var + eps)        mean, biased var over the row
 *       a_{l+1} = xhat * gamma_l + beta_l
 *   Tensor 2l is gamma_l [features], tensor 2l+1 is beta_l [features]; they are passed
 *   where a dense layer passes W_l and b_l.  Its backward pass has the same three parts:
 *   the error gradient through the normalisation (only above the deepest selected layer),
 *   d gamma = column sums of g * xhat and d beta = column sums of g for selected tensors.
 *
 *   Storage type (et_dtype) applies to weights, biases, activations, error gradients
 *   and delta-W; accumulation is always fp32.  Exported gradients and importances are
 *   fp32.  ET_BF16 stacks run on tcgen05 tensor cores and need every feature count to
 *   be a multiple of 8, and out_features/fold a multiple of 256 when fold > 1.
 *
 * Memory and errors
 *   Every "device" pointer is caller-owned CUDA device memory, 16-byte aligned, valid
 *   until the work enqueued on `stream` has finished.  Arrays of pointers, masks and
 *   reports are host memory, read before the call returns.  The library allocates no
 *   device memory: one caller-provided workspace (et_stack_workspace_bytes) holds
 *   saved activations, error gradients, split-K partials and a status word.
 *   Arguments are validated on the host before anything is launched; a call that
 *   returns an error has enqueued nothing.  Calls are asynchronous on `stream`
 *   (a cudaStream_t passed as void*, NULL = default stream) unless stated otherwise.
 *   Calls on one stack must not overlap on the GPU (they share the workspace).
 */
#ifndef ET_H_
#define ET_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ET_OK = 0,
  ET_ERR_INVALID_ARG = 1,   /* null pointer, bad enum, bad length */
  ET_ERR_SHAPE = 2,         /* layer widths do not chain, residual width mismatch */
  ET_ERR_DTYPE = 3,
  ET_ERR_STATE = 4,         /* not bound, backward before forward */
  ET_ERR_WORKSPACE = 5,     /* workspace too small or misaligned */
  ET_ERR_UNSUPPORTED = 6,   /* shape outside what the kernels handle */
  ET_ERR_CUDA = 7,          /* a CUDA runtime call failed; see et_last_cuda_error */
  ET_ERR_TIMEOUT = 8,       /* a bounded device-side wait gave up */
  ET_ERR_TOO_LARGE = 9,     /* problem exceeds the fixed built-in scratch of a *_noalloc call */
  ET_ERR_GUARD = 10         /* et_debug_check_guards found a guard word overwritten */
} et_status;

typedef enum { ET_F32 = 0, ET_BF16 = 1 } et_dtype;
typedef enum { ET_ACT_NONE = 0, ET_ACT_GELU_TANH = 1, ET_ACT_RELU = 2 } et_act;
typedef enum {
  ET_LAYER_DENSE = 0, ET_LAYER_NORM = 1, ET_LAYER_ATTENTION = 2, ET_LAYER_IM2COL = 3, ET_LAYER_BATCHNORM = 4
} et_layer_kind;

/* Cost-model reading for the selector (Section 2.2 / Eq. 7 versus the example after Eq. 3). */
typedef enum {
  ET_COST_STRICT = 0,      /* tensors after the deepest selected one pay t_dy */
  ET_COST_INCLUSIVE = 1    /* the deepest selected tensor pays its own t_dy too */
} et_cost_variant;

enum {
  ET_FLAG_FUSE_SGD = 1u,   /* et_backward_elastic also updates the selected tensors (w <- w - lr*g, or the
                              optimiser set with et_stack_set_optimizer) */
  ET_FLAG_DELTA_IS_SNAPSHOT = 2u  /* delta[k] is a copy of tensor k taken earlier; the update of Eq. 2 is
                                     dw = (current tensor) - delta[k], formed on the fly (Section 3.1: the
                                     weight update accumulated since the start of the evaluation period) */
};

typedef struct {
  int32_t in_features;
  int32_t out_features;
  int32_t act;            /* et_act; must be ET_ACT_NONE when fold > 1 */
  int32_t fold;           /* >= 1, divides out_features */
  int32_t residual_src;   /* -1, or j in [0, l]: add a_j to this layer's output */
  int32_t kind;           /* et_layer_kind.  ET_LAYER_NORM: in_features == out_features (a multiple of 8,
                             at most 2048), act = ET_ACT_NONE, fold = 1, residual_src = -1 */
  float eps;              /* ET_LAYER_NORM: added to the variance, > 0 or 0 */
  int32_t heads;          /* ET_LAYER_ATTENTION: in_features = 3 * out_features, out_features = 64 * heads;   */
  int32_t seq_len;        /*   rows form sequences of seq_len (<= 256) consecutive rows, M a multiple of it;  */
                          /*   ET_BF16 only; not the first or last layer; the layer below has no activation;   */
                          /*   act = ET_ACT_NONE, fold = 1, residual_src = -1.  Both fields 0 for other kinds. */
  int32_t height;         /* ET_LAYER_IM2COL: rows are images of height x width pixels, NHWC (M a multiple of  */
  int32_t width;          /*   height * width); in_features = channels (a multiple of 8), out_features =        */
  int32_t ksize;          /*   ksize^2 * channels, ksize odd and <= 7; act, fold, residual_src as for attention. */
} et_layer_desc;

/* What one et_backward_elastic call executed.  The four arrays are caller-owned host
 * memory (any may be NULL): dgrad/wgrad/bgrad have L entries, updated has 2L. */
typedef struct {
  uint8_t* dgrad;
  uint8_t* wgrad;
  uint8_t* bgrad;
  uint8_t* updated;
  int32_t deepest;          /* smallest layer index owning a selected tensor; L if none */
  int32_t launches;         /* kernels enqueued by the call */
  double flops_executed;    /* 2*M*K*N per executed dgrad / wgrad GEMM */
} et_exec_report;

typedef struct et_stack et_stack;

/* ---- stack object (host) ---------------------------------------------------------- */

/* Validates the layer chain and builds the host-side plan.  M = rows (tokens). */
et_status et_stack_create(const et_layer_desc* layers, int32_t L, int64_t M, et_dtype dtype,
                          et_stack** out);
et_status et_stack_destroy(et_stack* s);

/* Execution options of a stack (host state; take effect from the next call on).  They change how the
 * work is launched, never what is computed.
 *   ET_OPTION_TWO_STREAMS    1 (default): et_backward_elastic runs the error-gradient chain on an internal
 *                            high-priority stream beside the weight gradients; 0: everything on the caller's stream.
 *   ET_OPTION_LAUNCH_OVERLAP 1 (default): consecutive GEMMs of one stream start their prologue under the
 *                            previous kernel's tail (programmatic dependent launch); 0: plain launches.
 *   ET_OPTION_TILE_PLAN      ET_TILE_PLAN_AUTO (default): GEMM tile shapes made for a GPU shared by the two
 *                            streams when they run, for a GPU to itself otherwise; ET_TILE_PLAN_ALONE /
 *                            ET_TILE_PLAN_SHARED force one (per-kernel timing keeps kernels on one stream and
 *                            can still time the shapes the two-stream step launches).
 *   ET_OPTION_GEMM_LIST      1 (default): where every layer is a dense layer with widths that are multiples of 64 (bf16
 *                            stacks; no layer with both an activation and a residual), et_forward_stack runs all layers
 *                            as ONE cooperative launch whose work units wait on one another row tile by row tile; and
 *                            where every layer from the deepest selected one upwards is a dense layer
 *                            with widths that are multiples of 64 (bf16 stacks), et_backward_elastic runs all
 *                            error-gradient and weight-gradient GEMMs of the call as ONE cooperative launch whose
 *                            work units wait on one another row tile by row tile, followed by one grouped launch
 *                            for the split reductions (gradient export, Eq. 2, update) and one for the bias
 *                            gradients; 0: one launch per GEMM (the path other stacks always take).
 *   ET_OPTION_LIST_COOPERATIVE 1 (default): that launch is a cooperative one, which is what guarantees that all its
 *                            CTAs are resident while they wait on one another.  0: a plain launch of the same grid,
 *                            for a profiler that does not take cooperative launches; only safe while nothing else
 *                            runs on the GPU (every CTA then becomes resident at once because the grid is sized to
 *                            the device). */
typedef enum { ET_OPTION_TWO_STREAMS = 1, ET_OPTION_LAUNCH_OVERLAP = 2, ET_OPTION_TILE_PLAN = 3,
               ET_OPTION_GEMM_LIST = 4, ET_OPTION_LIST_COOPERATIVE = 5 } et_option;
typedef enum { ET_TILE_PLAN_AUTO = 0, ET_TILE_PLAN_ALONE = 1, ET_TILE_PLAN_SHARED = 2 } et_tile_plan;
et_status et_stack_set_option(et_stack* s, int32_t option, int32_t value);

/* Bytes of device workspace et_stack_bind needs (a multiple of 256). */
et_status et_stack_workspace_bytes(const et_stack* s, size_t* bytes);

/* Attaches parameters and workspace.  W, b: host arrays of L device pointers (storage
 * dtype).  The workspace must be 256-byte aligned.  The library zeroes what it needs on
 * `stream`.  May be called again to re-attach. */
et_status et_stack_bind(et_stack* s, void* const* W, void* const* b, void* workspace,
                        size_t workspace_bytes, void* stream);

/* Optional fp32 master copies for ET_BF16 stacks (the paper trains in fp32, Section 7; bf16
 * storage alone rounds an update lr*g away when it is below half an ulp of the weight).
 * W32, b32: host arrays of L device float* holding the same values as W, b (caller-owned,
 * caller-initialised), or both NULL to detach.  While attached, every masked update
 * (ET_FLAG_FUSE_SGD, et_sgd_masked) is applied to the master in fp32 and the bf16 tensor is
 * rewritten as its rounding; ET_FLAG_DELTA_IS_SNAPSHOT then expects fp32 snapshots of the
 * masters in `delta`.  Unselected tensors and their masters are never written.  Call after
 * et_stack_bind (which detaches). */
et_status et_stack_bind_master(et_stack* s, float* const* W32, float* const* b32);

/* The optimisers the paper trains with (Section 8): SGDW -- momentum 0.9, decoupled weight decay
 * 5e-4, cosine-scheduled learning rate -- for the convolutional models, Adam for ViT.  Masked like
 * everything else: only selected tensors and their state are read or written.
 *   ET_OPT_SGD :  w <- w - lr g
 *   ET_OPT_SGDW:  m <- momentum m + lr g ;  w <- w - m - wd w
 *   ET_OPT_ADAM:  m <- b1 m + (1-b1) g ;  v <- b2 v + (1-b2) g^2 ;
 *                 w <- w - lr (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps)
 * Schedules stay with the caller: `lr` is the argument of the updating call, the step number t
 * and this step's weight decay wd are set with et_stack_set_optimizer_step. */
typedef enum { ET_OPT_SGD = 0, ET_OPT_SGDW = 1, ET_OPT_ADAM = 2 } et_optimizer;
typedef struct {
  int32_t kind;         /* et_optimizer */
  float momentum;       /* SGDW */
  float weight_decay;   /* SGDW: initial wd (et_stack_set_optimizer_step overrides it per step) */
  float beta1, beta2;   /* Adam */
  float eps;            /* Adam */
} et_optimizer_config;

/* Selects the optimiser used by ET_FLAG_FUSE_SGD and et_update_masked.  state1 / state2: host
 * arrays of 2L device float* in tensor order, shaped like the tensors, caller-owned and
 * zero-initialised (state1 = momentum / first moment, needed for SGDW and Adam; state2 = second
 * moment, Adam only).  cfg == NULL or kind ET_OPT_SGD restores plain SGD.  Resets t to 1.
 * Call after et_stack_bind (which restores plain SGD). */
et_status et_stack_set_optimizer(et_stack* s, const et_optimizer_config* cfg, float* const* state1,
                                 float* const* state2);
/* Step number t >= 1 (Adam's bias correction) and weight decay of the next updating call. */
et_status et_stack_set_optimizer_step(et_stack* s, int32_t step, float weight_decay);

/* ---- forward and loss (precede the hot path; Eq. 3's T_forward) -------------------- */

/* x: device [M x in_features(0)], y: device [M x width(a_L)], storage dtype.  Saves every
 * a_l and the pre-activations of activated layers in the workspace.  x itself is
 * referenced, not copied: it must stay valid and unchanged until the backward call that
 * uses this forward pass has finished. */
et_status et_forward_stack(et_stack* s, const void* x, void* y, void* stream);

/* Mean-squared error over all M*D elements and its gradient dY = 2 (y - target) / (M*D).
 * y, target, dY: device, storage dtype; loss_dev: device float (may be NULL). */
et_status et_loss_mse_grad(et_stack* s, const void* y, const void* target, void* dY,
                           float* loss_dev, void* stream);

/* ---- the hot path ----------------------------------------------------------------- */

/* Elastic backward (Section 2.2, Section 5.1, Eq. 2).
 *   dY         device [M x width(a_L)], storage dtype: dL/da_L.
 *   mask       host uint8[n_tensors], n_tensors must equal 2L; non-zero = selected.
 *   grads      host array of 2L device float* (or NULL array): where selected gradients
 *              are written, dW_l as [in x out] row-major, db_l as [out].  An entry may be
 *              NULL when the gradient itself is not wanted.  Entries of unselected
 *              tensors are ignored and their buffers never touched.
 *   delta      host array of 2L device pointers, storage dtype, same shapes as the
 *              tensors (or NULL array): the recent update dw of Eq. 2 (or, with
 *              ET_FLAG_DELTA_IS_SNAPSHOT, the earlier weights it is measured from).  If given,
 *              importance_dev must be given too, and every selected tensor needs an entry.
 *   importance_dev  device float[2L]: S_k for selected tensors, 0 for the others.
 *   flags, lr  ET_FLAG_FUSE_SGD applies w <- w - lr*g (Section 2.2's weight update) to
 *              selected tensors inside the same call, after every read of the old weight.
 *              Unselected tensors are never written.
 *   report     host, optional.
 * Nothing is launched for layers below the deepest selected one; with an empty mask
 * nothing is launched at all except zeroing importance_dev.  Needs a preceding
 * et_forward_stack on the same stack.
 * How it is launched (see et_stack_set_option): stacks whose layers from the deepest selected one upwards
 * are all dense (bf16, widths multiples of 64) run every GEMM of the call as one cooperative launch,
 * followed by one grouped reducer and one grouped bias finisher, all on `stream`.  Other stacks launch
 * layer by layer: the error-gradient chain on an internal high-priority stream that forks from and joins
 * back into `stream` inside the call (weight gradients fill the SMs the chain leaves idle).  Either way,
 * to the caller everything is ordered on `stream`. */
et_status et_backward_elastic(et_stack* s, const void* dY, const uint8_t* mask, int32_t n_tensors,
                              float* const* grads, const void* const* delta,
                              float* importance_dev, uint32_t flags, float lr,
                              et_exec_report* report, void* stream);

/* Same call for host-resident buffers: copies dY (host, storage dtype) to the device,
 * runs et_backward_elastic, copies the 2L importances back to importance_host (if delta
 * is given) and synchronises `stream` before returning.  dY_host / importance_host should
 * be pinned for full copy bandwidth.  grads / delta stay device pointers as above. */
et_status et_backward_elastic_host(et_stack* s, const void* dY_host, const uint8_t* mask,
                                   int32_t n_tensors, float* const* grads,
                                   const void* const* delta, float* importance_host,
                                   uint32_t flags, float lr, et_exec_report* report, void* stream);

/* Stand-alone Eq. 2 on already materialised gradients: importance_dev[k] =
 * sum(grads[k] * delta[k]) for selected k, 0 otherwise. */
et_status et_importance(et_stack* s, const uint8_t* mask, int32_t n_tensors, float* const* grads,
                        const void* const* delta, float* importance_dev, void* stream);

/* The two importance metrics the paper compares Eq. 2 against in its ablation (Section 8, "Efficacy of
 * Tensor Importance Evaluator"): weight magnitudes and gradient feedback.  The paper gives no formula
 * for either; here they are the L1 norms  sum_i |w_i|  (of the tensors as bound, the fp32 masters
 * when attached) and  sum_i |g_i|  (of materialised fp32 gradients, as et_backward_elastic exports
 * them).  metric_dev receives n_tensors floats, 0 for unselected tensors.  Uses the importance
 * scratch of the workspace: do not overlap with a backward call.  Asynchronous on `stream`. */
typedef enum { ET_METRIC_WEIGHT_MAGNITUDE = 1, ET_METRIC_GRADIENT_MAGNITUDE = 2 } et_metric_kind;
et_status et_tensor_metric(et_stack* s, const uint8_t* mask, int32_t n_tensors, int32_t kind,
                           float* const* grads, float* metric_dev, void* stream);

/* Stand-alone masked SGD: w_k <- w_k - lr * grads[k] for selected k (fp32 arithmetic,
 * rounded once to the storage dtype), whatever optimiser is configured.  Unselected tensors
 * are never written. */
et_status et_sgd_masked(et_stack* s, const uint8_t* mask, int32_t n_tensors, float* const* grads,
                        float lr, void* stream);
/* Stand-alone masked update with the configured optimiser (et_stack_set_optimizer). */
et_status et_update_masked(et_stack* s, const uint8_t* mask, int32_t n_tensors, float* const* grads,
                           float lr, void* stream);

/* Bias gradient without any allocation.  (The paper has no counterpart for this call; it
 * exists for how this library gets embedded.)
 *
 * Who needs it: code that must not, or cannot, call cudaMalloc or hand the library a
 * workspace at the point where it needs a bias gradient -- for instance a plug-in running
 * inside a host application that owns all device memory and gives none out, a callback on a
 * latency-critical path where an allocation (which may synchronise the device) is forbidden,
 * or a process whose memory budget is fixed at start-up.  Such a caller still passes its own
 * input and output buffers; only the intermediate storage comes from the library.
 *
 * Computes db[j] = sum over the M rows of dZ[:, j] (Section 5.1's bias update, the same
 * two-stage fixed-order column reduction et_backward_elastic uses for selected biases).
 *   dZ     device [M x width], row-major, storage dtype `dtype`, 16-byte aligned
 *   db     device float[width]
 * The stage-1 partial sums live in a fixed array compiled into the library:
 * ET_NOALLOC_SCRATCH_FLOATS floats (4 MiB) on every GPU that loads the library, kept until
 * the process ends.  A problem needs ceil(M / 128) * width floats of it; a larger one (or one
 * of more than 65535 * 128 rows) is refused with ET_ERR_TOO_LARGE and nothing is launched.
 * The call itself performs no cudaMalloc / cudaFree and calls no allocating routine.
 * Every call looks up the device address of that array for the current device (nothing is
 * remembered between calls, so the call stays valid after the application resets the device
 * or switches the current context).  The first call on a device may load the library's
 * device code: make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps whatever the last call left in
 * it.  No clearing is needed (each call overwrites every entry it later reads), but two
 * calls that run concurrently on the same GPU -- different streams, or different host
 * threads -- race on it: serialise them.  Asynchronous on `stream`. */
#define ET_NOALLOC_SCRATCH_FLOATS (1 << 20)
et_status et_bias_grad_noalloc(const void* dZ, int64_t M, int32_t width, et_dtype dtype, float* db,
                               void* stream);

/* ---- selection support (host) ------------------------------------------------------ */

/* Times each layer's dgrad and wgrad(+bias) launches with CUDA events (median of `iters`)
 * and fills per-TENSOR cost vectors of length 2L following Section 5.1: kernel tensor:
 * t_dw = weight-gradient time, t_dy = error-gradient time (with the fused backward of the
 * non-trainable work below it, Section 5.3); bias tensor: t_dw = bias-gradient time,
 * t_dy = 0.  A normalisation layer is one black box (Section 5.2): the time of its whole
 * backward kernel (error gradient and d gamma together) plus its two finishing kernels goes
 * to t_dy of beta; t_dw of gamma and beta and t_dy of gamma are 0.  An attention layer is a
 * non-trainable layer (Section 5.3): its backward time is added to t_dy of the bias of the layer below.
 * t_fwd receives the forward time.  Milliseconds.  Synchronous.  Runs a forward
 * pass from x (writing y) and a full backward from dY first; weights are not changed. */
et_status et_profile_costs(et_stack* s, const void* x, void* y, const void* dY, int32_t iters,
                           double* t_dw, double* t_dy, double* t_fwd, void* stream);

/* Backward time of a selection under the model of Section 2.2 / Eq. 3 (host arithmetic). */
et_status et_time_selective(const uint8_t* mask, const double* t_dw, const double* t_dy,
                            int32_t n, int32_t variant, double* t_out);

/* Tensor selector (Section 6): maximise sum of importance[k] over selected k subject to
 * t_fwd + selected t_dw + charged t_dy <= rho * (t_fwd + sum t_dw + sum t_dy), by dynamic
 * programming over (depth from the output, quantised time), times quantised with
 * Eq. 8 at resolution Tq.  Host only, synchronous.  mask_out: uint8[n]; value_out: the
 * optimum of the quantised problem; est_time_out: unquantised backward time of the mask. */
et_status et_select_dp(const double* importance, const double* t_dw, const double* t_dy, int32_t n,
                       double t_fwd, double rho, int32_t Tq, int32_t variant,
                       uint8_t* mask_out, double* value_out, double* est_time_out);

/* What a run of the selector's dynamic program did (Section 6.3 counts subproblems). */
typedef struct {
  int64_t table_full;     /* n * (T + 1): subproblems of the unpruned table, t up to the full (quantised) backward time T */
  int64_t table_budget;   /* n * (budget + 1): without the invalid ones, whose t exceeds the time constraint */
  int64_t visited;        /* (k, t) entries evaluated: also without the redundant ones, whose t cannot even pay
                             the error-gradient path down to tensor k */
  int64_t transitions;    /* (k, k_c, t) candidates compared (the O(N^2 T) work of Section 6.2) */
  int32_t rows_reached;   /* tensors, from the output, that the budget reaches at all */
  int32_t threads;        /* threads that took part */
} et_dp_stats;

/* et_select_dp with the choices of Sections 6.3 exposed: `prune` = 1 skips invalid and redundant
 * subproblems (the default of et_select_dp), 0 evaluates the whole table, which must give a selection of
 * the same value; `threads` >= 1 host threads share each row of the table (for N in the thousands,
 * Section 6.3's last paragraph); `stats` may be NULL.  Host only, synchronous. */
et_status et_select_dp_ex(const double* importance, const double* t_dw, const double* t_dy, int32_t n,
                          double t_fwd, double rho, int32_t Tq, int32_t variant, int32_t threads,
                          int32_t prune, uint8_t* mask_out, double* value_out, double* est_time_out,
                          et_dp_stats* stats);
et_status et_select_dp_int_ex(const double* importance, const int64_t* t_dw, const int64_t* t_dy,
                              int32_t n, int64_t budget, int32_t variant, int32_t threads, int32_t prune,
                              uint8_t* mask_out, double* value_out, et_dp_stats* stats);

/* Same problem with integer costs given directly (no quantisation step). */
et_status et_select_dp_int(const double* importance, const int64_t* t_dw, const int64_t* t_dy,
                           int32_t n, int64_t budget, int32_t variant,
                           uint8_t* mask_out, double* value_out);

/* ---- debugging aid: guard words round the workspace regions ------------------------- */

/* on != 0: every stack created from now on (in this process) lays its workspace out with 256 guard
 * bytes after each region (saved activations, error gradients, split partials, bias partials, ...);
 * et_stack_bind fills them with a pattern.  A kernel that writes past the end of its region hits
 * them first.  Stands in for a memory checker on stacks whose kernels index by hand.  Costs 256 bytes
 * per region and nothing at run time. */
et_status et_debug_guard_regions(int32_t on);
/* Copies the guard words back and compares them (synchronises `stream`).  ET_OK, or ET_ERR_GUARD with
 * the index of the first damaged region (in layout order) in *first_bad_region (may be NULL).
 * A stack created without guards always returns ET_OK. */
et_status et_debug_check_guards(et_stack* s, void* stream, int32_t* first_bad_region);

/* ---- per-kernel timing (measurement support) ---------------------------------------- */

/* Kernel classes for et_timing_read. */
typedef enum {
  ET_K_FORWARD = 0,        /* forward GEMM (+bias, activation, fold, residual)          */
  ET_K_DGRAD = 1,          /* error-gradient GEMM with its fused epilogue (Section 5.1 T1, 5.3) */
  ET_K_WGRAD = 2,          /* weight-gradient GEMM writing split partials (T3)          */
  ET_K_WGRAD_REDUCE = 3,   /* split reduction + gradient export + importance + SGD      */
  ET_K_BGRAD = 4,          /* bias gradient: column sums + finish (T2)                  */
  ET_K_OTHER = 5,          /* loss gradient, top-layer activation backward, importance finalise */
  ET_K_NORM = 6,           /* normalisation layers: forward, backward (error gradient + d gamma), gamma finish */
  ET_K_ATTENTION = 7,      /* layers without tensors: attention core, patch gather; forward, backward */
  ET_K_LIST = 8,           /* the one-launch backward: every dgrad and wgrad GEMM of a call in one kernel */
  ET_K_CLASSES = 9
} et_kernel_class;

/* on != 0: every kernel this stack launches from now on is bracketed by a pair of CUDA
 * events on its stream (host objects; no device memory), and the backward pass keeps all its
 * kernels on the caller's stream, one after the other, so that a pair brackets exactly one
 * kernel's run.  on == 0: stop and drop them. */
et_status et_timing_enable(et_stack* s, int32_t on);
/* Waits for the recorded events, adds up device time (milliseconds) and launch counts per
 * class into ms[ET_K_CLASSES] / launches[ET_K_CLASSES] (either may be NULL), and clears the
 * record. */
et_status et_timing_read(et_stack* s, double* ms, int64_t* launches);

/* ---- status ------------------------------------------------------------------------ */

/* Synchronises `stream` and reports ET_ERR_TIMEOUT if a kernel's bounded wait gave up,
 * ET_ERR_CUDA if the stream is in error, else ET_OK.  (The kernels record the first such event
 * as a non-zero code in the first 32-bit word of the workspace; it stays set until the
 * workspace is re-bound.) */
et_status et_device_status(et_stack* s, void* stream);
const char* et_status_string(et_status st);
/* cudaError_t of the last failing CUDA call seen by this thread (0 if none). */
int32_t et_last_cuda_error(void);
/* Number of kernels this library has launched in this process. */
int64_t et_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* ET_H_ */
