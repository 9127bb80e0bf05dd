/*
 * nf.h -- C ABI of the local-layer training step of adaptive local learning
 * (NeuroFlux, arXiv 2402.14139) for NVIDIA B200 (sm_100a).
 *
 * The paper states the problem as: a CNN segmented into blocks by memory use, an
 * auxiliary network per layer, block-specific batch sizes, and cached block outputs
 * (Sections "Overview" and "Design").  The calls below are that statement:
 * a layer with its auxiliary head (Eq. 1, Eq. 2), one pass of the inner body of
 * Algorithm 2 over one batch (nf_layer_step), and the forward-only pass that fills
 * the activation cache of a finished block (nf_block_cache) from which the next
 * block draws batches of its own size (nf_cache_gather).
 *
 * Conventions
 *  - Every pointer named "device" is a CUDA device pointer, 16-byte aligned; "host"
 *    is ordinary host memory.  The library allocates no device memory: all state of
 *    a layer lives in the workspace the caller binds (nf_layer_bind_workspace).
 *  - Activations are channels-last: x[n][h][w][c], element type float (NF_F32) or
 *    bfloat16 (NF_BF16).  Parameters cross the ABI as float in the paper's logical
 *    order: W[Cout][Cin][3][3], Wa[F][Cout][3][3], Wf[classes][4F] where column
 *    f*4 + u*2 + v of Wf multiplies pooled bin (u,v) of aux filter f.
 *  - Calls enqueue work on the stream given to nf_set_stream (default stream 0) and
 *    return without synchronising unless stated.  Buffers must stay valid until the
 *    stream has passed the call.
 *  - Return value: NF_OK (0) or a negative nf_status.  Nothing throws, aborts or
 *    traps.  Conditions found on the device (bad label, non-finite loss, a bounded
 *    wait that ran out) are OR-ed into a per-layer status word read by nf_layer_status.
 */
#ifndef NF_H_
#define NF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct nf_layer nf_layer;
typedef struct nf_block nf_block;

enum nf_status {
  NF_OK = 0,
  NF_EINVAL = -1,       /* bad argument (NULL, non-positive size, unknown enum) */
  NF_EALIGN = -2,       /* a device pointer is not 16-byte aligned */
  NF_ENOWS = -3,        /* no workspace bound, or the bound one is too small */
  NF_EUNSUPPORTED = -4, /* a shape this build has no kernel for */
  NF_ECUDA = -5         /* a CUDA runtime call failed; see nf_last_cuda_error() */
};

/* bits of the device status word */
enum nf_device_flag {
  NF_ELABEL = 1,     /* a label was outside [0, classes); it was clamped */
  NF_ENONFINITE = 2, /* the loss was NaN or infinite */
  NF_ETIMEOUT = 4,   /* a bounded wait inside a kernel ran out; results of that step are invalid */
  NF_EINDEX = 8      /* nf_cache_gather: an index was outside [0, cache_rows); that output row was zero-filled */
};

enum nf_dtype { NF_F32 = 0, NF_BF16 = 1 };

/* Which tensor nf_layer_set_param / nf_layer_get_param address: a parameter id ... */
enum nf_param {
  NF_P_W = 0,     /* theta_n: main conv weights  [Cout][Cin][3][3] */
  NF_P_GAMMA = 1, /* BatchNorm scale             [Cout] */
  NF_P_BETA = 2,  /* BatchNorm shift             [Cout] */
  NF_P_WA = 3,    /* beta_n: aux conv weights    [F][Cout][3][3] */
  NF_P_BA = 4,    /* aux conv bias               [F] */
  NF_P_WF = 5,    /* gamma_n: linear weights     [classes][4F] */
  NF_P_BF = 6,    /* linear bias                 [classes] */
  NF_P_RMEAN = 7, /* running mean                [Cout]  (value only) */
  NF_P_RVAR = 8   /* running variance            [Cout]  (value only) */
};
/* ... plus one of these kinds */
enum nf_param_kind {
  NF_K_VALUE = 0,
  NF_K_MOMENTUM = 0x100, /* the momentum buffer v of the parameter */
  NF_K_GRAD = 0x200      /* the gradient computed by the last nf_layer_step (get only) */
};

/* Options fixed before the workspace is sized.  Zero-initialise, then set fields. */
typedef struct nf_layer_opts {
  int N;             /* batch size the block trains with (block-specific, Section "Adaptive batching") */
  int stride;        /* 1 or 2: stride of the main 3x3 convolution (the down-sampling P_n of ResNet shapes) */
  int maxpool;       /* 1: a 2x2/2 max-pool follows the ReLU and belongs to this layer (P_n of VGG shapes) */
  int dtype;         /* nf_dtype of x, act_out and of the stored activations */
  float momentum;    /* SGD momentum; 0 gives the plain update of the paper's Appendix B */
  float bn_eps;      /* BatchNorm epsilon */
  float bn_momentum; /* running-statistics momentum */
  int host_io;       /* 1: reserve staging so the *_step_host calls can be used; 2: a second input buffer too (nf_block_step_host_next) */
  int loss;          /* nf_loss: the loss L of Eq. 3 (the text beside it names squared error and cross entropy); 0 = cross entropy */
  int aux_pool;      /* nf_aux_pool: the down-sampling F_n of Eq. 2 (the text beside it names max and average pooling); 0 = average */
} nf_layer_opts;

enum nf_loss { NF_LOSS_CE = 0, NF_LOSS_MSE = 1 };        /* MSE: mean over batch and classes of (z - onehot)^2 */
enum nf_aux_pool { NF_POOL_AVG = 0, NF_POOL_MAX = 1 };   /* both adaptive to 2x2; max: first maximum of a bin in row-major order */

/* Create the description of layer n with its auxiliary network A_n (Eq. 1, Eq. 2):
 * conv3x3 Cin->Cout on an H x W input, BatchNorm, ReLU; aux conv3x3 Cout->F, ReLU,
 * average pooling to 2x2, linear 4F->classes.  Host object only; no device work.
 * Defaults: N=1, stride 1, no pool, NF_BF16, momentum 0.9, eps 1e-5, bn_momentum 0.1.
 * Returns NULL if any size is < 1. */
nf_layer* nf_layer_create(int Cin, int Cout, int H, int W, int F, int classes);
void nf_layer_destroy(nf_layer* layer);

/* Set the options; invalidates a bound workspace.  NF_EINVAL on bad values (N < 1, stride
 * not 1 or 2, pool with odd output size, unknown dtype). */
int nf_layer_configure(nf_layer* layer, const nf_layer_opts* opts);

/* Bytes of device memory the layer needs for parameters, momentum, gradients, stored
 * activations and reduction scratch at the configured options. */
size_t nf_layer_workspace_bytes(const nf_layer* layer);

/* Hand the layer its device memory (caller keeps ownership; must outlive the layer's use).
 * Enqueues a clear of the state region and the default initialisation (gamma = 1, running
 * variance = 1, everything else 0).  NF_EALIGN if dev is not 256-byte aligned, NF_ENOWS if
 * bytes < nf_layer_workspace_bytes(). */
int nf_layer_bind_workspace(nf_layer* layer, void* dev, size_t bytes);

/* Copy a parameter tensor (or its momentum) from/to HOST float memory, n = element count of
 * that tensor (NF_EINVAL if it differs).  Both synchronise the stream.  Setting a value also
 * refreshes the reduced-precision copy the kernels read. */
int nf_layer_set_param(nf_layer* layer, int which, const float* host, size_t n);
int nf_layer_get_param(nf_layer* layer, int which, float* host, size_t n);

/* One pass of the inner body of Algorithm 2 for this layer on one batch:
 *   x_{n+1} = ReLU(pool(BN(theta_n * x_n)))            (Eq. 1)      -> act_out
 *   z_{n+1} = gamma_n F_n beta_n x_{n+1}                (Eq. 2)
 *   L = mean cross-entropy(z_{n+1}, labels)             (Eq. 3)      -> loss_out
 *   gradients of (theta_n, beta_n, gamma_n) from L only, no gradient to x_n,
 *   momentum-SGD update with learning rate lr.
 * x:       device, [N][H][W][Cin] of the configured dtype; read only.
 * labels:  device, int32[N], each in [0, classes) (else NF_ELABEL and clamped).
 * loss_out: device, one float.
 * act_out: device, [N][Ha][Wa][Cout] of the configured dtype, Ha = Ho/2 with pool else Ho;
 *          computed with the weights as they were before this call's update; may be a
 *          slice of a cache buffer.  Required (the aux network reads it).
 * Asynchronous.  NF_ENOWS without workspace, NF_EINVAL on NULL, NF_EALIGN on alignment. */
int nf_layer_step(nf_layer* layer, const void* x, const int32_t* labels, float lr, float* loss_out,
                  void* act_out);

/* Same step with HOST buffers (x, labels in; loss and, if non-NULL, act_out back):
 * copies in, runs nf_layer_step, copies out, synchronises.  Needs opts.host_io = 1. */
int nf_layer_step_host(nf_layer* layer, const void* x_host, const int32_t* labels_host, float lr,
                       float* loss_host, void* act_out_host);

/* OR of nf_device_flag bits raised since the last call; synchronises the stream and clears the word. */
int nf_layer_status(nf_layer* layer);

/* A block: consecutive layers trained together at one batch size (Algorithm 1's output).
 * The layers must chain (Cout/Ha/Wa of one = Cin/H/W of the next), share dtype and have
 * workspaces bound.  The block borrows the layers; destroy it before them. */
nf_block* nf_block_create(nf_layer* const* layers, int n_layers);
void nf_block_destroy(nf_block* block);

/* Forward-only pass of a finished block over `count` samples, written to the activation
 * cache (Section "Efficient forward propagation via prefetching and adaptive batching"):
 * every layer runs conv, BatchNorm with its RUNNING statistics, ReLU and pool, so a sample's
 * cached row does not depend on its batch-mates.  No parameter changes.
 * x: device [count][H][W][Cin] of the first layer; out: device [count][Ha][Wa][Cout] of the
 * last layer.  count must be in [1, N] of the block's layers (call repeatedly to cover a
 * dataset); nf_block_cache uses count = N. */
int nf_block_cache(nf_block* block, const void* x, void* out);
int nf_block_cache_n(nf_block* block, const void* x, void* out, int count);

/* Identity shortcut of a residual network (the paper trains ResNet-18 but does not say how a shortcut enters a
 * layer-local step; the reading here: the shortcut tensor is added to the BatchNorm output before the ReLU,
 * x_{n+1} = P(ReLU(BN(theta_n x_n) + skip)), and carries no gradient, like the layer input).  `skip` is a device tensor
 * [N][Ho][Wo][Cout] of the layer's dtype — typically the input of the previous layer — used by every later
 * nf_layer_step / nf_block_step / nf_layer_predict / nf_block_cache call on this layer (for a call with count < N, its
 * first count samples) until it is changed; NULL removes it.  The caller keeps the tensor alive.  Layers with a
 * shortcut run their BatchNorm passes on the generic kernels.  NF_EALIGN if not 16-byte aligned. */
int nf_layer_set_skip(nf_layer* layer, const void* skip);

/* A TRAINABLE shortcut.  nf_layer_set_skip_grad makes every later step on this layer also write dz, the gradient at the sum
 * BN(theta_n x_n) + skip (after the ReLU mask and the pool routing), to dz_out: device, [N][Ho][Wo][Cout] of the layer's
 * dtype; NULL switches it off.  That is the gradient at the shortcut, from which whatever produced the shortcut can train.
 *
 * nf_proj: the projection shortcut of a down-sampling residual block (the paper trains ResNet-18, Section "Experimental
 * Setup", without saying how such a block enters a layer-local step).  Reading taken here: s = BN_p(Wp (*) x_b), a 1x1
 * convolution with stride 2 on the block input x_b [N][H][W][Cin] followed by BatchNorm with batch statistics, joins the
 * layer whose BatchNorm output has its shape, x_{n+1} = P(ReLU(BN(theta_n x_n) + s)); its parameters (Wp [Cout][Cin],
 * gamma_p, beta_p) are trained by THAT layer's local loss and the block input receives no gradient, like every layer input.
 * One local step of such a layer:
 *   nf_proj_forward(proj, x_b, s);  nf_layer_set_skip(layer, s);  nf_layer_set_skip_grad(layer, dz);
 *   nf_layer_step(layer, x, ...);   nf_proj_backward(proj, x_b, dz, lr);
 * nf_proj_forward normalises with the statistics of this batch and updates the running ones; nf_proj_forward_eval uses the
 * running statistics for `count` <= N samples (cache fill, early-exit evaluation); nf_proj_backward computes the gradients of
 * (Wp, gamma_p, beta_p) from dz and applies the momentum update with learning rate lr.  The projection owns no device
 * memory: like a layer it works in a caller-provided workspace (256-byte aligned).  Parameters are addressed by
 * NF_P_W / NF_P_GAMMA / NF_P_BETA / NF_P_RMEAN / NF_P_RVAR plus an nf_param_kind.  Same conventions and error codes as the
 * layer calls; NF_EUNSUPPORTED when Cin exceeds 1536 channels. */
typedef struct nf_proj nf_proj;
int nf_layer_set_skip_grad(nf_layer* layer, void* dz_out);
nf_proj* nf_proj_create(int Cin, int Cout, int H, int W);
void nf_proj_destroy(nf_proj* proj);
int nf_proj_configure(nf_proj* proj, int N, int dtype, float momentum, float bn_eps, float bn_momentum);
size_t nf_proj_workspace_bytes(const nf_proj* proj);
int nf_proj_bind_workspace(nf_proj* proj, void* dev, size_t bytes);
int nf_proj_set_param(nf_proj* proj, int which, const float* host, size_t n);
int nf_proj_get_param(nf_proj* proj, int which, float* host, size_t n);
int nf_proj_forward(nf_proj* proj, const void* xb, void* s_out);
int nf_proj_forward_eval(nf_proj* proj, const void* xb, int count, void* s_out);
int nf_proj_backward(nf_proj* proj, const void* xb, const void* dz, float lr);

/* Data-parallel local step (the paper names distributed training as the direction beyond a single device): the batch
 * of N * world samples is sharded over `world` ranks, every rank holds N of them and a full copy of the layer, and
 * BatchNorm uses the statistics of the WHOLE batch, so the result equals nf_layer_step on the whole batch (up to
 * summation order).  The step is cut where ranks must exchange sums; between phases the caller adds the buffer
 * nf_layer_dp_buffer names over all ranks (an all-reduce sum, in place):
 *   phase 0: conv forward, this rank's per-channel sums of y and y^2      -> all-reduce buffer 0 (2*Cout doubles)
 *   phase 1: normalise, auxiliary forward, loss, auxiliary backward, this rank's BatchNorm-backward sums
 *                                                                          -> all-reduce buffer 1 (2*Cout doubles)
 *   phase 2: BatchNorm backward, weight gradient                           -> all-reduce buffer 2 (every parameter
 *            gradient, fp32) and *loss_out (this rank's share of the mean loss)
 *   phase 3: momentum update (identical on every rank).
 * Same arguments in every phase; x, labels, act_out are this rank's shard.  NF_EINVAL for an unknown phase or world < 1. */
int nf_layer_step_dp(nf_layer* layer, int phase, const void* x, const int32_t* labels, float lr, float* loss_out, void* act_out,
                     int world);
/* Device address and size of exchange buffer `which` (0, 1, 2 as above) inside the bound workspace. */
int nf_layer_dp_buffer(nf_layer* layer, int which, void** dev_ptr, size_t* bytes);

/* The tensors a step leaves in the workspace, for inspection and element-wise checks: device address and size in bytes of
 *   NF_T_Y conv output y [N][Ho][Wo][Cout], NF_T_DY gradient at y, NF_T_H aux conv output after ReLU [N][Ha][Wa][Fp],
 *   NF_T_DH gradient at h, NF_T_DA gradient at the activation [N][Ha][Wa][Cout]  (all of the layer's dtype; Fp = F rounded
 *   up to a multiple of 8, the extra channels are zero),
 *   NF_T_P pooled aux output [N][4*Fp], NF_T_DP its gradient, NF_T_LOGITS [N][classes]  (float),
 *   NF_T_HMASK the signs of h, one bit per element: bytes [N][Ha][Wa][Fp/8], bit f%8 of byte f/8 set where h > 0.  A layer
 *   whose nf_layer_kernel_family(layer, 5) is "mask" keeps this instead of h (its aux forward pools h in its epilogue and
 *   never stores it; the mask shares h's memory); otherwise h is stored and the mask is not.
 * Valid after a step on that layer and until the next call on it; a kernel that does not need one of them on some
 * shape may leave it unwritten.  NF_EINVAL for an unknown id, NF_ENOWS without workspace. */
enum nf_stored { NF_T_Y = 0, NF_T_DY = 1, NF_T_H = 2, NF_T_DH = 3, NF_T_DA = 4, NF_T_P = 5, NF_T_DP = 6, NF_T_LOGITS = 7, NF_T_HMASK = 8 };
int nf_layer_stored_tensor(nf_layer* layer, int which, void** dev_ptr, size_t* bytes);

/* Early-exit evaluation (Section "Trained output CNN": every layer with its auxiliary network is a
 * prospective exit point).  Forward only, BatchNorm with running statistics, no parameter changes:
 *   act_out = x_{n+1} for `count` samples (device, [count][Ha][Wa][Cout]; NULL keeps it in the workspace),
 *   logits_out = z_{n+1} (device float [count][classes]; may be NULL),
 *   pred_out = arg-max class per sample, first maximum (device int32 [count]).
 * count must be in [1, N].  Feed act_out to the next layer's nf_layer_predict to evaluate deeper exits. */
int nf_layer_predict(nf_layer* layer, const void* x, int count, void* act_out, float* logits_out, int32_t* pred_out);

/* Validation accuracy of an exit: *count += #{i < n : a[i] == b[i]} (device int32 arrays, device 64-bit counter that
 * the caller zeroes; integer accumulation, so the result does not depend on launch order). */
int nf_count_equal(const int32_t* a, const int32_t* b, long long n, unsigned long long* count);

/* Parameters of a layer: part 0 = main path (W, gamma, beta), 1 = auxiliary network (Wa, ba, Wf, bf), 2 = both.
 * An early-exit model at layer n holds the main parts of layers 1..n plus the auxiliary part of layer n. */
long long nf_layer_param_count(const nf_layer* layer, int part);

/* Exit selection (host only): the index with the highest validation accuracy; among equals the one with the
 * fewest parameters.  NF_EINVAL on bad arguments. */
int nf_select_exit(const double* val_accuracy, const long long* params, int n_layers);

/* One pass of Algorithm 2's inner loop over ALL layers of the block on one batch: layer 1 steps
 * on x, every later layer steps on the activation its predecessor just produced (computed before
 * that predecessor's update), each with its own local loss.
 * x: device [N][H][W][Cin] of the first layer; labels: device int32[N];
 * loss_out: device float[n_layers] (one local loss per layer);
 * act_out: device [N][Ha][Wa][Cout] of the last layer, or NULL to keep it in the layer's workspace. */
int nf_block_step(nf_block* block, const void* x, const int32_t* labels, float lr, float* loss_out, void* act_out);

/* The same pass with HOST buffers: copies x and labels in, runs nf_block_step, copies the n_layers
 * losses (and, if act_out_host is non-NULL, the last activation) back, synchronises.
 * The first layer must have been configured with host_io = 1. */
int nf_block_step_host(nf_block* block, const void* x_host, const int32_t* labels_host, float lr,
                       float* loss_host, void* act_out_host);

/* nf_block_step_host for a stream of batches: while this batch trains, the NEXT batch's host buffers (pinned; may be
 * NULL for the last one) are copied into the second staging buffer on a copy stream; the following call, given those
 * same pointers as its batch, finds the copy done or in flight and only waits for it.  Every batch is still copied
 * host -> device exactly once and the call still returns after the step has finished and the losses are in loss_host.
 * Needs opts.host_io = 2 on the first layer.  The contents of a prefetched batch must not change until its step. */
int nf_block_step_host_next(nf_block* block, const void* x_host, const int32_t* labels_host, float lr, float* loss_host,
                            void* act_host, const void* next_x_host, const int32_t* next_labels_host);

/* Re-batching from the cache: out[i] = cache[idx[i]] for i < count, rows of row_bytes bytes
 * (a multiple of 16); labels likewise if both label pointers are non-NULL.  All device pointers.
 * Bit-exact copy.  cache_rows is the number of rows the cache holds: an index outside [0, cache_rows)
 * (a stale or corrupt permutation) reads nothing -- its output row is zero-filled, its label set to -1
 * and NF_EINDEX is raised in the status word nf_op_status() returns. */
int nf_cache_gather(const void* cache, const int32_t* cache_labels, int cache_rows, const int32_t* idx, int count,
                    size_t row_bytes, void* out, int32_t* out_labels);

/* Stand-alone forms of the two dense contractions of the step (Eq. 1's theta_n x_n and the
 * gradient of Algorithm 2's line "compute the gradient" with respect to theta_n), for callers that compose
 * their own step and for kernel-level checks.  All pointers device; activations channels-last of
 * `dtype`; weights w and the result dw are laid out [kh*3+kw][Cout][Cin] (w of `dtype`, dw float).
 *   nf_conv3x3_forward: y[n][i][j][co] = sum w[tap][co][ci] * x[n][i*stride+kh-1][j*stride+kw-1][ci], zero padding.
 *   nf_conv3x3_wgrad:   dw[tap][co][ci] = sum over n,i,j of g[n][i][j][co] * x[n][i*stride+kh-1][j*stride+kw-1][ci];
 *     needs nf_conv3x3_wgrad_scratch_bytes() of device scratch for its split partial sums (fully
 *     overwritten, nothing has to be cleared); NF_ENOWS if scratch_bytes is smaller.
 * Asynchronous on the library's stream. */
int nf_conv3x3_forward(int dtype, const void* x, const void* w, int N, int H, int W, int Cin, int Cout, int stride,
                       void* y);
/* OR of nf_device_flag bits raised by the stand-alone operations since the last call; synchronises. */
int nf_op_status(void);
size_t nf_conv3x3_wgrad_scratch_bytes(int N, int H, int W, int Cin, int Cout, int stride);
int nf_conv3x3_wgrad(int dtype, const void* x, const void* g, int N, int H, int W, int Cin, int Cout, int stride,
                     void* scratch, size_t scratch_bytes, float* dw);

/* The same weight gradient for callers that cannot hand over scratch memory.  (The paper has no
 * counterpart; this is a convenience of this library.)  Some callers are unable to allocate on the
 * device at the moment they need the gradient: a trainer that has already given its whole memory
 * budget to activations and caches, as the budgeted setting this method is built for does by
 * design, or code running where a device allocation's implicit synchronisation is unwelcome.  This
 * variant keeps the split partial sums in a fixed array inside the library image instead:
 *  - the array is NF_STATIC_SCRATCH_BYTES (16 MiB) and is held by every GPU that loads the library
 *    until the process exits;
 *  - a problem whose nf_conv3x3_wgrad_scratch_bytes() exceeds that is refused with NF_ENOWS and
 *    nothing is launched;
 *  - the first call on each device looks up the array's device address (with that device current);
 *    make that first call before starting any stream capture;
 *  - all calls share the one array and it keeps whatever the previous call left.  Nothing in it
 *    has to start at zero (every partial that is read is written first by the same call), but two
 *    calls that overlap on the GPU (different streams, different host threads) race on it: run
 *    them one after the other.
 * It makes no cudaMalloc/cudaFree and calls no allocating routine.  Arguments and result are
 * those of nf_conv3x3_wgrad without the scratch pair. */
#define NF_STATIC_SCRATCH_BYTES (16u << 20)
int nf_conv3x3_wgrad_static(int dtype, const void* x, const void* g, int N, int H, int W, int Cin, int Cout,
                            int stride, float* dw);

/* Algorithm 1 (host only, no device work): given each layer's largest feasible batch size,
 * cap at B and group consecutive layers while |b[i+1]-b[i]| <= rho*b[i]; a block's batch size
 * is the minimum over its members.  Writes up to n_layers entries of first layer index and
 * batch size; returns the number of blocks, or NF_EINVAL. */
int nf_partition(const int* max_batch, int n_layers, int B, double rho, int* block_first, int* block_batch);

/* The Profiler (Section "Modules"; host only, no device work).
 *
 * nf_aan_filters: the AAN-LL rule for the auxiliary filter counts.  channels[i] = filters of CNN layer i;
 * layers with index < first_downsample (those before the first down-sampling operation) get half the SMALLEST
 * entry of channels, all later layers half the LARGEST (VGG: 32 and 256).  Writes n_layers counts.
 *
 * nf_profile_layer: the device memory this library needs to train one layer (its workspace plus one input
 * batch) at each of the k given batch sizes, and the least-squares line bytes = intercept + slope * batch
 * through them (k >= 2 distinct sizes; bytes_out may be NULL).  opts->N is ignored.
 *
 * nf_fit_line: the same least-squares line through k >= 2 MEASURED (batch size, bytes) pairs, for a caller that profiles by
 * running steps and reading the device's memory counters, as the paper's Profiler does.
 *
 * nf_max_batch: the largest batch t with intercept + slope * t <= budget (first loop of Algorithm 1);
 * 0 if even one sample does not fit.  Feed the results to nf_partition.
 * All return NF_EINVAL on bad arguments. */
int nf_aan_filters(const int* channels, int n_layers, int first_downsample, int* filters_out);
int nf_profile_layer(int Cin, int Cout, int H, int W, int F, int classes, const nf_layer_opts* opts, const int* batches, int k,
                     double* bytes_out, double* slope, double* intercept);
int nf_fit_line(const double* batches, const double* bytes, int k, double* slope, double* intercept);
long long nf_max_batch(double slope, double intercept, double budget_bytes);

/* Stream for all later calls (a cudaStream_t); NULL selects the default stream. */
int nf_set_stream(void* cuda_stream);

/* Per-operation device timing (CUDA events on the library's stream around each group of kernels).
 * nf_trace_enable(1) starts recording and clears the totals; nf_trace_read synchronises the stream
 * and returns, for op in [0, NF_TRACE_OPS) and layer position slot in [0, NF_TRACE_SLOTS) (the index
 * of the layer inside the block for nf_block_step, 0 for a bare nf_layer_step), the summed
 * milliseconds and the number of timed groups.
 * Ops: 0 main conv forward (+statistics partials), 1 BatchNorm finalize+apply, 2 aux conv forward,
 * 3 pooling + linear + cross-entropy forward/backward, 4 aux conv backward, first part (dh and the aux weight and bias
 * gradients), 5 BatchNorm backward, 6 main conv weight gradient, 7 SGD update, 8 aux conv backward, second part (the
 * gradient at the aux input; on two-pass shapes its first run, the second being part of op 5). */
enum { NF_TRACE_OPS = 9, NF_TRACE_SLOTS = 32 };
int nf_trace_enable(int on);
int nf_trace_read(int op, int slot, double* ms_total, long long* groups);

/* Self-check of the hang safety of the tensor-core kernels.  Every wait inside them (on an mbarrier that a TMA copy or
 * a tcgen05.commit completes) is bounded in time; when one runs out the waiter sets an abort flag, every role of the CTA
 * leaves its loop, and NF_ETIMEOUT is raised instead of the kernel spinning forever.  This call exercises exactly that
 * wait routine in isolation: one CTA of one warp, no TMA, no tensor memory, waits limit_ns (1 .. 1e9) on a barrier that
 * nobody arrives at, gives up, raises NF_ETIMEOUT in the status word nf_op_status() returns and writes the nanoseconds
 * it waited to *waited_ns_dev (device, 8-byte aligned).  Asynchronous on the library's stream. */
int nf_selftest_bounded_wait(unsigned long long limit_ns, unsigned long long* waited_ns_dev);

/* Kernel launches enqueued by this library since the process started. */
long long nf_launch_count(void);

/* Name of the kernel family a configured layer uses for op 0 = main forward,
 * 1 = main weight gradient, 2 = aux forward, 3 = aux backward: "tcgen05" or "cuda-core".
 * op 4: "fused" when the BatchNorm + ReLU pass of the step runs inside the aux forward kernel
 * (which then also writes act_out), "separate" otherwise.
 * op 5: "mask" when that kernel also pools the aux output h in its epilogue and keeps only one sign bit per element of it
 * (Eq. 2's F_n applied before h ever reaches memory), "stored" when h is written and pooled by separate kernels.
 * op 6: "two-pass" when the aux input gradient runs twice -- once to reduce the BatchNorm-backward sums, once more to write
 * the gradient at the conv output directly -- so that the gradient at the activation (NF_T_DA) is never stored and no
 * separate BatchNorm-backward pass runs; "stored" otherwise. */
const char* nf_layer_kernel_family(const nf_layer* layer, int op);

const char* nf_strerror(int status);
const char* nf_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* NF_H_ */
