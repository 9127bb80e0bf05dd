// Internal definitions shared by the translation units of libnf (not part of the ABI).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/nf.h"

typedef __nv_bfloat16 bf16;

// Parameter arena: all trainable tensors of a layer, contiguous, in the layout the kernels read.
//   W  : [tap = kh*3+kw][Cout][Cin]      gamma, beta : [Cout]
//   Wa : [tap][F][Cout]                  ba : [F]
//   Wf : [classes][4F]                   bf : [classes]
// Every tensor starts at a multiple of 64 elements.  Four parallel arenas share the offsets:
// fp32 value, fp32 momentum, fp32 gradient, bf16 copy of the value.
enum { NF_NPARAM = 7 };

struct nf_layer {
  // description
  int Cin, Cout, H, W, F, classes;  // F = aux filters as the kernels see them: the caller's count rounded up to a
                                    // multiple of 8; the extra filters have zero weights, get zero gradients, stay zero
  int Flog;                         // the caller's aux filter count
  nf_layer_opts o;
  int Ho, Wo, Ha, Wa;  // conv output size; size after the optional pool
  // arena
  size_t off[NF_NPARAM], cnt[NF_NPARAM], arena;  // element offsets / counts / total (padded)
  // workspace
  char* ws;
  size_t ws_bytes;
  int32_t* status;                     // device status word
  float *val, *mom, *grad;             // arenas
  bf16* shadow;                        // bf16 arena
  const void* skip;                    // identity shortcut for the next calls (nf_layer_set_skip), or NULL
  void* skip_grad;                     // where each step also writes dz, the gradient at the shortcut (nf_layer_set_skip_grad), or NULL
  bf16* wa_t;                          // [9][Cout][F] mirrored, transposed copy of Wa (only when F > 64)
  float *rmean, *rvar;                 // [Cout]
  float *scale, *shift, *mu, *invstd;  // [Cout] per-step BatchNorm coefficients
  float *sdz, *sdzx;                   // [Cout] reduced sums for BatchNorm backward
  void* y;                             // [N][Ho][Wo][Cout] conv output (dtype)
  void* dy;                            // [N][Ho][Wo][Cout] gradient at conv output (dtype)
  void* h;                             // [N][Ha][Wa][F] aux conv output after ReLU (dtype)
  void* dh;                            // [N][Ha][Wa][F]
  void* da;                            // [N][Ha][Wa][Cout]
  void* act;                           // [N][Ha][Wa][Cout] activation kept here when the caller gives no buffer
  float *p, *dp;                       // [N][4F]
  double* dptot;                       // [2][2][Cout] per-channel totals exchanged between ranks (data-parallel step)
  int32_t* parg;                       // [N][4F] position i*Wa+j of each bin's maximum (max-pool down-sampling only)
  float *logits, *dlogits;             // [N][classes]
  float* lossn;                        // [N]
  float* red;                          // reduction scratch (channel partials)
  size_t red_floats;
  float* wpart;                        // split-K partials of the weight gradients
  size_t wpart_floats;
  void* stage_x;                       // host_io staging
  void* stage_xb[2];                   // host_io = 2: two input staging buffers (stage_xb[0] == stage_x)
  int32_t* stage_lb[2];
  int stage_cur;                       // buffer the next step reads
  const void* pre_x;                   // host batch already on its way into buffer 1 - stage_cur (or NULL)
  const int32_t* pre_l;
  int32_t* stage_labels;
  void* stage_act;
  float* stage_loss;
  // kernel families chosen at configure time: 0 = cuda-core, 1 = tcgen05
  int fam[4];
  // First layers (a few input channels, e.g. RGB): cin_pad = 64 makes the main conv run on the tensor-core kernels over a
  // copy of the input batch whose pixels are zero-padded to 64 channels; 0 = the input is used as it is.
  int cin_pad;
  void* xpad;                          // [N][H][W][cin_pad] (bf16)
  bf16* wpad;                          // [9][Cout][cin_pad] operand copy of W, zero beyond Cin
  float* gwpad;                        // [9][Cout][cin_pad] weight gradient over the padded channels
};

struct nf_block {
  int n;
  nf_layer** layers;
};

// launch bookkeeping (nf_api.cu)
extern cudaStream_t g_nf_stream;
extern long long g_nf_launches;
int nf_cuda_check(cudaError_t e, const char* what);
#define NF_CUDA(x)                                        \
  do {                                                    \
    if (nf_cuda_check((x), #x) != NF_OK) return NF_ECUDA; \
  } while (0)
#define NF_LAUNCHED()                                                          \
  do {                                                                         \
    ++g_nf_launches;                                                           \
    if (nf_cuda_check(cudaGetLastError(), "launch") != NF_OK) return NF_ECUDA; \
  } while (0)

static inline size_t nf_align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline size_t nf_esize(int dtype) { return dtype == NF_F32 ? 4 : 2; }

// ---- generic CUDA-core kernels (nf_k_kernels.cu): any shape, fp32 or bf16 storage, fp32 accumulate
int nf_k_conv(int dtype, const void* x, int N, int H, int W, int Ci, const void* w, long ws_tap, long ws_co,
                long ws_ci, int flip, const float* bias, int relu, int stride, int Co, void* y);
int nf_k_wgrad_splits(int N, int Ho, int Ci, int Co);
int nf_k_wgrad(int dtype, const void* x, int N, int H, int W, int Ci, const void* g, int Co, int stride,
                 float* part, size_t part_floats, float* dw);
int nf_k_channel_blocks(size_t P, int C);
int nf_k_channel_sums(int dtype, const void* src, size_t P, int C, float* red, size_t red_floats, int* nblocks);
int nf_k_bn_finalize(const float* red, int nblocks, int C, double M, const float* gamma, const float* beta,
                       float eps, float bn_momentum, float* scale, float* shift, float* mu, float* invstd,
                       float* rmean, float* rvar);
int nf_k_bn_eval_coeffs(int C, const float* gamma, const float* beta, float eps, const float* rmean,
                          const float* rvar, float* scale, float* shift);
int nf_k_bn_apply(int dtype, const void* y, int N, int Ho, int Wo, int C, int pool, const float* scale,
                    const float* shift, void* out, const void* skip = nullptr);
int nf_k_avgpool(int dtype, const void* h, int N, int Ha, int Wa, int F, float* p);
// bf16 fast paths (F % 8 == 0, even Ha and Wa); NF_EUNSUPPORTED means "use the generic kernel"
int nf_k_avgpool_fast(const void* h, int N, int Ha, int Wa, int F, float* part, size_t part_floats, float* p);
int nf_k_dh_fast(const void* h, const float* dp, int N, int Ha, int Wa, int F, void* dh, float* red, size_t red_floats,
                   int* nblocks);
// average pool from the per-tile partials of the fused aux forward, and dh from its sign mask (see nf_tc_aux_pool_fused)
int nf_k_pool_finish(const float* part, int N, int th, int tw, int F, float inv_cnt, float* p);
int nf_k_dh_mask(const uint8_t* mask, const float* dp, int N, int Ha, int Wa, int F, void* dh, float* red, size_t red_floats,
                 int* nblocks);
int nf_k_fc_ce(const float* p, const int32_t* labels, int N, int D, int K, const float* Wf, const float* bf,
                 float* logits, float* dlogits, float* dp, float* lossn, int32_t* status, int loss_kind, int n_scale);
int nf_k_count_equal(const int32_t* a, const int32_t* b, long long n, unsigned long long* count);
int nf_k_auxmax(int dtype, const void* h, int N, int Ha, int Wa, int F, float* p, int32_t* parg);
int nf_k_dh_max(int dtype, const void* h, const float* dp, const int32_t* parg, int N, int Ha, int Wa, int F, void* dh);
int nf_k_flip_weights(const bf16* w, int F, int C, bf16* out);
// large-batch head (nf_head.cu)
bool nf_head_is_large(int N, int D, int K);
size_t nf_head_scratch_floats(int N, int D, int K);
int nf_head_logits(const float* p, int N, int D, int K, const float* Wf, const float* bf, float* logits, float* scratch);
int nf_head_predict(const float* logits, int N, int K, int32_t* pred);
int nf_head_step(const float* p, const int32_t* labels, int N, int D, int K, const float* Wf, const float* bf, float* logits,
                 float* dlogits, float* dp, float* lossn, int32_t* status, int loss_kind, float* gWf, float* gbf, float* loss_out,
                 float* scratch, size_t scratch_floats, int n_scale);
// small-batch head (nf_head_small.cu): class-sliced forward + backward of the linear layer and the loss; 0 floats = not covered
size_t nf_head_small_scratch_floats(int N, int D, int K);
int nf_head_small_step(const float* p, const int32_t* labels, int N, int D, int K, const float* Wf, const float* bf, float* logits,
                       float* dp, float* lossn, int32_t* status, int loss_kind, float* gWf, float* gbf, float* loss_out,
                       float* scratch, size_t scratch_floats, int n_scale);
int nf_k_partial_totals(const float* red, int nblocks, int C, double* tot);
int nf_k_bn_finalize_tot(const double* tot, int C, double M, const float* gamma, const float* beta, float eps, float bn_momentum,
                           float* scale, float* shift, float* mu, float* invstd, float* rmean, float* rvar);
int nf_k_bn_bwd_finalize_tot(const double* tot, int C, int world, float* sdz, float* sdzx, float* ggamma, float* gbeta);
int nf_k_fc_predict(const float* p, int N, int D, int K, const float* Wf, const float* bf, float* logits, int32_t* pred);
int nf_k_fc_wgrad(const float* p, const float* dlogits, const float* lossn, int N, int D, int K, float* gWf,
                    float* gbf, float* loss_out, int32_t* status, int n_scale);
int nf_k_dh(int dtype, const void* h, const float* dp, int N, int Ha, int Wa, int F, void* dh);
int nf_k_sum_partials(const float* red, int nblocks, int C, int which, float* out);
int nf_k_bn_bwd_reduce(int dtype, const void* y, const void* da, int N, int Ho, int Wo, int C, int pool,
                         const float* scale, const float* shift, const float* mu, const float* invstd, float* red,
                         size_t red_floats, int* nblocks, const void* skip = nullptr);
int nf_k_bn_bwd_finalize(const float* red, int nblocks, int C, float* sdz, float* sdzx, float* ggamma,
                           float* gbeta);
int nf_k_bn_bwd_apply(int dtype, const void* y, const void* da, int N, int Ho, int Wo, int C, int pool,
                        const float* scale, const float* shift, const float* mu, const float* invstd,
                        const float* sdz, const float* sdzx, double M, void* dy, const void* skip = nullptr);
int nf_k_write_dz(int dtype, const void* y, const void* da, int N, int Ho, int Wo, int C, int pool, const float* scale,
                  const float* shift, const void* skip, void* dz);
// channel padding of a first layer's input and weights, and the gradient of the real channels out of the padded result
int nf_k_pad_channels(const void* x, size_t P, int C, int Cp, void* xpad);
int nf_k_pad_weights(const bf16* w, size_t rows, int C, int Cp, bf16* wpad);
int nf_k_unpad_grad(const float* gwpad, size_t rows, int C, int Cp, float* gw);
int nf_k_sgd(float* val, float* mom, const float* grad, bf16* shadow, size_t n, float lr, float momentum);
// the same update over several arenas (the layers of a block) in one launch; first_block is filled by the callee
enum { kSgdMaxArenas = 48 };
struct SgdTable {
  int count;
  float* val[kSgdMaxArenas];
  float* mom[kSgdMaxArenas];
  const float* grad[kSgdMaxArenas];
  bf16* shadow[kSgdMaxArenas];
  size_t n[kSgdMaxArenas];
  int first_block[kSgdMaxArenas];
};
int nf_k_sgd_multi(const SgdTable& tb, float lr, float momentum);
int nf_k_shadow(const float* val, bf16* shadow, size_t n);
int nf_k_gather(const void* cache, const int32_t* cache_labels, int cache_rows, const int32_t* idx, int count, size_t row_bytes,
                void* out, int32_t* out_labels, int32_t* status);
