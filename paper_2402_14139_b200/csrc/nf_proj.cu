// Projection shortcut of a down-sampling residual block (the paper trains ResNet-18): s = BN(Wp (*) x_b), a 1x1 convolution
// with stride 2 on the block input x_b followed by BatchNorm with batch statistics.  s is added to the BatchNorm output of
// the layer it joins (nf_layer_set_skip); that layer's local loss trains (Wp, gamma_p, beta_p) through the gradient dz at
// the sum (nf_layer_set_skip_grad); the block input receives no gradient.  Generic CUDA-core kernels, fp32 or bf16 storage,
// fp32 arithmetic, every reduction in a fixed order.
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "nf_internal.h"
#include "nf_ldst.cuh"

struct nf_proj {
  int Cin, Cout, H, W, Ho, Wo;
  int N, dtype;
  float momentum, eps, bn_momentum;
  size_t arena, offW, offG, offB;   // arena: Wp in kernel layout [Cin][Cout], gamma, beta (each at a multiple of 64 floats)
  char* ws;
  float *val, *mom, *grad;
  bf16* shadow;
  float *rmean, *rvar, *scale, *shift, *mu, *invstd, *sdz, *sdzx;
  void* ys;                         // [N][Ho][Wo][Cout] conv output (dtype)
  void* dys;                        // [N][Ho][Wo][Cout] gradient at it (dtype)
  float* red;
  size_t red_floats;
  float* wpart;                     // [splits][Cin][Cout]
  int splits;
};

namespace {

constexpr int kPix = 8;  // output pixels per block of the forward kernel

// ys[pix][co] = sum_ci w[ci][co] * x[n][s*i][s*j][ci]; block: kPix pixels, thread <-> output channel (strided over Cout)
template <typename T>
__global__ void __launch_bounds__(256) proj_fwd_kernel(const T* __restrict__ x, const T* __restrict__ w, int H, int W, int Ci, int Co,
                                                       int Ho, int Wo, size_t P, int stride, T* __restrict__ ys) {
  extern __shared__ float xs[];  // [kPix][Ci]
  const size_t p0 = (size_t)blockIdx.x * kPix;
  for (int i = threadIdx.x; i < kPix * Ci; i += 256) {
    const size_t p = p0 + i / Ci;
    float v = 0.f;
    if (p < P) {
      const int j = (int)(p % Wo), r = (int)((p / Wo) % Ho);
      const size_t n = p / ((size_t)Wo * Ho);
      v = ldf(x, ((n * H + (size_t)r * stride) * W + (size_t)j * stride) * Ci + i % Ci);
    }
    xs[i] = v;
  }
  __syncthreads();
  for (int co = threadIdx.x; co < Co; co += 256) {
    float acc[kPix];
#pragma unroll
    for (int q = 0; q < kPix; ++q) acc[q] = 0.f;
    for (int ci = 0; ci < Ci; ++ci) {
      const float wv = ldf(w, (size_t)ci * Co + co);
#pragma unroll
      for (int q = 0; q < kPix; ++q) acc[q] = fmaf(wv, xs[q * Ci + ci], acc[q]);
    }
#pragma unroll
    for (int q = 0; q < kPix; ++q)
      if (p0 + q < P) stf(ys, (p0 + q) * Co + co, acc[q]);
  }
}

// s = ys * scale + shift (no activation: the sum with the layer's BatchNorm output passes through the layer's ReLU)
template <typename T>
__global__ void proj_affine_kernel(const T* __restrict__ ys, int C, const float* __restrict__ scale, const float* __restrict__ shift,
                                   size_t total, T* __restrict__ s) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int c = (int)(e % C);
  stf(s, e, fmaf(ldf(ys, e), scale[c], shift[c]));
}

// partial sums of (dz, dz * shat), shat = (ys - mu) * invstd: red[(block*2 + k)*C + c], pixel ranges per block, fixed order
template <typename T>
__global__ void __launch_bounds__(256) proj_bwd_reduce_kernel(const T* __restrict__ ys, const T* __restrict__ dz, size_t P, int C,
                                                              const float* __restrict__ mu, const float* __restrict__ invstd,
                                                              float* __restrict__ red) {
  const size_t p0 = P * blockIdx.x / gridDim.x, p1 = P * (blockIdx.x + 1) / gridDim.x;
  for (int c = threadIdx.x; c < C; c += 256) {
    float a = 0.f, b = 0.f;
    const float m = mu[c], is = invstd[c];
    for (size_t p = p0; p < p1; ++p) {
      const float g = ldf(dz, p * C + c);
      a += g;
      b = fmaf(g, (ldf(ys, p * C + c) - m) * is, b);
    }
    red[((size_t)blockIdx.x * 2 + 0) * C + c] = a;
    red[((size_t)blockIdx.x * 2 + 1) * C + c] = b;
  }
}

// dys = scale * (dz - sum(dz)/M - shat * sum(dz*shat)/M)
template <typename T>
__global__ void proj_bwd_apply_kernel(const T* __restrict__ ys, const T* __restrict__ dz, int C, const float* __restrict__ scale,
                                      const float* __restrict__ mu, const float* __restrict__ invstd, const float* __restrict__ sdz,
                                      const float* __restrict__ sdzx, float invM, size_t total, T* __restrict__ dys) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int c = (int)(e % C);
  const float sh = (ldf(ys, e) - mu[c]) * invstd[c];
  stf(dys, e, scale[c] * (ldf(dz, e) - sdz[c] * invM - sh * sdzx[c] * invM));
}

// part[split][ci][co] = sum over the split's pixel range (ascending) of dys[pix][co] * x[n][s*i][s*j][ci];
// block: 16 input channels x 64 output channels, thread <-> (4 input channels, one output channel)
template <typename T>
__global__ void __launch_bounds__(256) proj_wgrad_kernel(const T* __restrict__ x, const T* __restrict__ dys, int H, int W, int Ci, int Co,
                                                         int Ho, int Wo, size_t P, int stride, int splits, float* __restrict__ part) {
  __shared__ float xs[16][16];   // [pixel][ci]
  __shared__ float gs[16][64];   // [pixel][co]
  const int ci0 = blockIdx.x * 16, co0 = blockIdx.y * 64, sp = blockIdx.z;
  const size_t p0 = P * sp / splits, p1 = P * (sp + 1) / splits;
  const int tco = threadIdx.x & 63, tci = (threadIdx.x >> 6) * 4;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (size_t pb = p0; pb < p1; pb += 16) {
    {
      const int q = threadIdx.x >> 4, c = threadIdx.x & 15;
      const size_t p = pb + q;
      float v = 0.f;
      if (p < p1 && ci0 + c < Ci) {
        const int j = (int)(p % Wo), r = (int)((p / Wo) % Ho);
        const size_t n = p / ((size_t)Wo * Ho);
        v = ldf(x, ((n * H + (size_t)r * stride) * W + (size_t)j * stride) * Ci + ci0 + c);
      }
      xs[q][c] = v;
    }
    for (int i = threadIdx.x; i < 16 * 64; i += 256) {
      const int q = i >> 6, c = i & 63;
      const size_t p = pb + q;
      gs[q][c] = (p < p1 && co0 + c < Co) ? ldf(dys, p * Co + co0 + c) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 16; ++q) {
      const float g = gs[q][tco];
#pragma unroll
      for (int u = 0; u < 4; ++u) acc[u] = fmaf(g, xs[q][tci + u], acc[u]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < 4; ++u)
    if (ci0 + tci + u < Ci && co0 + tco < Co) part[((size_t)sp * Ci + ci0 + tci + u) * Co + co0 + tco] = acc[u];
}

__global__ void proj_sum_splits_kernel(const float* __restrict__ part, int splits, size_t n, float* __restrict__ out) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float s = 0.f;
  for (int k = 0; k < splits; ++k) s += part[(size_t)k * n + i];
  out[i] = s;
}

inline unsigned blocks_for(size_t n, int per) { return (unsigned)((n + per - 1) / per); }

}  // namespace

namespace {

constexpr int kProjBlocks = 296;  // pixel ranges of the BatchNorm-backward reduction

size_t proj_plan(nf_proj* P, char* base) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    off = nf_align_up(off, 256);
    void* p = base ? base + off : nullptr;
    off += bytes;
    return p;
  };
  const size_t C = P->Cout, es = nf_esize(P->dtype), ny = (size_t)P->N * P->Ho * P->Wo * C;
  P->val = (float*)take(P->arena * 4);
  P->mom = (float*)take(P->arena * 4);
  P->grad = (float*)take(P->arena * 4);
  P->shadow = (bf16*)take(P->arena * 2);
  float** small[] = {&P->rmean, &P->rvar, &P->scale, &P->shift, &P->mu, &P->invstd, &P->sdz, &P->sdzx};
  for (float** q : small) *q = (float*)take(C * 4);
  const size_t state_end = off;
  P->ys = take(ny * es);
  P->dys = take(ny * es);
  const size_t r1 = (size_t)nf_k_channel_blocks((size_t)P->N * P->Ho * P->Wo, (int)C) * 2 * C, r2 = (size_t)kProjBlocks * 2 * C;
  P->red_floats = r1 > r2 ? r1 : r2;
  P->red = (float*)take(P->red_floats * 4);
  const size_t pix = (size_t)P->N * P->Ho * P->Wo;
  const int tiles = ((P->Cin + 15) / 16) * ((P->Cout + 63) / 64);
  long sp = 592 / tiles;  // about four waves of blocks
  if (sp < 1) sp = 1;
  if ((size_t)sp > (pix + 15) / 16) sp = (long)((pix + 15) / 16);
  P->splits = (int)sp;
  P->wpart = (float*)take((size_t)sp * P->Cin * P->Cout * 4);
  (void)state_end;
  return nf_align_up(off, 256);
}

void proj_derive(nf_proj* P) {
  P->Ho = (P->H - 1) / 2 + 1;
  P->Wo = (P->W - 1) / 2 + 1;
  P->offW = 0;
  P->offG = nf_align_up((size_t)P->Cin * P->Cout, 64);
  P->offB = nf_align_up(P->offG + P->Cout, 64);
  P->arena = nf_align_up(P->offB + P->Cout, 64);
}

}  // namespace

extern "C" {

nf_proj* nf_proj_create(int Cin, int Cout, int H, int W) {
  if (Cin < 1 || Cout < 1 || H < 1 || W < 1) return nullptr;
  nf_proj* P = (nf_proj*)calloc(1, sizeof(nf_proj));
  if (!P) return nullptr;
  P->Cin = Cin; P->Cout = Cout; P->H = H; P->W = W;
  P->N = 1; P->dtype = NF_BF16; P->momentum = 0.9f; P->eps = 1e-5f; P->bn_momentum = 0.1f;
  proj_derive(P);
  return P;
}

void nf_proj_destroy(nf_proj* P) { free(P); }

int nf_proj_configure(nf_proj* P, int N, int dtype, float momentum, float bn_eps, float bn_momentum) {
  if (!P || N < 1 || (dtype != NF_F32 && dtype != NF_BF16) || !(momentum >= 0.f && momentum < 1.f) || !(bn_eps > 0.f) ||
      !(bn_momentum >= 0.f && bn_momentum <= 1.f))
    return NF_EINVAL;
  P->N = N; P->dtype = dtype; P->momentum = momentum; P->eps = bn_eps; P->bn_momentum = bn_momentum;
  P->ws = nullptr;
  return NF_OK;
}

size_t nf_proj_workspace_bytes(const nf_proj* P) {
  if (!P) return 0;
  nf_proj tmp = *P;
  return proj_plan(&tmp, nullptr);
}

int nf_proj_bind_workspace(nf_proj* P, void* dev, size_t bytes) {
  if (!P || !dev) return NF_EINVAL;
  if ((uintptr_t)dev & 255) return NF_EALIGN;
  if (bytes < nf_proj_workspace_bytes(P)) return NF_ENOWS;
  proj_plan(P, (char*)dev);
  P->ws = (char*)dev;
  const size_t state = (size_t)((char*)P->ys - (char*)dev);
  NF_CUDA(cudaMemsetAsync(dev, 0, state, g_nf_stream));
  std::vector<float> ones(P->Cout, 1.0f);
  NF_CUDA(cudaMemcpyAsync(P->val + P->offG, ones.data(), P->Cout * 4, cudaMemcpyHostToDevice, g_nf_stream));
  NF_CUDA(cudaMemcpyAsync(P->rvar, ones.data(), P->Cout * 4, cudaMemcpyHostToDevice, g_nf_stream));
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  return nf_k_shadow(P->val, P->shadow, P->arena);
}

// which: NF_P_W (logical [Cout][Cin]), NF_P_GAMMA, NF_P_BETA, NF_P_RMEAN, NF_P_RVAR, plus an nf_param_kind
static int proj_param(nf_proj* P, int which, float** dev, size_t* n) {
  const int id = which & 0xff, kind = which & 0xf00;
  if (id == NF_P_RMEAN || id == NF_P_RVAR) {
    if (kind != NF_K_VALUE) return NF_EINVAL;
    *dev = id == NF_P_RMEAN ? P->rmean : P->rvar;
    *n = P->Cout;
    return NF_OK;
  }
  float* base = kind == NF_K_VALUE ? P->val : kind == NF_K_MOMENTUM ? P->mom : kind == NF_K_GRAD ? P->grad : nullptr;
  if (!base) return NF_EINVAL;
  if (id == NF_P_W) { *dev = base + P->offW; *n = (size_t)P->Cin * P->Cout; return NF_OK; }
  if (id == NF_P_GAMMA) { *dev = base + P->offG; *n = P->Cout; return NF_OK; }
  if (id == NF_P_BETA) { *dev = base + P->offB; *n = P->Cout; return NF_OK; }
  return NF_EINVAL;
}

int nf_proj_set_param(nf_proj* P, int which, const float* host, size_t n) {
  if (!P || !host) return NF_EINVAL;
  if (!P->ws) return NF_ENOWS;
  if ((which & 0xf00) == NF_K_GRAD) return NF_EINVAL;
  float* dev; size_t cnt;
  const int rc = proj_param(P, which, &dev, &cnt);
  if (rc != NF_OK) return rc;
  if (n != cnt) return NF_EINVAL;
  std::vector<float> tmp(host, host + cnt);
  if ((which & 0xff) == NF_P_W)  // logical [Cout][Cin] -> kernel [Cin][Cout]
    for (int co = 0; co < P->Cout; ++co)
      for (int ci = 0; ci < P->Cin; ++ci) tmp[(size_t)ci * P->Cout + co] = host[(size_t)co * P->Cin + ci];
  NF_CUDA(cudaMemcpyAsync(dev, tmp.data(), cnt * 4, cudaMemcpyHostToDevice, g_nf_stream));
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  if ((which & 0xf00) == NF_K_VALUE && (which & 0xff) < NF_P_RMEAN) {
    const int r2 = nf_k_shadow(P->val, P->shadow, P->arena);
    if (r2 != NF_OK) return r2;
    NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  }
  return NF_OK;
}

int nf_proj_get_param(nf_proj* P, int which, float* host, size_t n) {
  if (!P || !host) return NF_EINVAL;
  if (!P->ws) return NF_ENOWS;
  float* dev; size_t cnt;
  const int rc = proj_param(P, which, &dev, &cnt);
  if (rc != NF_OK) return rc;
  if (n != cnt) return NF_EINVAL;
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  std::vector<float> tmp(cnt);
  NF_CUDA(cudaMemcpy(tmp.data(), dev, cnt * 4, cudaMemcpyDeviceToHost));
  if ((which & 0xff) == NF_P_W) {
    for (int co = 0; co < P->Cout; ++co)
      for (int ci = 0; ci < P->Cin; ++ci) host[(size_t)co * P->Cin + ci] = tmp[(size_t)ci * P->Cout + co];
  } else {
    memcpy(host, tmp.data(), cnt * 4);
  }
  return NF_OK;
}

}  // extern "C"

namespace {

#define PROJ_DISPATCH(dtype, CALL_F32, CALL_BF16)               \
  do {                                                          \
    if ((dtype) == NF_F32) { CALL_F32; } else { CALL_BF16; }    \
  } while (0)

int proj_conv(nf_proj* P, const void* xb, int count) {
  const size_t pix = (size_t)count * P->Ho * P->Wo;
  const size_t smem = (size_t)kPix * P->Cin * sizeof(float);
  if (smem > 48 * 1024) return NF_EUNSUPPORTED;
  const unsigned grid = blocks_for(pix, kPix);
  PROJ_DISPATCH(P->dtype,
                (proj_fwd_kernel<float><<<grid, 256, smem, g_nf_stream>>>((const float*)xb, P->val + P->offW, P->H, P->W, P->Cin, P->Cout,
                                                                        P->Ho, P->Wo, pix, 2, (float*)P->ys)),
                (proj_fwd_kernel<bf16><<<grid, 256, smem, g_nf_stream>>>((const bf16*)xb, P->shadow + P->offW, P->H, P->W, P->Cin, P->Cout,
                                                                       P->Ho, P->Wo, pix, 2, (bf16*)P->ys)));
  NF_LAUNCHED();
  return NF_OK;
}

int proj_affine(nf_proj* P, int count, void* s_out) {
  const size_t total = (size_t)count * P->Ho * P->Wo * P->Cout;
  PROJ_DISPATCH(P->dtype,
                (proj_affine_kernel<float><<<blocks_for(total, 256), 256, 0, g_nf_stream>>>((const float*)P->ys, P->Cout, P->scale, P->shift,
                                                                                         total, (float*)s_out)),
                (proj_affine_kernel<bf16><<<blocks_for(total, 256), 256, 0, g_nf_stream>>>((const bf16*)P->ys, P->Cout, P->scale, P->shift,
                                                                                        total, (bf16*)s_out)));
  NF_LAUNCHED();
  return NF_OK;
}

}  // namespace

extern "C" {

int nf_proj_forward(nf_proj* P, const void* xb, void* s_out) {
  if (!P || !xb || !s_out) return NF_EINVAL;
  if (!P->ws) return NF_ENOWS;
  if (((uintptr_t)xb | (uintptr_t)s_out) & 15) return NF_EALIGN;
  int rc = proj_conv(P, xb, P->N);
  if (rc != NF_OK) return rc;
  int nb = 0;
  const size_t pix = (size_t)P->N * P->Ho * P->Wo;
  if ((rc = nf_k_channel_sums(P->dtype, P->ys, pix, P->Cout, P->red, P->red_floats, &nb)) != NF_OK) return rc;
  if ((rc = nf_k_bn_finalize(P->red, nb, P->Cout, (double)pix, P->val + P->offG, P->val + P->offB, P->eps, P->bn_momentum, P->scale,
                             P->shift, P->mu, P->invstd, P->rmean, P->rvar)) != NF_OK)
    return rc;
  return proj_affine(P, P->N, s_out);
}

int nf_proj_forward_eval(nf_proj* P, const void* xb, int count, void* s_out) {
  if (!P || !xb || !s_out || count < 1 || count > P->N) return NF_EINVAL;
  if (!P->ws) return NF_ENOWS;
  if (((uintptr_t)xb | (uintptr_t)s_out) & 15) return NF_EALIGN;
  int rc = proj_conv(P, xb, count);
  if (rc != NF_OK) return rc;
  if ((rc = nf_k_bn_eval_coeffs(P->Cout, P->val + P->offG, P->val + P->offB, P->eps, P->rmean, P->rvar, P->scale, P->shift)) != NF_OK)
    return rc;
  return proj_affine(P, count, s_out);
}

int nf_proj_backward(nf_proj* P, const void* xb, const void* dz, float lr) {
  if (!P || !xb || !dz) return NF_EINVAL;
  if (!P->ws) return NF_ENOWS;
  if (((uintptr_t)xb | (uintptr_t)dz) & 15) return NF_EALIGN;
  const int C = P->Cout;
  const size_t pix = (size_t)P->N * P->Ho * P->Wo, total = pix * C;
  const int nb = (int)(pix < (size_t)kProjBlocks ? pix : (size_t)kProjBlocks);
  PROJ_DISPATCH(P->dtype,
                (proj_bwd_reduce_kernel<float><<<nb, 256, 0, g_nf_stream>>>((const float*)P->ys, (const float*)dz, pix, C, P->mu, P->invstd, P->red)),
                (proj_bwd_reduce_kernel<bf16><<<nb, 256, 0, g_nf_stream>>>((const bf16*)P->ys, (const bf16*)dz, pix, C, P->mu, P->invstd, P->red)));
  NF_LAUNCHED();
  int rc = nf_k_bn_bwd_finalize(P->red, nb, C, P->sdz, P->sdzx, P->grad + P->offG, P->grad + P->offB);
  if (rc != NF_OK) return rc;
  const float invM = (float)(1.0 / (double)pix);
  PROJ_DISPATCH(P->dtype,
                (proj_bwd_apply_kernel<float><<<blocks_for(total, 256), 256, 0, g_nf_stream>>>((const float*)P->ys, (const float*)dz, C, P->scale, P->mu,
                                                                                            P->invstd, P->sdz, P->sdzx, invM, total, (float*)P->dys)),
                (proj_bwd_apply_kernel<bf16><<<blocks_for(total, 256), 256, 0, g_nf_stream>>>((const bf16*)P->ys, (const bf16*)dz, C, P->scale, P->mu,
                                                                                           P->invstd, P->sdz, P->sdzx, invM, total, (bf16*)P->dys)));
  NF_LAUNCHED();
  const dim3 grid((P->Cin + 15) / 16, (C + 63) / 64, P->splits);
  PROJ_DISPATCH(P->dtype,
                (proj_wgrad_kernel<float><<<grid, 256, 0, g_nf_stream>>>((const float*)xb, (const float*)P->dys, P->H, P->W, P->Cin, C, P->Ho, P->Wo,
                                                                       pix, 2, P->splits, P->wpart)),
                (proj_wgrad_kernel<bf16><<<grid, 256, 0, g_nf_stream>>>((const bf16*)xb, (const bf16*)P->dys, P->H, P->W, P->Cin, C, P->Ho, P->Wo,
                                                                      pix, 2, P->splits, P->wpart)));
  NF_LAUNCHED();
  const size_t nw = (size_t)P->Cin * C;
  proj_sum_splits_kernel<<<blocks_for(nw, 256), 256, 0, g_nf_stream>>>(P->wpart, P->splits, nw, P->grad + P->offW);
  NF_LAUNCHED();
  return nf_k_sgd(P->val, P->mom, P->grad, P->shadow, P->arena, lr, P->momentum);
}

}  // extern "C"
