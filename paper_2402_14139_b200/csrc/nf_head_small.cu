// The linear head gamma_n of Eq. 2 with the loss of Eq. 3, forward and backward, for batches where the three products
//   logits = p Wf^T + bf,   gWf = dlogits^T p,   dp = dlogits Wf
// are too small to tile as matrix products (a few million multiply-adds: e.g. 64 samples x 64 inputs x 1000 classes).
// Such a head is pure latency, so the work is cut by CLASS SLICES instead of by samples: a CTA keeps its slice of Wf and a
// chunk of the pooled inputs p in shared memory and produces every output that depends on them.
//   1. head_logits_slice_kernel  (slice, sample chunk): logits of the slice and, per sample, the slice's share of the
//      softmax normaliser (running maximum and sum of exponentials) or of the squared error.
//   2. head_grad_slice_kernel    (slice): log-sum-exp per sample from all slices' shares, dlogits of the slice (kept in
//      shared memory only), gWf and gbf of the slice summed over the whole batch, and the slice's share of dp.
//   3. head_finish_kernel: dp = sum of the slices' shares in slice order; mean loss.
// fp32 throughout, every sum in a fixed order: results do not depend on scheduling.
#include <math.h>

#include "nf_internal.h"

namespace {

constexpr int kHsThreads = 256;
constexpr int kHsRegs = 8;  // gWf outputs per thread of the gradient kernel: KS * D <= kHsThreads * kHsRegs

struct HsPlan {
  int ok, KS, S, NC, chunks;
  size_t smem_fwd, smem_bwd, scratch_floats;
};

HsPlan hs_plan(int N, int D, int K) {
  HsPlan pl{};
  if (N < 1 || D < 1 || K < 1 || D > kHsThreads * kHsRegs) return pl;
  // Slicing by classes pays when there are many classes per sample (ImageNet-shaped heads: 64 samples x 1000 classes, where
  // one block per sample leaves most SMs idle and walks all of Wf 64 times).  With few classes and a larger batch
  // (10 or 100 classes, 128 ... 512 samples) there are too few slices and each walks the whole batch: one block per sample
  // measured faster there (0.88 vs 0.93 ms per 4-layer step at 128 samples x 10 classes, 1.21 vs 1.30 ms at 512 x 100).
  if ((long)K < 4L * N) return pl;
  int KS = (K + 47) / 48;  // about 48 slices: enough CTAs to spread the latency, few enough partial results to add up
  if (KS * D > kHsThreads * kHsRegs) KS = kHsThreads * kHsRegs / D;
  int NC = 64;
  while (NC > 1 && (size_t)NC * (D + 1) * 4 > 40000) NC >>= 1;
  if (NC > N) NC = N;
  pl.KS = KS;
  pl.S = (K + KS - 1) / KS;
  pl.NC = NC;
  pl.chunks = (N + NC - 1) / NC;
  pl.smem_fwd = ((size_t)(NC + KS) * (D + 1) + (size_t)KS * NC) * 4;
  pl.smem_bwd = pl.smem_fwd + (size_t)(2 * kHsThreads + NC) * 4;
  if (pl.smem_bwd > 96 * 1024) return pl;
  pl.scratch_floats = (size_t)pl.S * N * (D + 2);  // per slice: [N][2] softmax shares, then [N][D] shares of dp
  pl.ok = 1;
  return pl;
}

__device__ __forceinline__ int clamp_label(int lab, int K) { return lab < 0 ? 0 : lab >= K ? K - 1 : lab; }

// grid (S, chunks).  share[(s*N + n)*2 + {0,1}]: cross entropy (running max m, sum exp(l - m)); squared error (0, sum e^2)
__global__ void __launch_bounds__(kHsThreads) head_logits_slice_kernel(const float* __restrict__ p, const int32_t* __restrict__ labels,
                                                                       int N, int D, int K, int KS, int NC,
                                                                       const float* __restrict__ Wf, const float* __restrict__ bf,
                                                                       float* __restrict__ logits, float* __restrict__ share,
                                                                       int loss_kind) {
  extern __shared__ float sm[];
  const int Dp = D + 1;
  float* ps = sm;                 // [NC][D+1]
  float* ws = ps + NC * Dp;       // [KS][D+1]
  float* lg = ws + KS * Dp;       // [KS][NC]
  const int t = threadIdx.x, s = blockIdx.x;
  const int k0 = s * KS, kn = min(KS, K - k0), n0 = blockIdx.y * NC, nn = min(NC, N - n0);
  for (int i = t; i < nn * D; i += kHsThreads) ps[(i / D) * Dp + i % D] = p[(size_t)n0 * D + i];
  for (int i = t; i < kn * D; i += kHsThreads) ws[(i / D) * Dp + i % D] = Wf[(size_t)k0 * D + i];
  __syncthreads();
  for (int i = t; i < kn * nn; i += kHsThreads) {
    const int k = i / nn, n = i % nn;
    const float* w = ws + k * Dp;
    const float* x = ps + n * Dp;
    float acc = bf[k0 + k];
    for (int d = 0; d < D; ++d) acc = fmaf(w[d], x[d], acc);
    lg[k * NC + n] = acc;
    logits[(size_t)(n0 + n) * K + k0 + k] = acc;
  }
  __syncthreads();
  if (t < nn) {
    float a, b;
    if (loss_kind == 1) {
      const int lab = clamp_label(labels[n0 + t], K);
      a = 0.f;
      b = 0.f;
      for (int k = 0; k < kn; ++k) {
        const float e = lg[k * NC + t] - (k0 + k == lab ? 1.f : 0.f);
        b = fmaf(e, e, b);
      }
    } else {
      a = -INFINITY;
      for (int k = 0; k < kn; ++k) a = fmaxf(a, lg[k * NC + t]);
      b = 0.f;
      for (int k = 0; k < kn; ++k) b += expf(lg[k * NC + t] - a);
    }
    share[((size_t)s * N + n0 + t) * 2] = a;
    share[((size_t)s * N + n0 + t) * 2 + 1] = b;
  }
}

// grid S.  dps[(s*N + n)*D + d]: the slice's share of dp.  lossn[n] is written by slice 0 (squared error) or by the slice that
// holds the sample's label (cross entropy).
__global__ void __launch_bounds__(kHsThreads) head_grad_slice_kernel(const float* __restrict__ p, const int32_t* __restrict__ labels,
                                                                     int N, int D, int K, int KS, int NC, int S,
                                                                     const float* __restrict__ Wf, const float* __restrict__ logits,
                                                                     const float* __restrict__ share, float* __restrict__ dps,
                                                                     float* __restrict__ gWf, float* __restrict__ gbf,
                                                                     float* __restrict__ lossn, int32_t* __restrict__ status,
                                                                     int loss_kind, int n_scale) {
  extern __shared__ float sm[];
  const int Dp = D + 1;
  float* ps = sm;                 // [NC][D+1]
  float* ws = ps + NC * Dp;       // [KS][D+1]
  float* dl = ws + KS * Dp;       // [KS][NC]
  float* cm = dl + KS * NC;       // [256] partial maxima / [256] partial sums while the shares are combined
  float* cs = cm + kHsThreads;
  float* lse = cs + kHsThreads;   // [NC] log-sum-exp (cross entropy) or total squared error (squared-error loss)
  const int t = threadIdx.x, s = blockIdx.x;
  const int k0 = s * KS, kn = min(KS, K - k0);
  float gacc[kHsRegs];
#pragma unroll
  for (int r = 0; r < kHsRegs; ++r) gacc[r] = 0.f;
  float gb = 0.f;
  for (int i = t; i < kn * D; i += kHsThreads) ws[(i / D) * Dp + i % D] = Wf[(size_t)k0 * D + i];
  const float invN = 1.f / (float)n_scale;
  const float mse_scale = 2.f / ((float)n_scale * (float)K);
  const int parts = kHsThreads / NC;  // threads that share one sample while the slices' shares are combined
  for (int n0 = 0; n0 < N; n0 += NC) {
    const int nn = min(NC, N - n0);
    __syncthreads();  // the previous chunk is done with ps, dl and lse
    for (int i = t; i < nn * D; i += kHsThreads) ps[(i / D) * Dp + i % D] = p[(size_t)n0 * D + i];
    {
      // thread (n, part) folds the slices part, part + parts, ... in slice order; the parts are folded in part order
      const int n = t % NC, part = t / NC;
      float m = -INFINITY, q = 0.f;
      if (n < nn && part < parts) {
        for (int j = part; j < S; j += parts) {
          const float mj = share[((size_t)j * N + n0 + n) * 2], qj = share[((size_t)j * N + n0 + n) * 2 + 1];
          if (loss_kind == 1) {
            q += qj;
          } else {
            const float mm = fmaxf(m, mj);
            q = q * expf(m - mm) + qj * expf(mj - mm);
            m = mm;
          }
        }
      }
      cm[t] = m;
      cs[t] = q;
    }
    __syncthreads();
    if (t < nn) {
      float m = cm[t], q = cs[t];
      for (int part = 1; part < parts; ++part) {
        const float mj = cm[part * NC + t], qj = cs[part * NC + t];
        if (loss_kind == 1) {
          q += qj;
        } else if (mj > -INFINITY) {
          const float mm = fmaxf(m, mj);
          q = q * expf(m - mm) + qj * expf(mj - mm);
          m = mm;
        }
      }
      lse[t] = loss_kind == 1 ? q : m + logf(q);
      const int lab = labels[n0 + t];
      if (s == 0) {
        if (lab < 0 || lab >= K) atomicOr(status, NF_ELABEL);
        if (loss_kind == 1) lossn[n0 + t] = q / (float)K;
      }
    }
    __syncthreads();
    for (int i = t; i < kn * nn; i += kHsThreads) {
      const int k = i / nn, n = i % nn;
      const float l = logits[(size_t)(n0 + n) * K + k0 + k];
      const int lab = clamp_label(labels[n0 + n], K);
      const float hit = k0 + k == lab ? 1.f : 0.f;
      float g;
      if (loss_kind == 1) {
        g = (l - hit) * mse_scale;
      } else {
        g = (expf(l - lse[n]) - hit) * invN;
        if (hit != 0.f) lossn[n0 + n] = lse[n] - l;
      }
      dl[k * NC + n] = g;
    }
    __syncthreads();
    // gWf[k][d] += sum over the chunk's samples (ascending) of dlogits[n][k] * p[n][d]
#pragma unroll
    for (int r = 0; r < kHsRegs; ++r) {
      const int i = t + kHsThreads * r;
      if (i < kn * D) {
        const int k = i / D, d = i % D;
        float a = gacc[r];
        for (int n = 0; n < nn; ++n) a = fmaf(dl[k * NC + n], ps[n * Dp + d], a);
        gacc[r] = a;
      }
    }
    if (t < kn)
      for (int n = 0; n < nn; ++n) gb += dl[t * NC + n];
    // the slice's share of dp[n][d] = sum over its classes (ascending) of dlogits[n][k] * Wf[k][d]
    for (int i = t; i < nn * D; i += kHsThreads) {
      const int n = i / D, d = i % D;
      float a = 0.f;
      for (int k = 0; k < kn; ++k) a = fmaf(dl[k * NC + n], ws[k * Dp + d], a);
      dps[((size_t)s * N + n0) * D + i] = a;
    }
  }
#pragma unroll
  for (int r = 0; r < kHsRegs; ++r) {
    const int i = t + kHsThreads * r;
    if (i < kn * D) gWf[(size_t)k0 * D + i] = gacc[r];
  }
  if (t < kn) gbf[k0 + t] = gb;
}

// dp[i] = sum over the slices (ascending) of their shares; block 0 also reduces the mean loss
__global__ void __launch_bounds__(kHsThreads) head_finish_kernel(const float* __restrict__ dps, int S, size_t ND, float* __restrict__ dp,
                                                                 const float* __restrict__ lossn, int N, int n_scale,
                                                                 float* __restrict__ loss_out, int32_t* __restrict__ status) {
  const size_t i = (size_t)blockIdx.x * kHsThreads + threadIdx.x;
  if (i < ND) {
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;  // four interleaved chains over the slices, combined in a fixed order
    int j = 0;
    for (; j + 3 < S; j += 4) {
      a0 += dps[(size_t)j * ND + i];
      a1 += dps[(size_t)(j + 1) * ND + i];
      a2 += dps[(size_t)(j + 2) * ND + i];
      a3 += dps[(size_t)(j + 3) * ND + i];
    }
    for (; j < S; ++j) a0 += dps[(size_t)j * ND + i];
    dp[i] = (a0 + a1) + (a2 + a3);
  }
  if (blockIdx.x == 0) {
    __shared__ double red[kHsThreads];
    double a = 0.0;
    for (int n = threadIdx.x; n < N; n += kHsThreads) a += (double)lossn[n];
    red[threadIdx.x] = a;
    __syncthreads();
    for (int o = kHsThreads / 2; o > 0; o >>= 1) {
      if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
      __syncthreads();
    }
    if (threadIdx.x == 0) {
      const float L = (float)(red[0] / (double)n_scale);
      *loss_out = L;
      if (!isfinite(L)) atomicOr(status, NF_ENONFINITE);
    }
  }
}

// the two slice kernels may use up to 96 KB of dynamic shared memory: allowed once per device
int allow_smem() {
  static bool done[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
  if (done[dev]) return NF_OK;
  NF_CUDA(cudaFuncSetAttribute(head_logits_slice_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024));
  NF_CUDA(cudaFuncSetAttribute(head_grad_slice_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024));
  done[dev] = true;
  return NF_OK;
}

}  // namespace

size_t nf_head_small_scratch_floats(int N, int D, int K) {
  const HsPlan pl = hs_plan(N, D, K);
  return pl.ok ? pl.scratch_floats : 0;
}

int nf_head_small_step(const float* p, const int32_t* labels, int N, int D, int K, const float* Wf, const float* bf, float* logits,
                       float* dp, float* lossn, int32_t* status, int loss_kind, float* gWf, float* gbf, float* loss_out,
                       float* scratch, size_t scratch_floats, int n_scale) {
  const HsPlan pl = hs_plan(N, D, K);
  if (!pl.ok) return NF_EUNSUPPORTED;
  if (pl.scratch_floats > scratch_floats) return NF_ENOWS;
  float* share = scratch;                       // [S][N][2]
  float* dps = scratch + (size_t)pl.S * N * 2;  // [S][N][D]
  const int rc = allow_smem();
  if (rc != NF_OK) return rc;
  head_logits_slice_kernel<<<dim3(pl.S, pl.chunks), kHsThreads, pl.smem_fwd, g_nf_stream>>>(p, labels, N, D, K, pl.KS, pl.NC, Wf, bf,
                                                                                             logits, share, loss_kind);
  NF_LAUNCHED();
  head_grad_slice_kernel<<<pl.S, kHsThreads, pl.smem_bwd, g_nf_stream>>>(p, labels, N, D, K, pl.KS, pl.NC, pl.S, Wf, logits, share, dps,
                                                                         gWf, gbf, lossn, status, loss_kind, n_scale);
  NF_LAUNCHED();
  const size_t ND = (size_t)N * D;
  head_finish_kernel<<<(unsigned)((ND + kHsThreads - 1) / kHsThreads), kHsThreads, 0, g_nf_stream>>>(dps, pl.S, ND, dp, lossn, N, n_scale,
                                                                                                    loss_out, status);
  NF_LAUNCHED();
  return NF_OK;
}
