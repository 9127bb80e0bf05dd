// Memory-bound kernels of the local-layer step: BatchNorm statistics / apply / backward, pooling,
// the linear + softmax cross-entropy head, momentum SGD and the cache gather.  Storage fp32 or
// bf16, arithmetic fp32, cross-block sums finished in fp64 in a fixed order (deterministic).
#include <algorithm>
#include "nf_internal.h"
#include "nf_ldst.cuh"

namespace {

__host__ __device__ inline int pow2ceil_cap256(int c) {
  int l = 1;
  while (l < c && l < 256) l <<= 1;
  return l;
}

// dz at full-resolution pixel p = ((n*Ho)+i)*Wo+j, channel c: gradient that reaches the BatchNorm
// output through ReLU and the optional 2x2 max-pool (first maximum in scan order wins).
template <typename T>
__device__ __forceinline__ float dz_at(const T* __restrict__ y, const T* __restrict__ da, size_t p, int c, int C,
                                       int Ho, int Wo, int pool, float sc, float sh, const T* __restrict__ skip = nullptr) {
  const float z = fmaf(ldf(y, p * C + c), sc, sh) + (skip ? ldf(skip, p * C + c) : 0.f);
  if (!(z > 0.f)) return 0.f;
  if (!pool) return ldf(da, p * C + c);
  const int j = (int)(p % Wo), i = (int)((p / Wo) % Ho);
  const size_t n = p / ((size_t)Wo * Ho);
  const int i0 = i & ~1, j0 = j & ~1;
  float best = -1.f;
  int arg = 0;
#pragma unroll
  for (int d = 0; d < 4; ++d) {
    const size_t q = ((n * Ho + i0 + (d >> 1)) * Wo + j0 + (d & 1)) * C + c;
    const float r = rnd<T>(fmaxf(fmaf(ldf(y, q), sc, sh) + (skip ? ldf(skip, q) : 0.f), 0.f));
    if (r > best) { best = r; arg = d; }
  }
  if (arg != (i - i0) * 2 + (j - j0)) return 0.f;
  return ldf(da, ((n * (Ho / 2) + i / 2) * (Wo / 2) + j / 2) * C + c);
}

struct StatsFn {  // (v, v^2) of a stored tensor
  template <typename T>
  __device__ __forceinline__ void operator()(const T* src, const T*, size_t p, int c, int C, float& a, float& b) const {
    const float v = ldf(src, p * C + c);
    a = v;
    b = v * v;
  }
};

struct BnBwdFn {  // (dz, dz*xhat)
  int Ho, Wo, pool;
  const float *scale, *shift, *mu, *invstd;
  const void* skip;  // identity shortcut added before the ReLU, or NULL
  template <typename T>
  __device__ __forceinline__ void operator()(const T* y, const T* da, size_t p, int c, int C, float& a, float& b) const {
    const float dz = dz_at(y, da, p, c, C, Ho, Wo, pool, scale[c], shift[c], (const T*)skip);
    a = dz;
    b = dz * (ldf(y, p * C + c) - mu[c]) * invstd[c];
  }
};

// red[(block*2 + k)*C + c] = sum over the block's pixel range of value k at channel c
template <typename T, typename Fn>
__global__ void __launch_bounds__(256) channel_reduce_kernel(const T* __restrict__ s0, const T* __restrict__ s1, size_t P,
                                                             int C, Fn fn, float* __restrict__ red) {
  __shared__ float sm[2][256];
  const int lanes = pow2ceil_cap256(C), planes = 256 / lanes;
  const int lc = threadIdx.x % lanes, pl = threadIdx.x / lanes;
  const size_t p0 = P * blockIdx.x / gridDim.x, p1 = P * (blockIdx.x + 1) / gridDim.x;
  for (int c0 = 0; c0 < C; c0 += lanes) {
    const int c = c0 + lc;
    float a = 0.f, b = 0.f;
    if (c < C)
      for (size_t p = p0 + pl; p < p1; p += planes) {
        float u, v;
        fn(s0, s1, p, c, C, u, v);
        a += u;
        b += v;
      }
    sm[0][threadIdx.x] = a;
    sm[1][threadIdx.x] = b;
    __syncthreads();
    if (pl == 0 && c < C) {
      float ta = 0.f, tb = 0.f;
      for (int q = 0; q < planes; ++q) {
        ta += sm[0][q * lanes + lc];
        tb += sm[1][q * lanes + lc];
      }
      red[((size_t)blockIdx.x * 2 + 0) * C + c] = ta;
      red[((size_t)blockIdx.x * 2 + 1) * C + c] = tb;
    }
    __syncthreads();
  }
}


// Sums the per-block partials of 32 consecutive channels: block (32 channels x 32 lanes over the partials),
// fp64, fixed order.  Returns the two totals to the threads with threadIdx.y == 0.
__device__ __forceinline__ void reduce_partials32(const float* __restrict__ red, int nb, int C, double& S, double& Q) {
  __shared__ double sm[2][32][33];
  const int c = blockIdx.x * 32 + threadIdx.x;
  double a = 0.0, b = 0.0;
  if (c < C) {
    int k = threadIdx.y;
    for (; k + 7 * 32 < nb; k += 8 * 32) {  // eight independent pairs of loads in flight, added in index order
      float u[8], v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        u[j] = red[((size_t)(k + 32 * j) * 2 + 0) * C + c];
        v[j] = red[((size_t)(k + 32 * j) * 2 + 1) * C + c];
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        a += (double)u[j];
        b += (double)v[j];
      }
    }
    for (; k < nb; k += 32) {
      a += (double)red[((size_t)k * 2 + 0) * C + c];
      b += (double)red[((size_t)k * 2 + 1) * C + c];
    }
  }
  sm[0][threadIdx.y][threadIdx.x] = a;
  sm[1][threadIdx.y][threadIdx.x] = b;
  __syncthreads();
  S = 0.0;
  Q = 0.0;
  if (threadIdx.y == 0)
    for (int k = 0; k < 32; ++k) {
      S += sm[0][k][threadIdx.x];
      Q += sm[1][k][threadIdx.x];
    }
}

__global__ void bn_finalize_kernel(const float* __restrict__ red, int nb, int C, double M, const float* __restrict__ gamma,
                                   const float* __restrict__ beta, float eps, float bnm, float* scale, float* shift,
                                   float* mu, float* invstd, float* rmean, float* rvar) {
  double S, Q;
  reduce_partials32(red, nb, C, S, Q);
  const int c = blockIdx.x * 32 + threadIdx.x;
  if (c >= C || threadIdx.y != 0) return;
  const double m = S / M;
  double v = Q / M - m * m;
  if (v < 0.0) v = 0.0;
  const double is = 1.0 / sqrt(v + (double)eps);
  const float sc = (float)((double)gamma[c] * is);
  scale[c] = sc;
  shift[c] = (float)((double)beta[c] - m * (double)gamma[c] * is);
  mu[c] = (float)m;
  invstd[c] = (float)is;
  if (rmean) {
    rmean[c] = (float)((1.0 - bnm) * (double)rmean[c] + (double)bnm * m);
    const double unb = M > 1.0 ? v * M / (M - 1.0) : v;
    rvar[c] = (float)((1.0 - bnm) * (double)rvar[c] + (double)bnm * unb);
  }
}

// Data-parallel BatchNorm: a rank turns its per-block partials into per-channel totals (fp64, [2][C]) that the
// ranks add up; the statistics and the backward sums are then finished from the totals of the whole batch.
__global__ void partial_totals_kernel(const float* __restrict__ red, int nb, int C, double* __restrict__ tot) {
  double S, Q;
  reduce_partials32(red, nb, C, S, Q);
  const int c = blockIdx.x * 32 + threadIdx.x;
  if (c >= C || threadIdx.y != 0) return;
  tot[c] = S;
  tot[C + c] = Q;
}

__global__ void bn_finalize_tot_kernel(const double* __restrict__ tot, int C, double M, const float* __restrict__ gamma,
                                       const float* __restrict__ beta, float eps, float bnm, float* scale, float* shift, float* mu,
                                       float* invstd, float* rmean, float* rvar) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  const double m = tot[c] / M;
  double v = tot[C + c] / M - m * m;
  if (v < 0.0) v = 0.0;
  const double is = 1.0 / sqrt(v + (double)eps);
  scale[c] = (float)((double)gamma[c] * is);
  shift[c] = (float)((double)beta[c] - m * (double)gamma[c] * is);
  mu[c] = (float)m;
  invstd[c] = (float)is;
  rmean[c] = (float)((1.0 - bnm) * (double)rmean[c] + (double)bnm * m);
  const double unb = M > 1.0 ? v * M / (M - 1.0) : v;
  rvar[c] = (float)((1.0 - bnm) * (double)rvar[c] + (double)bnm * unb);
}

// the gradients of gamma and beta are divided by the number of ranks: the sum over ranks that follows restores them
__global__ void bn_bwd_finalize_tot_kernel(const double* __restrict__ tot, int C, double inv_world, float* sdz, float* sdzx, float* gg,
                                           float* gb) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  sdz[c] = (float)tot[c];
  sdzx[c] = (float)tot[C + c];
  gb[c] = (float)(tot[c] * inv_world);
  gg[c] = (float)(tot[C + c] * inv_world);
}

__global__ void bn_eval_coeffs_kernel(int C, const float* gamma, const float* beta, float eps, const float* rmean,
                                      const float* rvar, float* scale, float* shift) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  const double is = 1.0 / sqrt((double)rvar[c] + (double)eps);
  scale[c] = (float)((double)gamma[c] * is);
  shift[c] = (float)((double)beta[c] - (double)rmean[c] * (double)gamma[c] * is);
}

// out[n,ia,ja,c] = max over the pool window (or the single pixel) of ReLU(y*scale+shift)
template <typename T>
__global__ void bn_apply_kernel(const T* __restrict__ y, int Ho, int Wo, int C, int pool, const float* __restrict__ scale,
                                const float* __restrict__ shift, size_t total, T* __restrict__ out, const T* __restrict__ skip) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int c = (int)(e % C);
  const size_t q = e / C;
  const float sc = scale[c], sh = shift[c];
  if (!pool) {
    stf(out, e, fmaxf(fmaf(ldf(y, e), sc, sh) + (skip ? ldf(skip, e) : 0.f), 0.f));
    return;
  }
  const int Wa = Wo / 2, Ha = Ho / 2;
  const int ja = (int)(q % Wa), ia = (int)((q / Wa) % Ha);
  const size_t n = q / ((size_t)Wa * Ha);
  float best = 0.f;
#pragma unroll
  for (int d = 0; d < 4; ++d) {
    const size_t src = ((n * Ho + 2 * ia + (d >> 1)) * Wo + 2 * ja + (d & 1)) * C + c;
    best = fmaxf(best, fmaf(ldf(y, src), sc, sh) + (skip ? ldf(skip, src) : 0.f));
  }
  stf(out, e, best);
}

__device__ __forceinline__ void bin_range(int u, int H, int& lo, int& hi) {
  lo = (u * H) / 2;
  hi = ((u + 1) * H + 1) / 2;
}

// p[n][f*4 + u*2 + v] = mean of h over bin (u,v);  one block per (n, bin)
// the same for bins of at most 16 pixels: one thread per output p[n][f*4 + bin] (consecutive threads = consecutive channels)
template <typename T>
__global__ void avgpool_small_kernel(const T* __restrict__ h, int Ha, int Wa, int F, size_t total, float* __restrict__ p) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int f = (int)(e % F), bin = (int)((e / F) % 4);
  const size_t n = e / ((size_t)4 * F);
  int i0, i1, j0, j1;
  bin_range(bin / 2, Ha, i0, i1);
  bin_range(bin % 2, Wa, j0, j1);
  float a = 0.f;
  for (int i = i0; i < i1; ++i)
    for (int j = j0; j < j1; ++j) a += ldf(h, ((n * Ha + i) * Wa + j) * F + f);
  p[n * 4 * F + (size_t)f * 4 + bin] = a / (float)((i1 - i0) * (j1 - j0));
}

template <typename T>
__global__ void __launch_bounds__(256) avgpool_kernel(const T* __restrict__ h, int Ha, int Wa, int F, float* __restrict__ p) {
  __shared__ float sm[256];
  const int n = blockIdx.x / 4, bin = blockIdx.x % 4, u = bin / 2, v = bin % 2;
  int i0, i1, j0, j1;
  bin_range(u, Ha, i0, i1);
  bin_range(v, Wa, j0, j1);
  const int bw = j1 - j0, cnt = (i1 - i0) * bw;
  const int lanes = pow2ceil_cap256(F), planes = 256 / lanes;
  const int lf = threadIdx.x % lanes, pl = threadIdx.x / lanes;
  for (int f0 = 0; f0 < F; f0 += lanes) {
    const int f = f0 + lf;
    float a = 0.f;
    if (f < F)
      for (int k = pl; k < cnt; k += planes) {
        const int i = i0 + k / bw, j = j0 + k % bw;
        a += ldf(h, (((size_t)n * Ha + i) * Wa + j) * F + f);
      }
    sm[threadIdx.x] = a;
    __syncthreads();
    if (pl == 0 && f < F) {
      float t = 0.f;
      for (int q = 0; q < planes; ++q) t += sm[q * lanes + lf];
      p[(size_t)n * 4 * F + f * 4 + bin] = t / (float)cnt;
    }
    __syncthreads();
  }
}

// Max-pool down-sampling: p[n][f*4 + bin] = max of h over bin (u,v), parg = position i*Wa+j of the FIRST maximum in
// row-major order; one block per (n, bin).  A thread scans its pixels in increasing order and keeps the first
// maximum; the lanes of a filter are then combined preferring the larger value, the smaller position on ties.
template <typename T>
__global__ void __launch_bounds__(256) auxmax_kernel(const T* __restrict__ h, int Ha, int Wa, int F, float* __restrict__ p,
                                                     int32_t* __restrict__ parg) {
  __shared__ float sv[256];
  __shared__ int si[256];
  const int n = blockIdx.x / 4, bin = blockIdx.x % 4, u = bin / 2, v = bin % 2;
  int i0, i1, j0, j1;
  bin_range(u, Ha, i0, i1);
  bin_range(v, Wa, j0, j1);
  const int bw = j1 - j0, cnt = (i1 - i0) * bw;
  const int lanes = pow2ceil_cap256(F), planes = 256 / lanes;
  const int lf = threadIdx.x % lanes, pl = threadIdx.x / lanes;
  for (int f0 = 0; f0 < F; f0 += lanes) {
    const int f = f0 + lf;
    float best = -INFINITY;
    int at = 0x7fffffff;
    if (f < F)
      for (int k = pl; k < cnt; k += planes) {
        const int i = i0 + k / bw, j = j0 + k % bw;
        const float t = ldf(h, (((size_t)n * Ha + i) * Wa + j) * F + f);
        if (t > best) { best = t; at = i * Wa + j; }
      }
    sv[threadIdx.x] = best;
    si[threadIdx.x] = at;
    __syncthreads();
    if (pl == 0 && f < F) {
      float b = sv[lf];
      int a = si[lf];
      for (int q = 1; q < planes; ++q) {
        const float t = sv[q * lanes + lf];
        const int ti = si[q * lanes + lf];
        if (t > b || (t == b && ti < a)) { b = t; a = ti; }
      }
      p[(size_t)n * 4 * F + f * 4 + bin] = b;
      parg[(size_t)n * 4 * F + f * 4 + bin] = a;
    }
    __syncthreads();
  }
}

// dh[n,i,j,f] = 1[h>0] * sum over the bins whose maximum sits at (i,j) of dp[n][f*4+bin]
template <typename T>
__global__ void dh_max_kernel(const T* __restrict__ h, const float* __restrict__ dp, const int32_t* __restrict__ parg, int Ha, int Wa,
                              int F, size_t total, T* __restrict__ dh) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int f = (int)(e % F);
  const size_t q = e / F;
  const int j = (int)(q % Wa), i = (int)((q / Wa) % Ha);
  const size_t n = q / ((size_t)Wa * Ha);
  float g = 0.f;
  if (ldf(h, e) > 0.f) {
    const int pos = i * Wa + j;
#pragma unroll
    for (int b = 0; b < 4; ++b)
      if (parg[n * 4 * F + f * 4 + b] == pos) g += dp[n * 4 * F + f * 4 + b];
  }
  stf(dh, e, g);
}

__device__ __forceinline__ float block_reduce(float v, float* sm, bool is_max) {
  const int t = threadIdx.x;
  sm[t] = v;
  __syncthreads();
  for (int s = blockDim.x / 2; s > 0; s >>= 1) {
    if (t < s) sm[t] = is_max ? fmaxf(sm[t], sm[t + s]) : sm[t] + sm[t + s];
    __syncthreads();
  }
  const float r = sm[0];
  __syncthreads();
  return r;
}

// one block per sample: logits, softmax cross-entropy, dlogits = (softmax-onehot)/N, dp = dlogits * Wf
__global__ void __launch_bounds__(256) fc_ce_kernel(const float* __restrict__ p, const int32_t* __restrict__ labels, int N,
                                                    int D, int K, const float* __restrict__ Wf, const float* __restrict__ bf,
                                                    float* __restrict__ logits, float* __restrict__ dlogits,
                                                    float* __restrict__ dp, float* __restrict__ lossn, int32_t* status,
                                                    int loss_kind, int n_scale) {
  extern __shared__ float dyn[];
  float* ps = dyn;          // [D]
  float* ls = dyn + D;      // [K]
  __shared__ float red[256];
  const int n = blockIdx.x, t = threadIdx.x;
  for (int d = t; d < D; d += 256) ps[d] = p[(size_t)n * D + d];
  __syncthreads();
  float mx = -INFINITY;
  for (int k = t; k < K; k += 256) {
    float s = bf[k];
    const float* w = Wf + (size_t)k * D;
    for (int d = 0; d < D; ++d) s = fmaf(w[d], ps[d], s);
    ls[k] = s;
    logits[(size_t)n * K + k] = s;
    mx = fmaxf(mx, s);
  }
  mx = block_reduce(mx, red, true);
  int lab = labels[n];
  if (lab < 0 || lab >= K) {
    if (t == 0) atomicOr(status, NF_ELABEL);
    lab = lab < 0 ? 0 : K - 1;
  }
  if (loss_kind == 1) {
    // mean squared error against the one-hot target: lossn = sum_k e^2 / K, dlogits = 2 e / (N K)
    float se = 0.f;
    const float sc = 2.f / ((float)n_scale * (float)K);
    for (int k = t; k < K; k += 256) {
      const float e = ls[k] - (k == lab ? 1.f : 0.f);
      se = fmaf(e, e, se);
      ls[k] = e * sc;
      dlogits[(size_t)n * K + k] = e * sc;
    }
    se = block_reduce(se, red, false);
    if (t == 0) lossn[n] = se / (float)K;
  } else {
    float se = 0.f;
    for (int k = t; k < K; k += 256) se += expf(ls[k] - mx);
    se = block_reduce(se, red, false);
    const float lse = mx + logf(se);
    if (t == 0) lossn[n] = lse - ls[lab];
    const float invN = 1.f / (float)n_scale;
    for (int k = t; k < K; k += 256) {
      const float g = (expf(ls[k] - lse) - (k == lab ? 1.f : 0.f)) * invN;
      ls[k] = g;
      dlogits[(size_t)n * K + k] = g;
    }
  }
  __syncthreads();
  // dp[d] = sum_k g[k] Wf[k][d]: the classes are cut into G contiguous ranges (G = 256 / D lanes per d when D <= 128),
  // every range is summed in index order and the G range sums are added in range order
  const int G = D <= 128 ? 256 / D : 1;
  if (G > 1) {
    const int d = t % D, kg = t / D;
    float s = 0.f;
    if (kg < G) {
      const int per = (K + G - 1) / G, k0 = kg * per, k1 = min(K, k0 + per);
      int k = k0;
      for (; k + 3 < k1; k += 4) {
        const float w0 = Wf[(size_t)k * D + d], w1 = Wf[(size_t)(k + 1) * D + d], w2 = Wf[(size_t)(k + 2) * D + d],
                    w3 = Wf[(size_t)(k + 3) * D + d];
        s = fmaf(ls[k], w0, s);
        s = fmaf(ls[k + 1], w1, s);
        s = fmaf(ls[k + 2], w2, s);
        s = fmaf(ls[k + 3], w3, s);
      }
      for (; k < k1; ++k) s = fmaf(ls[k], Wf[(size_t)k * D + d], s);
    }
    red[t] = s;
    __syncthreads();
    if (t < D) {
      float tot = 0.f;
      for (int g = 0; g < G; ++g) tot += red[g * D + t];
      dp[(size_t)n * D + t] = tot;
    }
  } else {
    for (int d = t; d < D; d += 256) {
      float s = 0.f;
      for (int k = 0; k < K; ++k) s = fmaf(ls[k], Wf[(size_t)k * D + d], s);
      dp[(size_t)n * D + d] = s;
    }
  }
}


// one block per sample: logits = Wf p + bf (optionally stored) and the class = first arg-max
__global__ void __launch_bounds__(256) fc_predict_kernel(const float* __restrict__ p, int D, int K, const float* __restrict__ Wf,
                                                         const float* __restrict__ bf, float* __restrict__ logits,
                                                         int32_t* __restrict__ pred) {
  extern __shared__ float dyn[];
  float* ps = dyn;
  __shared__ float bv[256];
  __shared__ int bi[256];
  const int n = blockIdx.x, t = threadIdx.x;
  for (int d = t; d < D; d += 256) ps[d] = p[(size_t)n * D + d];
  __syncthreads();
  float best = -INFINITY;
  int arg = 0x7fffffff;
  for (int k = t; k < K; k += 256) {
    float s = bf[k];
    const float* w = Wf + (size_t)k * D;
    for (int d = 0; d < D; ++d) s = fmaf(w[d], ps[d], s);
    if (logits) logits[(size_t)n * K + k] = s;
    if (s > best) { best = s; arg = k; }   // k ascending within a thread: keeps the first maximum
  }
  bv[t] = best;
  bi[t] = arg;
  __syncthreads();
  for (int s2 = 128; s2 > 0; s2 >>= 1) {
    if (t < s2 && (bv[t + s2] > bv[t] || (bv[t + s2] == bv[t] && bi[t + s2] < bi[t]))) {
      bv[t] = bv[t + s2];
      bi[t] = bi[t + s2];
    }
    __syncthreads();
  }
  if (t == 0) pred[n] = bi[0];
}

// one block per class k: gWf[k][:] = sum_n dlogits[n][k] p[n][:], gbf[k]; block 0 also reduces the loss
__global__ void __launch_bounds__(256) fc_wgrad_kernel(const float* __restrict__ p, const float* __restrict__ dl,
                                                       const float* __restrict__ lossn, int N, int D, int K,
                                                       float* __restrict__ gWf, float* __restrict__ gbf,
                                                       float* __restrict__ loss_out, int32_t* status, int n_scale) {
  // Sums over the batch run as four interleaved chains (samples n % 4) that are combined in a fixed order, and the
  // two scalar sums are spread over a warp: the serial chains of one load per sample were pure latency.
  const int k = blockIdx.x, t = threadIdx.x;
  for (int d = t; d < D; d += 256) {
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    int n = 0;
    for (; n + 3 < N; n += 4) {
      s0 = fmaf(dl[(size_t)n * K + k], p[(size_t)n * D + d], s0);
      s1 = fmaf(dl[(size_t)(n + 1) * K + k], p[(size_t)(n + 1) * D + d], s1);
      s2 = fmaf(dl[(size_t)(n + 2) * K + k], p[(size_t)(n + 2) * D + d], s2);
      s3 = fmaf(dl[(size_t)(n + 3) * K + k], p[(size_t)(n + 3) * D + d], s3);
    }
    for (; n < N; ++n) s0 = fmaf(dl[(size_t)n * K + k], p[(size_t)n * D + d], s0);
    gWf[(size_t)k * D + d] = (s0 + s1) + (s2 + s3);
  }
  const int warp = t >> 5, lane = t & 31;
  if (warp == 7) {  // gbf[k]: lane sums over n = lane, lane + 32, ..., then a fixed butterfly
    float s = 0.f;
    for (int n = lane; n < N; n += 32) s += dl[(size_t)n * K + k];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) gbf[k] = s;
  }
  if (k == 0 && warp == 6) {
    double s = 0.0;
    for (int n = lane; n < N; n += 32) s += (double)lossn[n];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) {
      const float L = (float)(s / (double)n_scale);
      *loss_out = L;
      if (!isfinite(L)) atomicOr(status, NF_ENONFINITE);
    }
  }
}

// dh[n,i,j,f] = 1[h>0] * sum over bins containing (i,j) of dp[n][f*4+bin] / |bin|
template <typename T>
__global__ void dh_kernel(const T* __restrict__ h, const float* __restrict__ dp, int Ha, int Wa, int F, size_t total,
                          T* __restrict__ dh) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int f = (int)(e % F);
  const size_t q = e / F;
  const int j = (int)(q % Wa), i = (int)((q / Wa) % Ha);
  const size_t n = q / ((size_t)Wa * Ha);
  float g = 0.f;
  if (ldf(h, e) > 0.f) {
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      int i0, i1;
      bin_range(u, Ha, i0, i1);
      if (i < i0 || i >= i1) continue;
#pragma unroll
      for (int v = 0; v < 2; ++v) {
        int j0, j1;
        bin_range(v, Wa, j0, j1);
        if (j < j0 || j >= j1) continue;
        g += dp[n * 4 * F + f * 4 + u * 2 + v] / (float)((i1 - i0) * (j1 - j0));
      }
    }
  }
  stf(dh, e, g);
}

__global__ void sum_partials_kernel(const float* __restrict__ red, int nb, int C, int which, float* __restrict__ out) {
  double S, Q;
  reduce_partials32(red, nb, C, S, Q);
  const int c = blockIdx.x * 32 + threadIdx.x;
  if (c >= C || threadIdx.y != 0) return;
  out[c] = (float)(which ? Q : S);
}

__global__ void bn_bwd_finalize_kernel(const float* __restrict__ red, int nb, int C, float* sdz, float* sdzx, float* gg,
                                       float* gb) {
  double a, b;
  reduce_partials32(red, nb, C, a, b);
  const int c = blockIdx.x * 32 + threadIdx.x;
  if (c >= C || threadIdx.y != 0) return;
  sdz[c] = (float)a;
  sdzx[c] = (float)b;
  gb[c] = (float)a;
  gg[c] = (float)b;
}

// dy = gamma*invstd * (dz - sum(dz)/M - xhat * sum(dz*xhat)/M)
template <typename T>
__global__ void bn_bwd_apply_kernel(const T* __restrict__ y, const T* __restrict__ da, int Ho, int Wo, int C, int pool,
                                    const float* __restrict__ scale, const float* __restrict__ shift,
                                    const float* __restrict__ mu, const float* __restrict__ invstd,
                                    const float* __restrict__ sdz, const float* __restrict__ sdzx, float invM,
                                    size_t total, T* __restrict__ dy, const T* __restrict__ skip) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int c = (int)(e % C);
  const size_t p = e / C;
  const float dz = dz_at(y, da, p, c, C, Ho, Wo, pool, scale[c], shift[c], skip);
  const float xh = (ldf(y, e) - mu[c]) * invstd[c];
  stf(dy, e, scale[c] * (dz - sdz[c] * invM - xh * sdzx[c] * invM));
}

// dz = da * 1[BN(y) + skip > 0], routed through the optional max-pool: the gradient at the layer's BatchNorm output, which is
// also the gradient at a trainable shortcut added there
template <typename T>
__global__ void write_dz_kernel(const T* __restrict__ y, const T* __restrict__ da, int Ho, int Wo, int C, int pool,
                                const float* __restrict__ scale, const float* __restrict__ shift, const T* __restrict__ skip,
                                size_t total, T* __restrict__ dz) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int c = (int)(e % C);
  stf(dz, e, dz_at(y, da, e / C, c, C, Ho, Wo, pool, scale[c], shift[c], skip));
}

// xpad[p][0..Cp) = (x[p][0..C), 0, ...): one thread per 8-channel chunk (16 bytes) of the padded pixel, C <= 8
__global__ void pad_channels_kernel(const bf16* __restrict__ x, size_t P, int C, int Cp8, uint4* __restrict__ xpad) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= P * Cp8) return;
  const size_t p = e / Cp8;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (e % Cp8 == 0) {
    unsigned short h[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int c = 0; c < C; ++c) h[c] = __bfloat16_as_ushort(x[p * C + c]);
    v = make_uint4(h[0] | ((uint32_t)h[1] << 16), h[2] | ((uint32_t)h[3] << 16), h[4] | ((uint32_t)h[5] << 16), h[6] | ((uint32_t)h[7] << 16));
  }
  xpad[e] = v;
}
__global__ void pad_weights_kernel(const bf16* __restrict__ w, size_t rows, int C, int Cp, bf16* __restrict__ wpad) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= rows * Cp) return;
  const int c = (int)(e % Cp);
  wpad[e] = c < C ? w[(e / Cp) * C + c] : __float2bfloat16(0.f);
}
__global__ void unpad_grad_kernel(const float* __restrict__ gwpad, size_t rows, int C, int Cp, float* __restrict__ gw) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= rows * C) return;
  gw[e] = gwpad[(e / C) * Cp + e % C];
}

// Momentum SGD over up to kSgdMaxArenas parameter arenas in one launch (all layers of a block).  An arena is a multiple
// of 64 floats and 256-byte aligned, so every thread owns four consecutive elements: 16-byte loads of value, momentum and
// gradient, 16-byte stores of value and momentum, one 8-byte store of the four bf16 copies.  Blocks are dealt to arenas
// through the table of first-block indices.
__global__ void __launch_bounds__(256) sgd_multi_kernel(const SgdTable tb, float lr, float mu) {
  int a = 0;
  while (a + 1 < tb.count && (int)blockIdx.x >= tb.first_block[a + 1]) ++a;
  const size_t i4 = (size_t)(blockIdx.x - tb.first_block[a]) * blockDim.x + threadIdx.x;
  if (i4 * 4 >= tb.n[a]) return;
  const float4 g = reinterpret_cast<const float4*>(tb.grad[a])[i4];
  float4 m = reinterpret_cast<const float4*>(tb.mom[a])[i4];
  float4 t = reinterpret_cast<const float4*>(tb.val[a])[i4];
  m.x = fmaf(mu, m.x, g.x); m.y = fmaf(mu, m.y, g.y); m.z = fmaf(mu, m.z, g.z); m.w = fmaf(mu, m.w, g.w);
  t.x = fmaf(-lr, m.x, t.x); t.y = fmaf(-lr, m.y, t.y); t.z = fmaf(-lr, m.z, t.z); t.w = fmaf(-lr, m.w, t.w);
  reinterpret_cast<float4*>(tb.mom[a])[i4] = m;
  reinterpret_cast<float4*>(tb.val[a])[i4] = t;
  const __nv_bfloat162 lo = __floats2bfloat162_rn(t.x, t.y), hi = __floats2bfloat162_rn(t.z, t.w);
  reinterpret_cast<uint2*>(tb.shadow[a])[i4] =
      make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
}

__global__ void shadow_kernel(const float* __restrict__ val, bf16* __restrict__ shadow, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) shadow[i] = __float2bfloat16_rn(val[i]);
}

// out row r = cache row idx[r], 16 bytes per thread
// An index outside [0, cache_rows) reads nothing: its output row is zero-filled, its label set to -1 and NF_EINDEX raised.
__global__ void gather_kernel(const uint4* __restrict__ cache, const int32_t* __restrict__ cache_labels, int cache_rows,
                              const int32_t* __restrict__ idx, int count, size_t row16, uint4* __restrict__ out,
                              int32_t* __restrict__ out_labels, int32_t* __restrict__ status) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (size_t)count * row16) return;
  const size_t r = e / row16, k = e % row16;
  const int32_t src = idx[r];
  const bool ok = src >= 0 && src < cache_rows;
  out[e] = ok ? cache[(size_t)src * row16 + k] : make_uint4(0u, 0u, 0u, 0u);
  if (k == 0) {
    if (out_labels) out_labels[r] = ok ? cache_labels[src] : -1;
    if (!ok) atomicOr(status, NF_EINDEX);
  }
}


// ------------------------------------------------------------------ vectorised bf16 paths (C % 8 == 0, no pool)
// One thread owns 8 consecutive channels of a pixel: 16-byte loads and stores, coalesced along channels.
struct bf16x8 { uint4 u; };
__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  uint4 u;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  return u;
}

// out = ReLU(y*scale+shift); grid-stride over (pixel, channel group)
__global__ void __launch_bounds__(256) bn_apply_vec_kernel(const uint4* __restrict__ y, int C8, const float* __restrict__ scale,
                                                           const float* __restrict__ shift, size_t total8,
                                                           uint4* __restrict__ out) {
  extern __shared__ float cs[];  // scale[C], shift[C]
  const int C = C8 * 8;
  for (int i = threadIdx.x; i < C; i += 256) {
    cs[i] = scale[i];
    cs[C + i] = shift[i];
  }
  __syncthreads();
  for (size_t e = (size_t)blockIdx.x * 256 + threadIdx.x; e < total8; e += (size_t)gridDim.x * 256) {
    const int c0 = (int)(e % C8) * 8;
    float v[8];
    unpack8(__ldg(y + e), v);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = fmaxf(fmaf(v[i], cs[c0 + i], cs[C + c0 + i]), 0.f);
    out[e] = pack8(v);
  }
}


// per-thread constants variant (256 % C8 == 0)
__global__ void __launch_bounds__(256) bn_apply_vec2_kernel(const uint4* __restrict__ y, int C8, const float* __restrict__ scale,
                                                            const float* __restrict__ shift, size_t total8, uint4* __restrict__ out) {
  const int c0 = (threadIdx.x % C8) * 8;
  float A[8], B[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    A[i] = scale[c0 + i];
    B[i] = shift[c0 + i];
  }
  const size_t stride = (size_t)gridDim.x * 256;
  for (size_t e0 = (size_t)blockIdx.x * 256 + threadIdx.x; e0 < total8; e0 += 2 * stride) {
    const size_t e1 = e0 + stride;
    const bool two = e1 < total8;
    const uint4 ya = __ldg(y + e0);
    const uint4 yb = two ? __ldg(y + e1) : ya;
    float v[8];
    unpack8(ya, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = fmaxf(fmaf(v[i], A[i], B[i]), 0.f);
    out[e0] = pack8(v);
    if (two) {
      unpack8(yb, v);
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = fmaxf(fmaf(v[i], A[i], B[i]), 0.f);
      out[e1] = pack8(v);
    }
  }
}

// partial sums of (dz, dz*xhat) with dz = da * 1[y*scale+shift > 0]; red[(block*2+k)*C + c]
__global__ void __launch_bounds__(256) bn_bwd_reduce_vec_kernel(const uint4* __restrict__ y, const uint4* __restrict__ da,
                                                                size_t P, int C8, const float* __restrict__ scale,
                                                                const float* __restrict__ shift, const float* __restrict__ mu,
                                                                const float* __restrict__ invstd, float* __restrict__ red) {
  __shared__ float sm[16][256];
  const int C = C8 * 8;
  const int planes = 256 / C8, g = threadIdx.x % C8, pl = threadIdx.x / C8;
  const int c0 = g * 8;
  float sc[8], sh[8], m[8], is[8], a[8], b[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    sc[i] = scale[c0 + i]; sh[i] = shift[c0 + i]; m[i] = mu[c0 + i]; is[i] = invstd[c0 + i];
    a[i] = 0.f; b[i] = 0.f;
  }
  const size_t p0 = P * blockIdx.x / gridDim.x, p1 = P * (blockIdx.x + 1) / gridDim.x;
  if (pl < planes) {
    size_t p = p0 + pl;
    for (; p + planes < p1; p += 2 * (size_t)planes) {  // two pixels per iteration: four 16-byte loads in flight
      const uint4 y0 = __ldg(y + p * C8 + g), d0 = __ldg(da + p * C8 + g);
      const uint4 y1 = __ldg(y + (p + planes) * C8 + g), d1 = __ldg(da + (p + planes) * C8 + g);
      float yv[8], dv[8];
      unpack8(y0, yv);
      unpack8(d0, dv);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float dz = fmaf(yv[i], sc[i], sh[i]) > 0.f ? dv[i] : 0.f;
        a[i] += dz;
        b[i] = fmaf(dz, (yv[i] - m[i]) * is[i], b[i]);
      }
      unpack8(y1, yv);
      unpack8(d1, dv);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float dz = fmaf(yv[i], sc[i], sh[i]) > 0.f ? dv[i] : 0.f;
        a[i] += dz;
        b[i] = fmaf(dz, (yv[i] - m[i]) * is[i], b[i]);
      }
    }
    for (; p < p1; p += planes) {
      float yv[8], dv[8];
      unpack8(__ldg(y + p * C8 + g), yv);
      unpack8(__ldg(da + p * C8 + g), dv);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float dz = fmaf(yv[i], sc[i], sh[i]) > 0.f ? dv[i] : 0.f;
        a[i] += dz;
        b[i] = fmaf(dz, (yv[i] - m[i]) * is[i], b[i]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    sm[i][threadIdx.x] = a[i];
    sm[8 + i][threadIdx.x] = b[i];
  }
  __syncthreads();
  // thread t < 2*C finishes value k = t / C of channel c = t % C
  for (int t = threadIdx.x; t < 2 * C; t += 256) {
    const int k = t / C, c = t % C, gg = c / 8, i = c % 8;
    float s = 0.f;
    for (int q = 0; q < planes; ++q) s += sm[k * 8 + i][q * C8 + gg];
    red[((size_t)blockIdx.x * 2 + k) * C + c] = s;
  }
}

// dy = scale * (dz - sum(dz)/M - xhat * sum(dz*xhat)/M)
__global__ void __launch_bounds__(256) bn_bwd_apply_vec_kernel(const uint4* __restrict__ y, const uint4* __restrict__ da, int C8,
                                                               const float* __restrict__ scale, const float* __restrict__ shift,
                                                               const float* __restrict__ mu, const float* __restrict__ invstd,
                                                               const float* __restrict__ sdz, const float* __restrict__ sdzx,
                                                               float invM, size_t total8, uint4* __restrict__ dy) {
  extern __shared__ float cs[];  // per channel: scale, shift, mu, invstd, sdz/M, sdzx/M
  const int C = C8 * 8;
  for (int i = threadIdx.x; i < C; i += 256) {
    cs[i] = scale[i];
    cs[C + i] = shift[i];
    cs[2 * C + i] = mu[i];
    cs[3 * C + i] = invstd[i];
    cs[4 * C + i] = sdz[i] * invM;
    cs[5 * C + i] = sdzx[i] * invM;
  }
  __syncthreads();
  const size_t stride = (size_t)gridDim.x * 256;
  for (size_t e0 = (size_t)blockIdx.x * 256 + threadIdx.x; e0 < total8; e0 += 2 * stride) {  // two vectors per iteration
    const size_t e1 = e0 + stride;
    const bool two = e1 < total8;
    const uint4 ya = __ldg(y + e0), da0 = __ldg(da + e0);
    uint4 yb = ya, db = da0;
    if (two) {
      yb = __ldg(y + e1);
      db = __ldg(da + e1);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      if (h == 1 && !two) break;
      const size_t e = h ? e1 : e0;
      const int c0 = (int)(e % C8) * 8;
      float yv[8], dv[8], o[8];
      unpack8(h ? yb : ya, yv);
      unpack8(h ? db : da0, dv);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int c = c0 + i;
        const float dz = fmaf(yv[i], cs[c], cs[C + c]) > 0.f ? dv[i] : 0.f;
        const float xh = (yv[i] - cs[2 * C + c]) * cs[3 * C + c];
        o[i] = cs[c] * (dz - cs[4 * C + c] - xh * cs[5 * C + c]);
      }
      dy[e] = pack8(o);
    }
  }
}


// Same result with per-thread constants: when 256 % C8 == 0 a thread keeps its 8 channels over the whole
// grid-stride loop, and dy = s*dz + k1*y + k0 with k1 = -s*m2*invstd, k0 = s*(m2*invstd*mu - m1),
// m1 = sum(dz)/M, m2 = sum(dz*xhat)/M: five instructions per element.
__global__ void __launch_bounds__(256) bn_bwd_apply_vec2_kernel(const uint4* __restrict__ y, const uint4* __restrict__ da, int C8,
                                                                const float* __restrict__ scale, const float* __restrict__ shift,
                                                                const float* __restrict__ mu, const float* __restrict__ invstd,
                                                                const float* __restrict__ sdz, const float* __restrict__ sdzx,
                                                                float invM, size_t total8, uint4* __restrict__ dy) {
  const int c0 = (threadIdx.x % C8) * 8;
  float A[8], B[8], K1[8], K0[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float s = scale[c0 + i], m1 = sdz[c0 + i] * invM, m2 = sdzx[c0 + i] * invM, is = invstd[c0 + i];
    A[i] = s;
    B[i] = shift[c0 + i];
    K1[i] = -s * m2 * is;
    K0[i] = s * (m2 * is * mu[c0 + i] - m1);
  }
  const size_t stride = (size_t)gridDim.x * 256;
  for (size_t e0 = (size_t)blockIdx.x * 256 + threadIdx.x; e0 < total8; e0 += 2 * stride) {
    const size_t e1 = e0 + stride;
    const bool two = e1 < total8;
    const uint4 ya = __ldg(y + e0), da0 = __ldg(da + e0);
    uint4 yb = ya, db = da0;
    if (two) {
      yb = __ldg(y + e1);
      db = __ldg(da + e1);
    }
    float yv[8], dv[8], o[8];
    unpack8(ya, yv);
    unpack8(da0, dv);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float dz = fmaf(yv[i], A[i], B[i]) > 0.f ? dv[i] : 0.f;
      o[i] = fmaf(A[i], dz, fmaf(K1[i], yv[i], K0[i]));
    }
    dy[e0] = pack8(o);
    if (two) {
      unpack8(yb, yv);
      unpack8(db, dv);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float dz = fmaf(yv[i], A[i], B[i]) > 0.f ? dv[i] : 0.f;
        o[i] = fmaf(A[i], dz, fmaf(K1[i], yv[i], K0[i]));
      }
      dy[e1] = pack8(o);
    }
  }
}

// partial sums of (v, v^2) of a bf16 tensor; same layout of partials as channel_reduce_kernel
__global__ void __launch_bounds__(256) channel_sums_vec_kernel(const uint4* __restrict__ src, size_t P, int C8,
                                                               float* __restrict__ red) {
  __shared__ float sm[16][256];
  const int C = C8 * 8;
  const int planes = 256 / C8, g = threadIdx.x % C8, pl = threadIdx.x / C8;
  float a[8], b[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) a[i] = b[i] = 0.f;
  const size_t p0 = P * blockIdx.x / gridDim.x, p1 = P * (blockIdx.x + 1) / gridDim.x;
  if (pl < planes)
    for (size_t p = p0 + pl; p < p1; p += planes) {
      float v[8];
      unpack8(__ldg(src + p * C8 + g), v);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        a[i] += v[i];
        b[i] = fmaf(v[i], v[i], b[i]);
      }
    }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    sm[i][threadIdx.x] = a[i];
    sm[8 + i][threadIdx.x] = b[i];
  }
  __syncthreads();
  for (int t = threadIdx.x; t < 2 * C; t += 256) {
    const int k = t / C, c = t % C, gg = c / 8, i = c % 8;
    float s = 0.f;
    for (int q = 0; q < planes; ++q) s += sm[k * 8 + i][q * C8 + gg];
    red[((size_t)blockIdx.x * 2 + k) * C + c] = s;
  }
}


// dh = 1[h>0] * dp[n][f*4+bin]/|bin| for even sizes (every pixel lies in exactly one bin), 8 filters per
// thread, fused with the per-filter sum of dh (the aux bias gradient): red[(block*2+0)*F + f].
__global__ void __launch_bounds__(256) dh_vec_kernel(const uint4* __restrict__ h, const float* __restrict__ dp, int Ha, int Wa,
                                                     int F8, size_t P, uint4* __restrict__ dh, float* __restrict__ red) {
  __shared__ float sm[8][256];
  const int F = F8 * 8;
  const int planes = 256 / F8, g = threadIdx.x % F8, pl = threadIdx.x / F8;
  const float inv_bin = 1.f / (float)((Ha / 2) * (Wa / 2));
  float a[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) a[i] = 0.f;
  const size_t p0 = P * blockIdx.x / gridDim.x, p1 = P * (blockIdx.x + 1) / gridDim.x;
  auto one = [&](size_t p, const uint4 hq) {
    int i, j;
    size_t n;
    if (p <= 0xffffffffull) {  // 32-bit index arithmetic where it fits
      const uint32_t p32 = (uint32_t)p, row = p32 / (uint32_t)Wa;
      j = (int)(p32 - row * (uint32_t)Wa);
      n = row / (uint32_t)Ha;
      i = (int)(row - (uint32_t)n * (uint32_t)Ha);
    } else {
      j = (int)(p % Wa);
      i = (int)((p / Wa) % Ha);
      n = p / ((size_t)Wa * Ha);
    }
    const int bin = (i >= Ha / 2 ? 2 : 0) + (j >= Wa / 2 ? 1 : 0);
    float hv[8], o[8];
    unpack8(hq, hv);
    const float* d = dp + n * 4 * F + (size_t)(g * 8) * 4 + bin;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      o[e] = hv[e] > 0.f ? d[e * 4] * inv_bin : 0.f;
    }
    const uint4 packed = pack8(o);
    dh[p * F8 + g] = packed;
    float r[8];
    unpack8(packed, r);  // the bias gradient sums the values as stored
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] += r[e];
  };
  size_t p = p0 + pl;
  for (; p + 3 * (size_t)planes < p1; p += 4 * (size_t)planes) {  // four loads in flight, handled in index order
    uint4 q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) q[u] = __ldg(h + (p + (size_t)u * planes) * F8 + g);
#pragma unroll
    for (int u = 0; u < 4; ++u) one(p + (size_t)u * planes, q[u]);
  }
  for (; p < p1; p += planes) one(p, __ldg(h + p * F8 + g));
#pragma unroll
  for (int e = 0; e < 8; ++e) sm[e][threadIdx.x] = a[e];
  __syncthreads();
  for (int t = threadIdx.x; t < F; t += 256) {
    const int gg = t / 8, e = t % 8;
    float s = 0.f;
    for (int q = 0; q < planes; ++q) s += sm[e][q * F8 + gg];
    red[((size_t)blockIdx.x * 2 + 0) * F + t] = s;
    red[((size_t)blockIdx.x * 2 + 1) * F + t] = 0.f;
  }
}

// average pool, stage 1: partial bin sums over a slice of rows; part[(n*4+bin)*S + s][F]
__global__ void __launch_bounds__(256) avgpool_part_vec_kernel(const uint4* __restrict__ h, int Ha, int Wa, int F8, int S,
                                                               float* __restrict__ part) {
  __shared__ float sm[8][256];
  const int F = F8 * 8;
  const int planes = 256 / F8, g = threadIdx.x % F8, pl = threadIdx.x / F8;
  const int sidx = blockIdx.x % S, bin = (blockIdx.x / S) % 4, n = blockIdx.x / (4 * S);
  const int bh = Ha / 2, bw = Wa / 2, i0 = (bin >> 1) * bh, j0 = (bin & 1) * bw;
  const int cnt = bh * bw, k0 = (int)((long)cnt * sidx / S), k1 = (int)((long)cnt * (sidx + 1) / S);
  float a[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) a[i] = 0.f;
  const uint4* hn = h + (size_t)n * Ha * Wa * F8 + g;
  int k = k0 + pl;
  for (; k + 3 * planes < k1; k += 4 * planes) {  // four loads in flight, added in index order
    uint4 q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int kk = k + u * planes;
      q[u] = __ldg(hn + ((size_t)(i0 + kk / bw) * Wa + j0 + kk % bw) * F8);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float v[8];
      unpack8(q[u], v);
#pragma unroll
      for (int e = 0; e < 8; ++e) a[e] += v[e];
    }
  }
  for (; k < k1; k += planes) {
    float v[8];
    unpack8(__ldg(hn + ((size_t)(i0 + k / bw) * Wa + j0 + k % bw) * F8), v);
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] += v[e];
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) sm[e][threadIdx.x] = a[e];
  __syncthreads();
  for (int t = threadIdx.x; t < F; t += 256) {
    const int gg = t / 8, e = t % 8;
    float s = 0.f;
    for (int q = 0; q < planes; ++q) s += sm[e][q * F8 + gg];
    part[(size_t)blockIdx.x * F + t] = s;
  }
}
// stage 2: p[n][f*4+bin] = sum over slices / |bin|
// Average pool to 2 x 2 from the partials the fused aux forward leaves: part[tile][4][F] holds, per 14 x 8-pixel tile (tiles in
// row-major order per image, th x tw of them) and epilogue warp, the channel sums over the warp's pixels.  One block per
// (image, quadrant); thread (f, lane) adds every `lanes`-th of the quadrant's th/2 * tw/2 * 4 partials in index order, the lane
// sums are added in lane order.
__global__ void __launch_bounds__(256) pool_finish_kernel(const float* __restrict__ part, int th, int tw, int F, float inv_cnt,
                                                          float* __restrict__ p) {
  __shared__ float sm[256];
  const int n = blockIdx.x >> 2, bin = blockIdx.x & 3, u = bin >> 1, v = bin & 1;
  const int lanes = 256 / F, f = threadIdx.x % F, ln = threadIdx.x / F;
  const int qh = th / 2, qw = tw / 2, cnt = qh * qw * 4;
  float s = 0.f;
  if (ln < lanes) {
    auto at = [&](int k) {
      const int w4 = k & 3, tq = k >> 2, ty = u * qh + tq / qw, tx = v * qw + tq % qw;
      return part[(((size_t)n * th + ty) * tw + tx) * 4 * F + (size_t)w4 * F + f];
    };
    int k = ln;
    for (; k + 3 * lanes < cnt; k += 4 * lanes) {  // four loads in flight, added in index order
      const float a0 = at(k), a1 = at(k + lanes), a2 = at(k + 2 * lanes), a3 = at(k + 3 * lanes);
      s += a0;
      s += a1;
      s += a2;
      s += a3;
    }
    for (; k < cnt; k += lanes) s += at(k);
  }
  sm[threadIdx.x] = s;
  __syncthreads();
  if (ln == 0) {
    float t = 0.f;
    for (int l = 0; l < lanes; ++l) t += sm[l * F + f];
    p[(size_t)n * 4 * F + f * 4 + bin] = t * inv_cnt;
  }
}

// dh from the sign mask of h (one bit per element, byte g of a pixel = channels 8g .. 8g+7): dh = bit ? dp[n][f*4+bin] / |bin| : 0,
// stored in bf16; per-block partial sums of the stored values for the bias gradient, laid out as dh_vec_kernel does.
__global__ void __launch_bounds__(256) dh_mask_vec_kernel(const uint8_t* __restrict__ mask, const float* __restrict__ dp, int Ha, int Wa,
                                                          int F8, size_t P, uint4* __restrict__ dh, float* __restrict__ red) {
  __shared__ float sm[8][256];
  __shared__ __align__(16) float tab[4][4][64];  // dp / |bin| of up to four images, [image][bin][channel]: 16-byte reads per thread
  const int F = F8 * 8;
  const int planes = 256 / F8, g = threadIdx.x % F8, pl = threadIdx.x / F8;
  const float inv_bin = 1.f / (float)((Ha / 2) * (Wa / 2));
  float a[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) a[i] = 0.f;
  const size_t p0 = P * blockIdx.x / gridDim.x, p1 = P * (blockIdx.x + 1) / gridDim.x;
  const size_t img = (size_t)Wa * Ha;
  const size_t n_lo = p0 / img, n_hi = p1 > p0 ? (p1 - 1) / img : n_lo;
  const bool tabled = F <= 64 && n_hi - n_lo < 4;  // the block's pixel range touches few images: their dp rows fit the table
  if (tabled)
    for (int i = threadIdx.x; i < (int)(n_hi - n_lo + 1) * 4 * F; i += 256) {
      const int f = i % F, bin = (i / F) % 4, ni = i / (4 * F);
      tab[ni][bin][f] = dp[(n_lo + ni) * 4 * F + (size_t)f * 4 + bin] * inv_bin;
    }
  __syncthreads();
  auto one = [&](size_t p, uint32_t m) {
    // 32-bit index arithmetic (the host keeps P below 2^31): three 64-bit divisions per pixel had made this kernel compute-bound
    const uint32_t p32 = (uint32_t)p, row = p32 / (uint32_t)Wa;
    const int j = (int)(p32 - row * (uint32_t)Wa), i = (int)(row % (uint32_t)Ha);
    const size_t n = row / (uint32_t)Ha;
    const int bin = (i >= Ha / 2 ? 2 : 0) + (j >= Wa / 2 ? 1 : 0);
    float o[8];
    if (tabled) {
      const float4 t0 = *reinterpret_cast<const float4*>(&tab[n - n_lo][bin][g * 8]);
      const float4 t1 = *reinterpret_cast<const float4*>(&tab[n - n_lo][bin][g * 8 + 4]);
      const float tv[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
#pragma unroll
      for (int e = 0; e < 8; ++e) o[e] = (m >> e) & 1u ? tv[e] : 0.f;
    } else {
      const float* d = dp + n * 4 * F + (size_t)(g * 8) * 4 + bin;
#pragma unroll
      for (int e = 0; e < 8; ++e) o[e] = (m >> e) & 1u ? d[e * 4] * inv_bin : 0.f;
    }
    const uint4 packed = pack8(o);
    dh[p * F8 + g] = packed;
    float r[8];
    unpack8(packed, r);  // the bias gradient sums the values as stored
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] += r[e];
  };
  if (pl < planes) {  // threads beyond planes * F8 (F8 not a divisor of 256) idle
    size_t p = p0 + pl;
    for (; p + 3 * (size_t)planes < p1; p += 4 * (size_t)planes) {  // four mask bytes in flight, handled in index order
      uint32_t m[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) m[u] = mask[(p + (size_t)u * planes) * F8 + g];
#pragma unroll
      for (int u = 0; u < 4; ++u) one(p + (size_t)u * planes, m[u]);
    }
    for (; p < p1; p += planes) one(p, mask[p * F8 + g]);
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) sm[e][threadIdx.x] = a[e];
  __syncthreads();
  for (int t = threadIdx.x; t < F; t += 256) {
    const int gg = t / 8, e = t % 8;
    float s = 0.f;
    for (int q = 0; q < planes; ++q) s += sm[e][q * F8 + gg];
    red[((size_t)blockIdx.x * 2 + 0) * F + t] = s;
    red[((size_t)blockIdx.x * 2 + 1) * F + t] = 0.f;
  }
}

__global__ void avgpool_finish_kernel(const float* __restrict__ part, int N, int F, int S, float inv_cnt, float* __restrict__ p) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= N * 4 * F) return;
  const int f = e % F, bin = (e / F) % 4, n = e / (4 * F);
  float s = 0.f;
  for (int k = 0; k < S; ++k) s += part[((size_t)(n * 4 + bin) * S + k) * F + f];
  p[(size_t)n * 4 * F + f * 4 + bin] = s * inv_cnt;
}


// ------------------------------------------------------------------ vectorised bf16 paths for pooled layers
// One thread owns 8 channels of one POOLED pixel: it reads the four conv outputs of the 2x2 window.
__device__ __forceinline__ size_t div_small(size_t e, int d) {  // e / d in 32 bits where e fits
  return e <= 0xffffffffull ? (size_t)((uint32_t)e / (uint32_t)d) : e / (size_t)d;
}
__device__ __forceinline__ size_t win_base(size_t q, int Ho, int Wo, int C8) {  // q = pooled pixel index
  const int Wa = Wo / 2, Ha = Ho / 2;
  if (q <= 0xffffffffull) {  // 32-bit index arithmetic where it fits: three 64-bit divisions per window made these kernels compute-bound
    const uint32_t q32 = (uint32_t)q, row = q32 / (uint32_t)Wa;
    const uint32_t ja = q32 - row * (uint32_t)Wa, n = row / (uint32_t)Ha, ia = row - n * (uint32_t)Ha;
    return (((size_t)n * Ho + 2 * ia) * Wo + 2 * ja) * C8;
  }
  const int ja = (int)(q % Wa), ia = (int)((q / Wa) % Ha);
  const size_t n = q / ((size_t)Wa * Ha);
  return ((n * Ho + 2 * ia) * Wo + 2 * ja) * C8;
}

__global__ void __launch_bounds__(256) bn_apply_pool_vec_kernel(const uint4* __restrict__ y, int Ho, int Wo, int C8,
                                                                const float* __restrict__ scale, const float* __restrict__ shift,
                                                                size_t total8, uint4* __restrict__ out) {
  const int c0 = (threadIdx.x % C8) * 8;
  float A[8], B[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { A[i] = scale[c0 + i]; B[i] = shift[c0 + i]; }
  for (size_t e = (size_t)blockIdx.x * 256 + threadIdx.x; e < total8; e += (size_t)gridDim.x * 256) {
    const size_t b = win_base(div_small(e, C8), Ho, Wo, C8) + threadIdx.x % C8;  // 256 % C8 == 0: the chunk of a thread is fixed
    const uint4 v4[4] = {__ldg(y + b), __ldg(y + b + C8), __ldg(y + b + (size_t)Wo * C8), __ldg(y + b + (size_t)Wo * C8 + C8)};
    float best[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) best[i] = 0.f;
#pragma unroll
    for (int d = 0; d < 4; ++d) {
      float v[8];
      unpack8(v4[d], v);
#pragma unroll
      for (int i = 0; i < 8; ++i) best[i] = fmaxf(best[i], fmaf(v[i], A[i], B[i]));
    }
    out[e] = pack8(best);
  }
}

// dz of the four window positions: the first maximum (scan order) of the bf16-rounded ReLU outputs takes da
// if its pre-activation is positive.  arg[i] = winning position of channel i, or -1.
__device__ __forceinline__ void pool_winner(const float (&yv)[4][8], const float (&A)[8], const float (&B)[8], int (&arg)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float best = -1.f;
    int a = 0;
    float zbest = 0.f;
#pragma unroll
    for (int d = 0; d < 4; ++d) {
      const float z = fmaf(yv[d][i], A[i], B[i]);
      const float r = __bfloat162float(__float2bfloat16_rn(fmaxf(z, 0.f)));
      if (r > best) { best = r; a = d; zbest = z; }
    }
    arg[i] = zbest > 0.f ? a : -1;
  }
}

__global__ void __launch_bounds__(256) bn_bwd_reduce_pool_vec_kernel(const uint4* __restrict__ y, const uint4* __restrict__ da,
                                                                     size_t Pq, int Ho, int Wo, int C8,
                                                                     const float* __restrict__ scale, const float* __restrict__ shift,
                                                                     const float* __restrict__ mu, const float* __restrict__ invstd,
                                                                     float* __restrict__ red) {
  __shared__ float sm[16][256];
  const int C = C8 * 8;
  const int planes = 256 / C8, g = threadIdx.x % C8, pl = threadIdx.x / C8;
  const int c0 = g * 8;
  float A[8], B[8], m[8], is[8], a[8], b[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    A[i] = scale[c0 + i]; B[i] = shift[c0 + i]; m[i] = mu[c0 + i]; is[i] = invstd[c0 + i];
    a[i] = 0.f; b[i] = 0.f;
  }
  const size_t q0 = Pq * blockIdx.x / gridDim.x, q1 = Pq * (blockIdx.x + 1) / gridDim.x;
  for (size_t q = q0 + pl; q < q1; q += planes) {
    const size_t bb = win_base(q, Ho, Wo, C8) + g;
    const uint4 v4[4] = {__ldg(y + bb), __ldg(y + bb + C8), __ldg(y + bb + (size_t)Wo * C8), __ldg(y + bb + (size_t)Wo * C8 + C8)};
    float yv[4][8], dv[8];
#pragma unroll
    for (int d = 0; d < 4; ++d) unpack8(v4[d], yv[d]);
    unpack8(__ldg(da + q * C8 + g), dv);
    int arg[8];
    pool_winner(yv, A, B, arg);
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (arg[i] >= 0) {
        const float yy = arg[i] == 0 ? yv[0][i] : arg[i] == 1 ? yv[1][i] : arg[i] == 2 ? yv[2][i] : yv[3][i];
        a[i] += dv[i];
        b[i] = fmaf(dv[i], (yy - m[i]) * is[i], b[i]);
      }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    sm[i][threadIdx.x] = a[i];
    sm[8 + i][threadIdx.x] = b[i];
  }
  __syncthreads();
  for (int t = threadIdx.x; t < 2 * C; t += 256) {
    const int k = t / C, c = t % C, gg = c / 8, i = c % 8;
    float s = 0.f;
    for (int qq = 0; qq < planes; ++qq) s += sm[k * 8 + i][qq * C8 + gg];
    red[((size_t)blockIdx.x * 2 + k) * C + c] = s;
  }
}

__global__ void __launch_bounds__(256) bn_bwd_apply_pool_vec_kernel(const uint4* __restrict__ y, const uint4* __restrict__ da, int Ho,
                                                                    int Wo, int C8, const float* __restrict__ scale,
                                                                    const float* __restrict__ shift, const float* __restrict__ mu,
                                                                    const float* __restrict__ invstd, const float* __restrict__ sdz,
                                                                    const float* __restrict__ sdzx, float invM, size_t total8,
                                                                    uint4* __restrict__ dy) {
  const int c0 = (threadIdx.x % C8) * 8;
  float A[8], B[8], K1[8], K0[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float s = scale[c0 + i], m1 = sdz[c0 + i] * invM, m2 = sdzx[c0 + i] * invM, is = invstd[c0 + i];
    A[i] = s; B[i] = shift[c0 + i];
    K1[i] = -s * m2 * is;
    K0[i] = s * (m2 * is * mu[c0 + i] - m1);
  }
  for (size_t e = (size_t)blockIdx.x * 256 + threadIdx.x; e < total8; e += (size_t)gridDim.x * 256) {  // e over pooled vectors
    const size_t bb = win_base(div_small(e, C8), Ho, Wo, C8) + threadIdx.x % C8;
    const size_t off[4] = {0, (size_t)C8, (size_t)Wo * C8, (size_t)Wo * C8 + C8};
    float yv[4][8], dv[8];
#pragma unroll
    for (int d = 0; d < 4; ++d) unpack8(__ldg(y + bb + off[d]), yv[d]);
    unpack8(__ldg(da + e), dv);
    int arg[8];
    pool_winner(yv, A, B, arg);
#pragma unroll
    for (int d = 0; d < 4; ++d) {
      float o[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) o[i] = fmaf(A[i], arg[i] == d ? dv[i] : 0.f, fmaf(K1[i], yv[d][i], K0[i]));
      dy[bb + off[d]] = pack8(o);
    }
  }
}

inline bool vec_ok(int dtype, int C, int pool) { return dtype == NF_BF16 && C % 8 == 0 && C <= 1024 && !pool; }
inline int vec_blocks(size_t work_items) {
  size_t b = (work_items + 256 * 8 - 1) / (256 * 8);
  if (b < 1) b = 1;
  if (b > 148 * 16) b = 148 * 16;
  return (int)b;
}

inline unsigned nblk(size_t n, int per) { return (unsigned)((n + per - 1) / per); }

}  // namespace

#define DISPATCH(dtype, CALL_F32, CALL_BF16) \
  do {                                       \
    if ((dtype) == NF_F32) { CALL_F32; } else { CALL_BF16; } \
  } while (0)

int nf_k_channel_blocks(size_t P, int C) {
  const int planes = 256 / pow2ceil_cap256(C);
  size_t nb = (P + (size_t)planes * 16 - 1) / ((size_t)planes * 16);
  if (nb < 1) nb = 1;
  if (nb > 1184) nb = 1184;
  return (int)nb;
}

int nf_k_channel_sums(int dtype, const void* src, size_t P, int C, float* red, size_t red_floats, int* nblocks) {
  const int nb = nf_k_channel_blocks(P, C);
  if ((size_t)nb * 2 * C > red_floats) return NF_ENOWS;
  if (vec_ok(dtype, C, 0) && 256 % (C / 8) == 0) {
    channel_sums_vec_kernel<<<nb, 256, 0, g_nf_stream>>>((const uint4*)src, P, C / 8, red);
    NF_LAUNCHED();
    *nblocks = nb;
    return NF_OK;
  }
  DISPATCH(dtype,
           (channel_reduce_kernel<float, StatsFn><<<nb, 256, 0, g_nf_stream>>>((const float*)src, nullptr, P, C, StatsFn(), red)),
           (channel_reduce_kernel<bf16, StatsFn><<<nb, 256, 0, g_nf_stream>>>((const bf16*)src, nullptr, P, C, StatsFn(), red)));
  NF_LAUNCHED();
  *nblocks = nb;
  return NF_OK;
}

int nf_k_bn_finalize(const float* red, int nblocks, int C, double M, const float* gamma, const float* beta,
                       float eps, float bn_momentum, float* scale, float* shift, float* mu, float* invstd,
                       float* rmean, float* rvar) {
  bn_finalize_kernel<<<nblk(C, 32), dim3(32, 32), 0, g_nf_stream>>>(red, nblocks, C, M, gamma, beta, eps, bn_momentum, scale,
                                                            shift, mu, invstd, rmean, rvar);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_partial_totals(const float* red, int nblocks, int C, double* tot) {
  partial_totals_kernel<<<nblk(C, 32), dim3(32, 32), 0, g_nf_stream>>>(red, nblocks, C, tot);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_bn_finalize_tot(const double* tot, int C, double M, const float* gamma, const float* beta, float eps, float bn_momentum,
                           float* scale, float* shift, float* mu, float* invstd, float* rmean, float* rvar) {
  bn_finalize_tot_kernel<<<nblk(C, 128), 128, 0, g_nf_stream>>>(tot, C, M, gamma, beta, eps, bn_momentum, scale, shift, mu, invstd,
                                                                rmean, rvar);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_bn_bwd_finalize_tot(const double* tot, int C, int world, float* sdz, float* sdzx, float* ggamma, float* gbeta) {
  bn_bwd_finalize_tot_kernel<<<nblk(C, 128), 128, 0, g_nf_stream>>>(tot, C, 1.0 / (double)world, sdz, sdzx, ggamma, gbeta);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_bn_eval_coeffs(int C, const float* gamma, const float* beta, float eps, const float* rmean,
                          const float* rvar, float* scale, float* shift) {
  bn_eval_coeffs_kernel<<<nblk(C, 128), 128, 0, g_nf_stream>>>(C, gamma, beta, eps, rmean, rvar, scale, shift);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_bn_apply(int dtype, const void* y, int N, int Ho, int Wo, int C, int pool, const float* scale,
                    const float* shift, void* out, const void* skip) {
  const size_t total = (size_t)N * (pool ? Ho / 2 : Ho) * (pool ? Wo / 2 : Wo) * C;
  if (skip) {  // residual layers take the generic kernels
    DISPATCH(dtype,
             (bn_apply_kernel<float><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const float*)y, Ho, Wo, C, pool, scale, shift, total, (float*)out, (const float*)skip)),
             (bn_apply_kernel<bf16><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const bf16*)y, Ho, Wo, C, pool, scale, shift, total, (bf16*)out, (const bf16*)skip)));
    NF_LAUNCHED();
    return NF_OK;
  }
  if (pool && vec_ok(dtype, C, 0) && 256 % (C / 8) == 0) {
    bn_apply_pool_vec_kernel<<<vec_blocks(total / 8), 256, 0, g_nf_stream>>>((const uint4*)y, Ho, Wo, C / 8, scale, shift, total / 8,
                                                                            (uint4*)out);
    NF_LAUNCHED();
    return NF_OK;
  }
  if (vec_ok(dtype, C, pool) && 256 % (C / 8) == 0) {
    bn_apply_vec2_kernel<<<vec_blocks(total / 8), 256, 0, g_nf_stream>>>((const uint4*)y, C / 8, scale, shift, total / 8, (uint4*)out);
    NF_LAUNCHED();
    return NF_OK;
  }
  if (vec_ok(dtype, C, pool)) {
    bn_apply_vec_kernel<<<vec_blocks(total / 8), 256, 2 * C * sizeof(float), g_nf_stream>>>((const uint4*)y, C / 8, scale, shift,
                                                                                         total / 8, (uint4*)out);
    NF_LAUNCHED();
    return NF_OK;
  }
  DISPATCH(dtype,
           (bn_apply_kernel<float><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const float*)y, Ho, Wo, C, pool, scale, shift, total, (float*)out, nullptr)),
           (bn_apply_kernel<bf16><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const bf16*)y, Ho, Wo, C, pool, scale, shift, total, (bf16*)out, nullptr)));
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_avgpool_slices(int N, int Ha, int Wa) {
  const long cnt = (long)(Ha / 2) * (Wa / 2);
  long S = 1184 / ((long)N * 4);
  if (S > cnt / 64) S = cnt / 64;
  if (S < 1) S = 1;
  return (int)S;
}

int nf_k_avgpool_fast(const void* h, int N, int Ha, int Wa, int F, float* part, size_t part_floats, float* p) {
  if (F % 8 || 256 % (F / 8) || (Ha & 1) || (Wa & 1)) return NF_EUNSUPPORTED;
  if ((long)(Ha / 2) * (Wa / 2) <= 16) return NF_EUNSUPPORTED;  // tiny maps: the caller's generic path has a kernel for them
  const int S = nf_k_avgpool_slices(N, Ha, Wa);
  if ((size_t)N * 4 * S * F > part_floats) return NF_EUNSUPPORTED;
  avgpool_part_vec_kernel<<<N * 4 * S, 256, 0, g_nf_stream>>>((const uint4*)h, Ha, Wa, F / 8, S, part);
  NF_LAUNCHED();
  avgpool_finish_kernel<<<nblk((size_t)N * 4 * F, 256), 256, 0, g_nf_stream>>>(part, N, F, S, 1.f / (float)((Ha / 2) * (Wa / 2)), p);
  NF_LAUNCHED();
  return NF_OK;
}

// dh with the fused aux-bias gradient partials (bf16, F % 8 == 0, even sizes); nblocks partials in red
int nf_k_pool_finish(const float* part, int N, int th, int tw, int F, float inv_cnt, float* p) {
  if (F < 1 || F > 256) return NF_EUNSUPPORTED;
  pool_finish_kernel<<<N * 4, 256, 0, g_nf_stream>>>(part, th, tw, F, inv_cnt, p);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_dh_mask(const uint8_t* mask, const float* dp, int N, int Ha, int Wa, int F, void* dh, float* red, size_t red_floats,
                 int* nblocks) {
  if (F % 8 || F > 2048 || (Ha & 1) || (Wa & 1)) return NF_EUNSUPPORTED;
  const size_t P = (size_t)N * Ha * Wa;
  if (P >= ((size_t)1 << 31)) return NF_EUNSUPPORTED;
  const int nb = nf_k_channel_blocks(P, F);
  if ((size_t)nb * 2 * F > red_floats) return NF_ENOWS;
  dh_mask_vec_kernel<<<nb, 256, 0, g_nf_stream>>>(mask, dp, Ha, Wa, F / 8, P, (uint4*)dh, red);
  NF_LAUNCHED();
  *nblocks = nb;
  return NF_OK;
}

int nf_k_dh_fast(const void* h, const float* dp, int N, int Ha, int Wa, int F, void* dh, float* red, size_t red_floats,
                   int* nblocks) {
  if (F % 8 || 256 % (F / 8) || (Ha & 1) || (Wa & 1)) return NF_EUNSUPPORTED;
  const size_t P = (size_t)N * Ha * Wa;
  const int nb = nf_k_channel_blocks(P, F);
  if ((size_t)nb * 2 * F > red_floats) return NF_EUNSUPPORTED;
  dh_vec_kernel<<<nb, 256, 0, g_nf_stream>>>((const uint4*)h, dp, Ha, Wa, F / 8, P, (uint4*)dh, red);
  NF_LAUNCHED();
  *nblocks = nb;
  return NF_OK;
}

int nf_k_avgpool(int dtype, const void* h, int N, int Ha, int Wa, int F, float* p) {
  if ((long)((Ha + 1) / 2) * ((Wa + 1) / 2) <= 16) {  // tiny maps (late blocks train at thousands of samples): a thread per output
    const size_t total = (size_t)N * 4 * F;
    DISPATCH(dtype, (avgpool_small_kernel<float><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const float*)h, Ha, Wa, F, total, p)),
             (avgpool_small_kernel<bf16><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const bf16*)h, Ha, Wa, F, total, p)));
    NF_LAUNCHED();
    return NF_OK;
  }
  DISPATCH(dtype, (avgpool_kernel<float><<<N * 4, 256, 0, g_nf_stream>>>((const float*)h, Ha, Wa, F, p)),
           (avgpool_kernel<bf16><<<N * 4, 256, 0, g_nf_stream>>>((const bf16*)h, Ha, Wa, F, p)));
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_fc_ce(const float* p, const int32_t* labels, int N, int D, int K, const float* Wf, const float* bf,
                 float* logits, float* dlogits, float* dp, float* lossn, int32_t* status, int loss_kind, int n_scale) {
  const size_t smem = (size_t)(D + K) * sizeof(float);
  if (smem > 40000) return NF_EUNSUPPORTED;
  fc_ce_kernel<<<N, 256, smem, g_nf_stream>>>(p, labels, N, D, K, Wf, bf, logits, dlogits, dp, lossn, status, loss_kind, n_scale);
  NF_LAUNCHED();
  return NF_OK;
}

__global__ void __launch_bounds__(256) count_equal_kernel(const int32_t* __restrict__ a, const int32_t* __restrict__ b, long long n,
                                                          unsigned long long* __restrict__ count) {
  unsigned c = 0;
  for (long long i = blockIdx.x * 256LL + threadIdx.x; i < n; i += 256LL * gridDim.x) c += a[i] == b[i];
  c = __reduce_add_sync(0xffffffffu, c);
  if ((threadIdx.x & 31) == 0 && c) atomicAdd(count, (unsigned long long)c);   // integer sum: order-independent
}

int nf_k_count_equal(const int32_t* a, const int32_t* b, long long n, unsigned long long* count) {
  const int blocks = (int)std::min<long long>((n + 255) / 256, 1184);
  count_equal_kernel<<<blocks, 256, 0, g_nf_stream>>>(a, b, n, count);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_fc_predict(const float* p, int N, int D, int K, const float* Wf, const float* bf, float* logits, int32_t* pred) {
  const size_t smem = (size_t)D * sizeof(float);
  if (smem > 40000) return NF_EUNSUPPORTED;
  fc_predict_kernel<<<N, 256, smem, g_nf_stream>>>(p, D, K, Wf, bf, logits, pred);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_fc_wgrad(const float* p, const float* dlogits, const float* lossn, int N, int D, int K, float* gWf,
                    float* gbf, float* loss_out, int32_t* status, int n_scale) {
  fc_wgrad_kernel<<<K, 256, 0, g_nf_stream>>>(p, dlogits, lossn, N, D, K, gWf, gbf, loss_out, status, n_scale);
  NF_LAUNCHED();
  return NF_OK;
}

// out[8 - tap][c][f] = w[tap][f][c]: the weights of the input-gradient convolution written as a forward convolution
__global__ void flip_weights_kernel(const bf16* __restrict__ w, int F, int C, bf16* __restrict__ out) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (size_t)9 * F * C) return;
  const int f = (int)(e % F), c = (int)((e / F) % C), tap = (int)(e / ((size_t)F * C));
  out[e] = w[((size_t)(8 - tap) * F + f) * C + c];
}

int nf_k_flip_weights(const bf16* w, int F, int C, bf16* out) {
  flip_weights_kernel<<<nblk((size_t)9 * F * C, 256), 256, 0, g_nf_stream>>>(w, F, C, out);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_auxmax(int dtype, const void* h, int N, int Ha, int Wa, int F, float* p, int32_t* parg) {
  DISPATCH(dtype, (auxmax_kernel<float><<<N * 4, 256, 0, g_nf_stream>>>((const float*)h, Ha, Wa, F, p, parg)),
           (auxmax_kernel<bf16><<<N * 4, 256, 0, g_nf_stream>>>((const bf16*)h, Ha, Wa, F, p, parg)));
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_dh_max(int dtype, const void* h, const float* dp, const int32_t* parg, int N, int Ha, int Wa, int F, void* dh) {
  const size_t total = (size_t)N * Ha * Wa * F;
  DISPATCH(dtype, (dh_max_kernel<float><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const float*)h, dp, parg, Ha, Wa, F, total, (float*)dh)),
           (dh_max_kernel<bf16><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const bf16*)h, dp, parg, Ha, Wa, F, total, (bf16*)dh)));
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_dh(int dtype, const void* h, const float* dp, int N, int Ha, int Wa, int F, void* dh) {
  const size_t total = (size_t)N * Ha * Wa * F;
  DISPATCH(dtype, (dh_kernel<float><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const float*)h, dp, Ha, Wa, F, total, (float*)dh)),
           (dh_kernel<bf16><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const bf16*)h, dp, Ha, Wa, F, total, (bf16*)dh)));
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_sum_partials(const float* red, int nblocks, int C, int which, float* out) {
  sum_partials_kernel<<<nblk(C, 32), dim3(32, 32), 0, g_nf_stream>>>(red, nblocks, C, which, out);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_bn_bwd_reduce(int dtype, const void* y, const void* da, int N, int Ho, int Wo, int C, int pool,
                         const float* scale, const float* shift, const float* mu, const float* invstd, float* red,
                         size_t red_floats, int* nblocks, const void* skip) {
  const size_t P = (size_t)N * Ho * Wo;
  const int nb = nf_k_channel_blocks(P, C);
  if ((size_t)nb * 2 * C > red_floats) return NF_ENOWS;
  if (!skip && pool && vec_ok(dtype, C, 0) && 256 % (C / 8) == 0) {
    bn_bwd_reduce_pool_vec_kernel<<<nb, 256, 0, g_nf_stream>>>((const uint4*)y, (const uint4*)da, P / 4, Ho, Wo, C / 8, scale, shift, mu,
                                                              invstd, red);
    NF_LAUNCHED();
    *nblocks = nb;
    return NF_OK;
  }
  if (!skip && vec_ok(dtype, C, pool) && 256 % (C / 8) == 0) {
    bn_bwd_reduce_vec_kernel<<<nb, 256, 0, g_nf_stream>>>((const uint4*)y, (const uint4*)da, P, C / 8, scale, shift, mu, invstd, red);
    NF_LAUNCHED();
    *nblocks = nb;
    return NF_OK;
  }
  BnBwdFn fn{Ho, Wo, pool, scale, shift, mu, invstd, skip};
  DISPATCH(dtype,
           (channel_reduce_kernel<float, BnBwdFn><<<nb, 256, 0, g_nf_stream>>>((const float*)y, (const float*)da, P, C, fn, red)),
           (channel_reduce_kernel<bf16, BnBwdFn><<<nb, 256, 0, g_nf_stream>>>((const bf16*)y, (const bf16*)da, P, C, fn, red)));
  NF_LAUNCHED();
  *nblocks = nb;
  return NF_OK;
}

int nf_k_write_dz(int dtype, const void* y, const void* da, int N, int Ho, int Wo, int C, int pool, const float* scale,
                  const float* shift, const void* skip, void* dz) {
  const size_t total = (size_t)N * Ho * Wo * C;
  DISPATCH(dtype,
           (write_dz_kernel<float><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const float*)y, (const float*)da, Ho, Wo, C, pool, scale, shift, (const float*)skip, total, (float*)dz)),
           (write_dz_kernel<bf16><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const bf16*)y, (const bf16*)da, Ho, Wo, C, pool, scale, shift, (const bf16*)skip, total, (bf16*)dz)));
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_bn_bwd_finalize(const float* red, int nblocks, int C, float* sdz, float* sdzx, float* ggamma,
                           float* gbeta) {
  bn_bwd_finalize_kernel<<<nblk(C, 32), dim3(32, 32), 0, g_nf_stream>>>(red, nblocks, C, sdz, sdzx, ggamma, gbeta);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_bn_bwd_apply(int dtype, const void* y, const void* da, int N, int Ho, int Wo, int C, int pool,
                        const float* scale, const float* shift, const float* mu, const float* invstd,
                        const float* sdz, const float* sdzx, double M, void* dy, const void* skip) {
  const size_t total = (size_t)N * Ho * Wo * C;
  const float invM = (float)(1.0 / M);
  if (skip) {
    DISPATCH(dtype,
             (bn_bwd_apply_kernel<float><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const float*)y, (const float*)da, Ho, Wo, C, pool, scale, shift, mu, invstd, sdz, sdzx, invM, total, (float*)dy, (const float*)skip)),
             (bn_bwd_apply_kernel<bf16><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const bf16*)y, (const bf16*)da, Ho, Wo, C, pool, scale, shift, mu, invstd, sdz, sdzx, invM, total, (bf16*)dy, (const bf16*)skip)));
    NF_LAUNCHED();
    return NF_OK;
  }
  if (pool && vec_ok(dtype, C, 0) && 256 % (C / 8) == 0) {
    bn_bwd_apply_pool_vec_kernel<<<vec_blocks(total / 32), 256, 0, g_nf_stream>>>((const uint4*)y, (const uint4*)da, Ho, Wo, C / 8, scale,
                                                                                 shift, mu, invstd, sdz, sdzx, invM, total / 32, (uint4*)dy);
    NF_LAUNCHED();
    return NF_OK;
  }
  if (vec_ok(dtype, C, pool) && 256 % (C / 8) == 0) {
    bn_bwd_apply_vec2_kernel<<<vec_blocks(total / 8), 256, 0, g_nf_stream>>>((const uint4*)y, (const uint4*)da, C / 8, scale, shift, mu,
                                                                            invstd, sdz, sdzx, invM, total / 8, (uint4*)dy);
    NF_LAUNCHED();
    return NF_OK;
  }
  if (vec_ok(dtype, C, pool)) {
    bn_bwd_apply_vec_kernel<<<vec_blocks(total / 8), 256, 6 * C * sizeof(float), g_nf_stream>>>(
        (const uint4*)y, (const uint4*)da, C / 8, scale, shift, mu, invstd, sdz, sdzx, invM, total / 8, (uint4*)dy);
    NF_LAUNCHED();
    return NF_OK;
  }
  DISPATCH(dtype,
           (bn_bwd_apply_kernel<float><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const float*)y, (const float*)da, Ho, Wo, C, pool, scale, shift, mu, invstd, sdz, sdzx, invM, total, (float*)dy, nullptr)),
           (bn_bwd_apply_kernel<bf16><<<nblk(total, 256), 256, 0, g_nf_stream>>>((const bf16*)y, (const bf16*)da, Ho, Wo, C, pool, scale, shift, mu, invstd, sdz, sdzx, invM, total, (bf16*)dy, nullptr)));
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_pad_channels(const void* x, size_t P, int C, int Cp, void* xpad) {
  if (C < 1 || C > 8 || Cp % 8) return NF_EUNSUPPORTED;
  pad_channels_kernel<<<nblk(P * (Cp / 8), 256), 256, 0, g_nf_stream>>>((const bf16*)x, P, C, Cp / 8, (uint4*)xpad);
  NF_LAUNCHED();
  return NF_OK;
}
int nf_k_pad_weights(const bf16* w, size_t rows, int C, int Cp, bf16* wpad) {
  pad_weights_kernel<<<nblk(rows * Cp, 256), 256, 0, g_nf_stream>>>(w, rows, C, Cp, wpad);
  NF_LAUNCHED();
  return NF_OK;
}
int nf_k_unpad_grad(const float* gwpad, size_t rows, int C, int Cp, float* gw) {
  unpad_grad_kernel<<<nblk(rows * C, 256), 256, 0, g_nf_stream>>>(gwpad, rows, C, Cp, gw);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_sgd_multi(const SgdTable& tb_in, float lr, float momentum) {
  if (tb_in.count < 1 || tb_in.count > kSgdMaxArenas) return NF_EINVAL;
  SgdTable tb = tb_in;
  int blocks = 0;
  for (int a = 0; a < tb.count; ++a) {
    if (tb.n[a] % 4) return NF_EINVAL;
    tb.first_block[a] = blocks;
    blocks += (int)nblk(tb.n[a] / 4, 256);
  }
  sgd_multi_kernel<<<blocks, 256, 0, g_nf_stream>>>(tb, lr, momentum);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_sgd(float* val, float* mom, const float* grad, bf16* shadow, size_t n, float lr, float momentum) {
  SgdTable tb{};
  tb.count = 1;
  tb.val[0] = val; tb.mom[0] = mom; tb.grad[0] = grad; tb.shadow[0] = shadow; tb.n[0] = n;
  return nf_k_sgd_multi(tb, lr, momentum);
}

int nf_k_shadow(const float* val, bf16* shadow, size_t n) {
  shadow_kernel<<<nblk(n, 256), 256, 0, g_nf_stream>>>(val, shadow, n);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_gather(const void* cache, const int32_t* cache_labels, int cache_rows, const int32_t* idx, int count, size_t row_bytes,
                  void* out, int32_t* out_labels, int32_t* status) {
  const size_t row16 = row_bytes / 16;
  gather_kernel<<<nblk((size_t)count * row16, 256), 256, 0, g_nf_stream>>>((const uint4*)cache, cache_labels, cache_rows, idx,
                                                                         count, row16, (uint4*)out, out_labels, status);
  NF_LAUNCHED();
  return NF_OK;
}
