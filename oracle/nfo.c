/*
 * nfo.c -- reference checker ("oracle") for the per-layer local training step
 * of adaptive local learning (NeuroFlux, arXiv 2402.14139).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, fp64 CPU
 * program written from the paper's definitions (Eq. 1-3, Algorithm 2) and is
 * used only to check the CUDA library and to time a CPU baseline.  It shares
 * no code, table or helper with the CUDA path and neither includes the other.
 *
 * Logical layout everywhere: NCHW, row-major, double.  All convolutions are
 * 3x3 with zero padding 1.  No blocking, no fusion, no reordering: each
 * function is the definition written out as loops.  OpenMP pragmas only
 * split independent outer iterations; they never change a summation order.
 *
 * Parts the paper leaves open and that are fixed here (the paper states only
 * conv / ReLU / down-sampling / aux conv / pooling / linear / loss / update):
 *   - BatchNorm with batch statistics between conv and ReLU      (parity unpinned by the paper)
 *   - aux conv is 3x3 pad 1 stride 1 with bias and ReLU          (parity unpinned by the paper)
 *   - momentum SGD  v <- mu v + g ; theta <- theta - lr v         (parity unpinned by the paper;
 *     the paper's Appendix B writes plain SGD, which is mu = 0)
 *   - running statistics: momentum 0.1, unbiased variance        (parity unpinned by the paper)
 *   - cache written by an eval-mode forward (running statistics) (parity unpinned by the paper)
 * Each of these is still pinned against mathematics (finite differences,
 * closed forms, library routines) by tests/test_oracle_*.py.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define IDX4(n, c, i, j, C, H, W) ((((size_t)(n) * (C) + (c)) * (H) + (i)) * (W) + (j))

int nfo_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

int nfo_out_size(int H, int stride) { return (H - 1) / stride + 1; }

/* Eq. 1 (theta_n x_n) and Eq. 2 (beta_n x_{n+1}): 3x3 convolution, pad 1.
 * y[n,co,i,j] = bias[co] + sum_{ci,kh,kw} w[co,ci,kh,kw] * x[n,ci,i*s+kh-1,j*s+kw-1]
 * with x taken as zero outside the image.  bias may be NULL. */
void nfo_conv3x3(const double* x, int N, int Cin, int H, int W, const double* w, int Cout,
                 const double* bias, int stride, double* y) {
  const int Ho = nfo_out_size(H, stride), Wo = nfo_out_size(W, stride);
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int co = 0; co < Cout; ++co)
      for (int i = 0; i < Ho; ++i)
        for (int j = 0; j < Wo; ++j) {
          double acc = bias ? bias[co] : 0.0;
          for (int ci = 0; ci < Cin; ++ci)
            for (int kh = 0; kh < 3; ++kh)
              for (int kw = 0; kw < 3; ++kw) {
                const int ii = i * stride + kh - 1, jj = j * stride + kw - 1;
                if (ii < 0 || ii >= H || jj < 0 || jj >= W) continue;
                acc += w[(((size_t)co * Cin + ci) * 3 + kh) * 3 + kw] * x[IDX4(n, ci, ii, jj, Cin, H, W)];
              }
          y[IDX4(n, co, i, j, Cout, Ho, Wo)] = acc;
        }
}

/* The projection shortcut of a down-sampling residual block (the paper trains ResNet-18, Section "Experimental
 * Setup"): a 1x1 convolution with stride s, y[n,co,i,j] = sum_ci w[co,ci] * x[n,ci,i*s,j*s], and the derivative of that
 * with respect to its weights, dw[co,ci] = sum_{n,i,j} g[n,co,i,j] * x[n,ci,i*s,j*s]. */
void nfo_conv1x1(const double* x, int N, int Cin, int H, int W, const double* w, int Cout, int stride, double* y) {
  const int Ho = nfo_out_size(H, stride), Wo = nfo_out_size(W, stride);
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int co = 0; co < Cout; ++co)
      for (int i = 0; i < Ho; ++i)
        for (int j = 0; j < Wo; ++j) {
          double acc = 0.0;
          for (int ci = 0; ci < Cin; ++ci) acc += w[(size_t)co * Cin + ci] * x[IDX4(n, ci, i * stride, j * stride, Cin, H, W)];
          y[IDX4(n, co, i, j, Cout, Ho, Wo)] = acc;
        }
}

void nfo_conv1x1_wgrad(const double* x, int N, int Cin, int H, int W, const double* g, int Cout, int stride, double* dw) {
  const int Ho = nfo_out_size(H, stride), Wo = nfo_out_size(W, stride);
#pragma omp parallel for collapse(2) schedule(static)
  for (int co = 0; co < Cout; ++co)
    for (int ci = 0; ci < Cin; ++ci) {
      double acc = 0.0;
      for (int n = 0; n < N; ++n)
        for (int i = 0; i < Ho; ++i)
          for (int j = 0; j < Wo; ++j)
            acc += g[IDX4(n, co, i, j, Cout, Ho, Wo)] * x[IDX4(n, ci, i * stride, j * stride, Cin, H, W)];
      dw[(size_t)co * Cin + ci] = acc;
    }
}

/* Algorithm 2, gradient step: derivative of the convolution with respect to its weights.
 * dw[co,ci,kh,kw] = sum_{n,i,j} g[n,co,i,j] * x[n,ci,i*s+kh-1,j*s+kw-1]. */
void nfo_conv3x3_wgrad(const double* x, int N, int Cin, int H, int W, const double* g, int Cout,
                       int stride, double* dw) {
  const int Ho = nfo_out_size(H, stride), Wo = nfo_out_size(W, stride);
#pragma omp parallel for collapse(2) schedule(static)
  for (int co = 0; co < Cout; ++co)
    for (int ci = 0; ci < Cin; ++ci)
      for (int kh = 0; kh < 3; ++kh)
        for (int kw = 0; kw < 3; ++kw) {
          double acc = 0.0;
          for (int n = 0; n < N; ++n)
            for (int i = 0; i < Ho; ++i)
              for (int j = 0; j < Wo; ++j) {
                const int ii = i * stride + kh - 1, jj = j * stride + kw - 1;
                if (ii < 0 || ii >= H || jj < 0 || jj >= W) continue;
                acc += g[IDX4(n, co, i, j, Cout, Ho, Wo)] * x[IDX4(n, ci, ii, jj, Cin, H, W)];
              }
          dw[(((size_t)co * Cin + ci) * 3 + kh) * 3 + kw] = acc;
        }
}

/* Derivative of the convolution with respect to its input (used for the aux conv only:
 * the main conv's input receives no gradient, the paper's "no feedback" property).
 * dx[n,ci,ii,jj] = sum over (co,i,j,kh,kw) with i*s+kh-1 = ii, j*s+kw-1 = jj of w * g. */
void nfo_conv3x3_dgrad(const double* w, int Cin, int Cout, const double* g, int N, int H, int W,
                       int stride, double* dx) {
  const int Ho = nfo_out_size(H, stride), Wo = nfo_out_size(W, stride);
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int ci = 0; ci < Cin; ++ci)
      for (int ii = 0; ii < H; ++ii)
        for (int jj = 0; jj < W; ++jj) {
          double acc = 0.0;
          for (int co = 0; co < Cout; ++co)
            for (int kh = 0; kh < 3; ++kh)
              for (int kw = 0; kw < 3; ++kw) {
                const int a = ii - kh + 1, b = jj - kw + 1;
                if (a < 0 || b < 0 || a % stride || b % stride) continue;
                const int i = a / stride, j = b / stride;
                if (i >= Ho || j >= Wo) continue;
                acc += w[(((size_t)co * Cin + ci) * 3 + kh) * 3 + kw] * g[IDX4(n, co, i, j, Cout, Ho, Wo)];
              }
          dx[IDX4(n, ci, ii, jj, Cin, H, W)] = acc;
        }
}

/* Batch normalisation with batch statistics: per channel mean and biased variance over
 * (n,i,j); xhat = (y-mu)/sqrt(var+eps); z = gamma*xhat + beta. */
void nfo_bn_train(const double* y, int N, int C, int HW, const double* gamma, const double* beta,
                  double eps, double* mu, double* var, double* xhat, double* z) {
  const double M = (double)N * HW;
#pragma omp parallel for schedule(static)
  for (int c = 0; c < C; ++c) {
    double s = 0.0;
    for (int n = 0; n < N; ++n)
      for (int k = 0; k < HW; ++k) s += y[((size_t)n * C + c) * HW + k];
    const double m = s / M;
    double q = 0.0;
    for (int n = 0; n < N; ++n)
      for (int k = 0; k < HW; ++k) {
        const double d = y[((size_t)n * C + c) * HW + k] - m;
        q += d * d;
      }
    const double v = q / M;
    mu[c] = m;
    var[c] = v;
    const double r = 1.0 / sqrt(v + eps);
    for (int n = 0; n < N; ++n)
      for (int k = 0; k < HW; ++k) {
        const size_t o = ((size_t)n * C + c) * HW + k;
        const double xh = (y[o] - m) * r;
        xhat[o] = xh;
        z[o] = gamma[c] * xh + beta[c];
      }
  }
}

/* Eval-mode normalisation with given (running) statistics. */
void nfo_bn_eval(const double* y, int N, int C, int HW, const double* gamma, const double* beta,
                 double eps, const double* rmean, const double* rvar, double* z) {
#pragma omp parallel for schedule(static)
  for (int c = 0; c < C; ++c) {
    const double r = 1.0 / sqrt(rvar[c] + eps);
    for (int n = 0; n < N; ++n)
      for (int k = 0; k < HW; ++k) {
        const size_t o = ((size_t)n * C + c) * HW + k;
        z[o] = gamma[c] * (y[o] - rmean[c]) * r + beta[c];
      }
  }
}

/* alpha in Eq. 1. */
void nfo_relu(const double* z, size_t n, double* r) {
  for (size_t k = 0; k < n; ++k) r[k] = z[k] > 0.0 ? z[k] : 0.0;
}

/* P_n in Eq. 1 for VGG-shaped nets: 2x2 max-pool, stride 2.  argmax holds, per output,
 * the flat position 2*di+dj (di,dj in {0,1}) of the first maximum in row-major scan order. */
void nfo_maxpool2(const double* r, int N, int C, int H, int W, double* a, int32_t* argmax) {
  const int Hp = H / 2, Wp = W / 2;
  for (int n = 0; n < N; ++n)
    for (int c = 0; c < C; ++c)
      for (int i = 0; i < Hp; ++i)
        for (int j = 0; j < Wp; ++j) {
          double best = r[IDX4(n, c, 2 * i, 2 * j, C, H, W)];
          int32_t arg = 0;
          for (int di = 0; di < 2; ++di)
            for (int dj = 0; dj < 2; ++dj) {
              const double v = r[IDX4(n, c, 2 * i + di, 2 * j + dj, C, H, W)];
              if (v > best) { best = v; arg = 2 * di + dj; }
            }
          a[IDX4(n, c, i, j, C, Hp, Wp)] = best;
          argmax[IDX4(n, c, i, j, C, Hp, Wp)] = arg;
        }
}

/* F_n in Eq. 2: adaptive average pooling to 2x2.  Bin u covers rows
 * [floor(u*H/2), ceil((u+1)*H/2)), the same for columns. */
static void bin_range(int u, int H, int* lo, int* hi) {
  *lo = (u * H) / 2;
  *hi = ((u + 1) * H + 1) / 2;
}

void nfo_avgpool_2x2(const double* h, int N, int F, int H, int W, double* p) {
  for (int n = 0; n < N; ++n)
    for (int f = 0; f < F; ++f)
      for (int u = 0; u < 2; ++u)
        for (int v = 0; v < 2; ++v) {
          int i0, i1, j0, j1;
          bin_range(u, H, &i0, &i1);
          bin_range(v, W, &j0, &j1);
          double s = 0.0;
          for (int i = i0; i < i1; ++i)
            for (int j = j0; j < j1; ++j) s += h[IDX4(n, f, i, j, F, H, W)];
          p[(((size_t)n * F + f) * 2 + u) * 2 + v] = s / (double)((i1 - i0) * (j1 - j0));
        }
}

/* Backward of the adaptive average pool: every element of a bin receives dp/|bin|;
 * an element that lies in two bins (odd sizes) receives both shares. */
void nfo_avgpool_2x2_bwd(const double* dp, int N, int F, int H, int W, double* dh) {
  memset(dh, 0, sizeof(double) * (size_t)N * F * H * W);
  for (int n = 0; n < N; ++n)
    for (int f = 0; f < F; ++f)
      for (int u = 0; u < 2; ++u)
        for (int v = 0; v < 2; ++v) {
          int i0, i1, j0, j1;
          bin_range(u, H, &i0, &i1);
          bin_range(v, W, &j0, &j1);
          const double g = dp[(((size_t)n * F + f) * 2 + u) * 2 + v] / (double)((i1 - i0) * (j1 - j0));
          for (int i = i0; i < i1; ++i)
            for (int j = j0; j < j1; ++j) dh[IDX4(n, f, i, j, F, H, W)] += g;
        }
}

/* F_n of Eq. 2 as adaptive MAX pooling to 2x2 (the paper names max or average pooling): the same bins as the
 * average pool; arg receives the position i*W+j of the first maximum of each bin in row-major scan order. */
void nfo_maxpool_2x2_adaptive(const double* h, int N, int F, int H, int W, double* p, int32_t* arg) {
  for (int n = 0; n < N; ++n)
    for (int f = 0; f < F; ++f)
      for (int u = 0; u < 2; ++u)
        for (int v = 0; v < 2; ++v) {
          int i0, i1, j0, j1;
          bin_range(u, H, &i0, &i1);
          bin_range(v, W, &j0, &j1);
          double m = h[IDX4(n, f, i0, j0, F, H, W)];
          int32_t at = i0 * W + j0;
          for (int i = i0; i < i1; ++i)
            for (int j = j0; j < j1; ++j) {
              const double t = h[IDX4(n, f, i, j, F, H, W)];
              if (t > m) { m = t; at = i * W + j; }
            }
          const size_t o = (((size_t)n * F + f) * 2 + u) * 2 + v;
          p[o] = m;
          arg[o] = at;
        }
}

/* Its backward: the whole of dp goes to the element that was the maximum of the bin; an element that is the
 * maximum of two overlapping bins (odd sizes) receives both. */
void nfo_maxpool_2x2_adaptive_bwd(const double* dp, const int32_t* arg, int N, int F, int H, int W, double* dh) {
  memset(dh, 0, sizeof(double) * (size_t)N * F * H * W);
  for (int n = 0; n < N; ++n)
    for (int f = 0; f < F; ++f)
      for (int b = 0; b < 4; ++b) {
        const size_t o = ((size_t)n * F + f) * 4 + b;
        dh[((size_t)n * F + f) * H * W + arg[o]] += dp[o];
      }
}

/* gamma_n in Eq. 2: logits[n,k] = bf[k] + sum_d Wf[k,d] * p[n,d]. */
void nfo_fc(const double* p, int N, int D, const double* Wf, const double* bf, int K, double* logits) {
  for (int n = 0; n < N; ++n)
    for (int k = 0; k < K; ++k) {
      double s = bf[k];
      for (int d = 0; d < D; ++d) s += Wf[(size_t)k * D + d] * p[(size_t)n * D + d];
      logits[(size_t)n * K + k] = s;
    }
}

/* Eq. 3 with the cross-entropy loss: L = (1/N) sum_n [ logsumexp(logits_n) - logits_n[y_n] ],
 * and its derivative dlogits = (softmax - onehot)/N.  dlogits may be NULL. */
double nfo_softmax_ce(const double* logits, const int32_t* labels, int N, int K, double* dlogits) {
  double loss = 0.0;
  for (int n = 0; n < N; ++n) {
    const double* l = logits + (size_t)n * K;
    double m = l[0];
    for (int k = 1; k < K; ++k) if (l[k] > m) m = l[k];
    double s = 0.0;
    for (int k = 0; k < K; ++k) s += exp(l[k] - m);
    const double lse = m + log(s);
    loss += lse - l[labels[n]];
    if (dlogits)
      for (int k = 0; k < K; ++k)
        dlogits[(size_t)n * K + k] = (exp(l[k] - lse) - (k == labels[n] ? 1.0 : 0.0)) / (double)N;
  }
  return loss / (double)N;
}

/* Eq. 3 with the mean-squared-error loss against one-hot targets t: L = (1/(N K)) sum_{n,k} (logits - t)^2,
 * dlogits = 2 (logits - t) / (N K).  dlogits may be NULL. */
double nfo_mse_onehot(const double* logits, const int32_t* labels, int N, int K, double* dlogits) {
  double loss = 0.0;
  const double inv = 1.0 / ((double)N * (double)K);
  for (int n = 0; n < N; ++n)
    for (int k = 0; k < K; ++k) {
      const double e = logits[(size_t)n * K + k] - (k == labels[n] ? 1.0 : 0.0);
      loss += e * e;
      if (dlogits) dlogits[(size_t)n * K + k] = 2.0 * e * inv;
    }
  return loss * inv;
}

/* Backward of train-mode BatchNorm.  With M = N*HW:
 * dbeta = sum dz ; dgamma = sum dz*xhat ;
 * dy = gamma/sqrt(var+eps) * (dz - dbeta/M - xhat*dgamma/M). */
void nfo_bn_bwd(const double* dz, const double* xhat, int N, int C, int HW, const double* gamma,
                const double* var, double eps, double* dgamma, double* dbeta, double* dy) {
  const double M = (double)N * HW;
#pragma omp parallel for schedule(static)
  for (int c = 0; c < C; ++c) {
    double sb = 0.0, sg = 0.0;
    for (int n = 0; n < N; ++n)
      for (int k = 0; k < HW; ++k) {
        const size_t o = ((size_t)n * C + c) * HW + k;
        sb += dz[o];
        sg += dz[o] * xhat[o];
      }
    dbeta[c] = sb;
    dgamma[c] = sg;
    const double r = gamma[c] / sqrt(var[c] + eps);
    for (int n = 0; n < N; ++n)
      for (int k = 0; k < HW; ++k) {
        const size_t o = ((size_t)n * C + c) * HW + k;
        dy[o] = r * (dz[o] - sb / M - xhat[o] * sg / M);
      }
  }
}

/* Algorithm 2, update step, with momentum: v <- mu*v + g ; theta <- theta - lr*v. */
void nfo_sgd(double* theta, double* v, const double* g, size_t n, double lr, double mu) {
  for (size_t k = 0; k < n; ++k) {
    v[k] = mu * v[k] + g[k];
    theta[k] -= lr * v[k];
  }
}

typedef struct {
  int N, Cin, Cout, H, W, stride, pool, F, classes;
  double eps, momentum, bn_momentum;
  int store_bf16; /* 1: bf16 configuration ("bf16 operands, wider accumulate").  The two tensors the method keeps
                     in bfloat16 (conv output y, activation x_{n+1}) are rounded to bfloat16 where they are
                     stored, so that every decision taken from them (ReLU masks, pool argmax) is taken in the
                     storage precision, and the two convolutions read bfloat16 copies of their weights W and
                     Wa (the master weights, their momentum and their update stay unrounded; the gradient of
                     the copy is applied to the master).  All arithmetic stays fp64. */
  int loss;       /* the loss of Eq. 3: 0 = cross entropy, 1 = mean squared error against one-hot targets */
  int aux_pool;   /* F_n of Eq. 2: 0 = adaptive average pool to 2x2, 1 = adaptive max pool to 2x2.  In the bf16
                     configuration the auxiliary activation h is then rounded to bfloat16 where it is stored, so that
                     the arg-max of a bin is decided among the stored values. */
  const double* skip; /* NULL, or an identity shortcut of a residual network: a tensor of the shape of the BatchNorm
                     output that is added before the ReLU, x_{n+1} = P(ReLU(BN(theta_n x_n) + skip)).  It comes from an
                     earlier layer and carries no gradient (training is local to the layer). */
} nfo_dims;

/* Round to the nearest bfloat16, ties to even (via float, as a bf16 store of an fp32 value does). */
double nfo_round_bf16(double v) {
  float f = (float)v;
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7f800000u) == 0x7f800000u) return (double)f; /* inf / nan unchanged */
  u = (u + 0x7fffu + ((u >> 16) & 1u)) & 0xffff0000u;
  memcpy(&f, &u, 4);
  return (double)f;
}
static void store_round(double* a, size_t n, int on) {
  if (on) for (size_t k = 0; k < n; ++k) a[k] = nfo_round_bf16(a[k]);
}

/* Parameters and optimiser state of one layer with its auxiliary head; updated in place. */
typedef struct {
  double *W, *gamma, *beta, *Wa, *ba, *Wf, *bf;        /* theta_n (W,gamma,beta), beta_n (Wa,ba), gamma_n (Wf,bf) */
  double *vW, *vgamma, *vbeta, *vWa, *vba, *vWf, *vbf; /* momentum buffers */
  double *rmean, *rvar;                                /* running statistics */
} nfo_params;

/* Optional copies of every intermediate; any pointer may be NULL. */
typedef struct {
  double *y, *mu, *var, *xhat, *z, *a, *h, *p, *logits, *dlogits, *dp, *dh, *da, *dz, *dy;
  double *gW, *ggamma, *gbeta, *gWa, *gba, *gWf, *gbf;
  int32_t* argmax;
} nfo_trace;

static double* dalloc(size_t n) { return (double*)calloc(n ? n : 1, sizeof(double)); }
static void keep(double* dst, const double* src, size_t n) {
  if (dst) memcpy(dst, src, n * sizeof(double));
}

/* One pass of the inner body of Algorithm 2 for one layer on one batch:
 * forward (Eq. 1), auxiliary prediction (Eq. 2), loss (Eq. 3), gradients of
 * (theta_n, beta_n, gamma_n), update.  act_out receives x_{n+1} computed with the
 * weights as they were BEFORE the update.  update = 0 computes everything but
 * leaves parameters, momentum and running statistics untouched.  Returns the loss. */
double nfo_layer_step(const nfo_dims* d, const double* x, const int32_t* labels, double lr,
                      nfo_params* P, double* act_out, nfo_trace* T, int update) {
  const int N = d->N, Ci = d->Cin, Co = d->Cout, H = d->H, W = d->W, s = d->stride, F = d->F, K = d->classes;
  const int Ho = nfo_out_size(H, s), Wo = nfo_out_size(W, s);
  const int Ha = d->pool ? Ho / 2 : Ho, Wa = d->pool ? Wo / 2 : Wo;
  const size_t ny = (size_t)N * Co * Ho * Wo, na = (size_t)N * Co * Ha * Wa, nh = (size_t)N * F * Ha * Wa;
  const int D = 4 * F;

  double *y = dalloc(ny), *xhat = dalloc(ny), *z = dalloc(ny), *r = dalloc(ny), *a = dalloc(na);
  double *mu = dalloc(Co), *var = dalloc(Co);
  int32_t* arg = (int32_t*)calloc(na, sizeof(int32_t));
  double *hpre = dalloc(nh), *h = dalloc(nh), *p = dalloc((size_t)N * D), *logits = dalloc((size_t)N * K);
  double *dlogits = dalloc((size_t)N * K), *dp = dalloc((size_t)N * D), *dh = dalloc(nh), *da = dalloc(na);
  double *dr = dalloc(ny), *dz = dalloc(ny), *dy = dalloc(ny);
  double *gW = dalloc((size_t)Co * Ci * 9), *gg = dalloc(Co), *gb = dalloc(Co);
  double *gWa = dalloc((size_t)F * Co * 9), *gba = dalloc(F), *gWf = dalloc((size_t)K * D), *gbf = dalloc(K);

  /* operand copies of the conv weights (bfloat16 in the bf16 configuration) */
  double *Wq = dalloc((size_t)Co * Ci * 9), *Waq = dalloc((size_t)F * Co * 9);
  memcpy(Wq, P->W, sizeof(double) * (size_t)Co * Ci * 9);
  memcpy(Waq, P->Wa, sizeof(double) * (size_t)F * Co * 9);
  store_round(Wq, (size_t)Co * Ci * 9, d->store_bf16);
  store_round(Waq, (size_t)F * Co * 9, d->store_bf16);

  /* forward: Eq. 1 */
  nfo_conv3x3(x, N, Ci, H, W, Wq, Co, NULL, s, y);
  store_round(y, ny, d->store_bf16);
  nfo_bn_train(y, N, Co, Ho * Wo, P->gamma, P->beta, d->eps, mu, var, xhat, z);
  if (d->skip)
    for (size_t k = 0; k < ny; ++k) z[k] += d->skip[k];
  nfo_relu(z, ny, r);
  store_round(r, ny, d->store_bf16); /* rounding is monotone: pooling rounded values = rounding the pooled value */
  if (d->pool) nfo_maxpool2(r, N, Co, Ho, Wo, a, arg);
  else memcpy(a, r, ny * sizeof(double));
  if (act_out) memcpy(act_out, a, na * sizeof(double));
  /* auxiliary network: Eq. 2 */
  nfo_conv3x3(a, N, Co, Ha, Wa, Waq, F, P->ba, 1, hpre);
  nfo_relu(hpre, nh, h);
  int32_t* parg = (int32_t*)calloc((size_t)N * D, sizeof(int32_t));
  if (d->aux_pool == 1) {
    store_round(h, nh, d->store_bf16);
    nfo_maxpool_2x2_adaptive(h, N, F, Ha, Wa, p, parg);
  } else {
    nfo_avgpool_2x2(h, N, F, Ha, Wa, p);
  }
  nfo_fc(p, N, D, P->Wf, P->bf, K, logits);
  /* loss: Eq. 3 */
  const double loss = d->loss == 1 ? nfo_mse_onehot(logits, labels, N, K, dlogits) : nfo_softmax_ce(logits, labels, N, K, dlogits);

  /* gradients of gamma_n: dWf = dlogits^T p ; dbf = sum_n dlogits ; dp = dlogits Wf */
  for (int k = 0; k < K; ++k) {
    double sb = 0.0;
    for (int n = 0; n < N; ++n) sb += dlogits[(size_t)n * K + k];
    gbf[k] = sb;
    for (int j = 0; j < D; ++j) {
      double sw = 0.0;
      for (int n = 0; n < N; ++n) sw += dlogits[(size_t)n * K + k] * p[(size_t)n * D + j];
      gWf[(size_t)k * D + j] = sw;
    }
  }
  for (int n = 0; n < N; ++n)
    for (int j = 0; j < D; ++j) {
      double sp = 0.0;
      for (int k = 0; k < K; ++k) sp += dlogits[(size_t)n * K + k] * P->Wf[(size_t)k * D + j];
      dp[(size_t)n * D + j] = sp;
    }
  /* gradients of beta_n */
  if (d->aux_pool == 1) nfo_maxpool_2x2_adaptive_bwd(dp, parg, N, F, Ha, Wa, dh);
  else nfo_avgpool_2x2_bwd(dp, N, F, Ha, Wa, dh);
  free(parg);
  for (size_t k = 0; k < nh; ++k) if (!(hpre[k] > 0.0)) dh[k] = 0.0;
  nfo_conv3x3_wgrad(a, N, Co, Ha, Wa, dh, F, 1, gWa);
  for (int f = 0; f < F; ++f) {
    double sb = 0.0;
    for (int n = 0; n < N; ++n)
      for (int k = 0; k < Ha * Wa; ++k) sb += dh[((size_t)n * F + f) * Ha * Wa + k];
    gba[f] = sb;
  }
  nfo_conv3x3_dgrad(Waq, Co, F, dh, N, Ha, Wa, 1, da);
  /* back through down-sampling and ReLU to the BatchNorm output */
  if (d->pool) {
    for (int n = 0; n < N; ++n)
      for (int c = 0; c < Co; ++c)
        for (int i = 0; i < Ha; ++i)
          for (int j = 0; j < Wa; ++j) {
            const int32_t g = arg[IDX4(n, c, i, j, Co, Ha, Wa)];
            dr[IDX4(n, c, 2 * i + g / 2, 2 * j + g % 2, Co, Ho, Wo)] = da[IDX4(n, c, i, j, Co, Ha, Wa)];
          }
  } else {
    memcpy(dr, da, ny * sizeof(double));
  }
  for (size_t k = 0; k < ny; ++k) dz[k] = z[k] > 0.0 ? dr[k] : 0.0;
  /* gradients of theta_n; the layer input x receives none */
  nfo_bn_bwd(dz, xhat, N, Co, Ho * Wo, P->gamma, var, d->eps, gg, gb, dy);
  nfo_conv3x3_wgrad(x, N, Ci, H, W, dy, Co, s, gW);

  if (T) {
    keep(T->y, y, ny); keep(T->mu, mu, Co); keep(T->var, var, Co); keep(T->xhat, xhat, ny); keep(T->z, z, ny);
    keep(T->a, a, na); keep(T->h, h, nh); keep(T->p, p, (size_t)N * D); keep(T->logits, logits, (size_t)N * K);
    keep(T->dlogits, dlogits, (size_t)N * K); keep(T->dp, dp, (size_t)N * D); keep(T->dh, dh, nh);
    keep(T->da, da, na); keep(T->dz, dz, ny); keep(T->dy, dy, ny);
    keep(T->gW, gW, (size_t)Co * Ci * 9); keep(T->ggamma, gg, Co); keep(T->gbeta, gb, Co);
    keep(T->gWa, gWa, (size_t)F * Co * 9); keep(T->gba, gba, F); keep(T->gWf, gWf, (size_t)K * D);
    keep(T->gbf, gbf, K);
    if (T->argmax) memcpy(T->argmax, arg, na * sizeof(int32_t));
  }

  if (update) {
    nfo_sgd(P->W, P->vW, gW, (size_t)Co * Ci * 9, lr, d->momentum);
    nfo_sgd(P->gamma, P->vgamma, gg, Co, lr, d->momentum);
    nfo_sgd(P->beta, P->vbeta, gb, Co, lr, d->momentum);
    nfo_sgd(P->Wa, P->vWa, gWa, (size_t)F * Co * 9, lr, d->momentum);
    nfo_sgd(P->ba, P->vba, gba, F, lr, d->momentum);
    nfo_sgd(P->Wf, P->vWf, gWf, (size_t)K * D, lr, d->momentum);
    nfo_sgd(P->bf, P->vbf, gbf, K, lr, d->momentum);
    const double M = (double)N * Ho * Wo;
    for (int c = 0; c < Co; ++c) {
      P->rmean[c] = (1.0 - d->bn_momentum) * P->rmean[c] + d->bn_momentum * mu[c];
      P->rvar[c] = (1.0 - d->bn_momentum) * P->rvar[c] + d->bn_momentum * var[c] * M / (M - 1.0);
    }
  }

  free(Wq); free(Waq);
  free(y); free(xhat); free(z); free(r); free(a); free(mu); free(var); free(arg);
  free(hpre); free(h); free(p); free(logits); free(dlogits); free(dp); free(dh); free(da);
  free(dr); free(dz); free(dy); free(gW); free(gg); free(gb); free(gWa); free(gba); free(gWf); free(gbf);
  return loss;
}

/* Eval-mode forward of one layer (what the activation cache stores for a trained block):
 * conv, normalisation with running statistics, ReLU, optional 2x2 max-pool. */
void nfo_layer_eval(const nfo_dims* d, const double* x, const nfo_params* P, double* out) {
  const int N = d->N, Co = d->Cout, s = d->stride;
  const int Ho = nfo_out_size(d->H, s), Wo = nfo_out_size(d->W, s);
  const size_t ny = (size_t)N * Co * Ho * Wo;
  double *y = dalloc(ny), *z = dalloc(ny), *r = dalloc(ny);
  double* Wq = dalloc((size_t)Co * d->Cin * 9);
  memcpy(Wq, P->W, sizeof(double) * (size_t)Co * d->Cin * 9);
  store_round(Wq, (size_t)Co * d->Cin * 9, d->store_bf16);
  nfo_conv3x3(x, N, d->Cin, d->H, d->W, Wq, Co, NULL, s, y);
  free(Wq);
  store_round(y, ny, d->store_bf16);
  nfo_bn_eval(y, N, Co, Ho * Wo, P->gamma, P->beta, d->eps, P->rmean, P->rvar, z);
  if (d->skip)
    for (size_t k = 0; k < ny; ++k) z[k] += d->skip[k];
  nfo_relu(z, ny, r);
  store_round(r, ny, d->store_bf16);
  if (d->pool) {
    int32_t* arg = (int32_t*)calloc(ny / 4 + 1, sizeof(int32_t));
    nfo_maxpool2(r, N, Co, Ho, Wo, out, arg);
    free(arg);
  } else {
    memcpy(out, r, ny * sizeof(double));
  }
  free(y); free(z); free(r);
}

/* Early-exit prediction of one layer (Section "Trained output CNN": every layer with its auxiliary
 * network is a prospective exit).  Forward only, normalisation with the running statistics:
 * act_out = x_{n+1} (Eq. 1), logits = z_{n+1} = gamma_n F_n beta_n x_{n+1} (Eq. 2).  The class is the
 * arg-max of the logits (taken by the caller: first maximum). */
void nfo_layer_predict(const nfo_dims* d, const double* x, const nfo_params* P, double* act_out, double* logits) {
  const int N = d->N, Co = d->Cout, F = d->F, K = d->classes, s = d->stride;
  const int Ho = nfo_out_size(d->H, s), Wo = nfo_out_size(d->W, s);
  const int Ha = d->pool ? Ho / 2 : Ho, Wa = d->pool ? Wo / 2 : Wo;
  const size_t na = (size_t)N * Co * Ha * Wa, nh = (size_t)N * F * Ha * Wa;
  double *a = dalloc(na), *hpre = dalloc(nh), *h = dalloc(nh), *p = dalloc((size_t)N * 4 * F);
  nfo_layer_eval(d, x, P, a);
  double* Waq = dalloc((size_t)F * Co * 9);
  memcpy(Waq, P->Wa, sizeof(double) * (size_t)F * Co * 9);
  store_round(Waq, (size_t)F * Co * 9, d->store_bf16);
  nfo_conv3x3(a, N, Co, Ha, Wa, Waq, F, P->ba, 1, hpre);
  nfo_relu(hpre, nh, h);
  if (d->aux_pool == 1) {
    int32_t* parg = (int32_t*)calloc((size_t)N * 4 * F, sizeof(int32_t));
    store_round(h, nh, d->store_bf16);
    nfo_maxpool_2x2_adaptive(h, N, F, Ha, Wa, p, parg);
    free(parg);
  } else {
    nfo_avgpool_2x2(h, N, F, Ha, Wa, p);
  }
  nfo_fc(p, N, 4 * F, P->Wf, P->bf, K, logits);
  if (act_out) memcpy(act_out, a, na * sizeof(double));
  free(a); free(hpre); free(h); free(p); free(Waq);
}
