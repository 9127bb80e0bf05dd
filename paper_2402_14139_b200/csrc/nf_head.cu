// The linear head gamma_n of Eq. 2 and the loss of Eq. 3 for LARGE batches (late blocks train at tens of
// thousands of samples, and with 256 auxiliary filters the head input has 1024 features): then
//   logits = p Wf^T + bf,   dp = dlogits Wf,   gWf = dlogits^T p
// are matrix products worth tiling.  fp32 on the CUDA cores (the fp32 configuration's tolerance rules out
// reduced-precision operands); every output element is produced by one thread that adds its products in
// index order, the reduction over the batch in gWf is cut into a fixed number of ranges whose partial results
// are added in range order: results do not depend on scheduling.
#include <algorithm>

#include "nf_internal.h"

namespace {

// C[i][j] (+ z * M * Nn when split) = sum_{k in the z-th range} A[i*sai + k*sak] * B[k*sbk + j*sbj]
// 64 x 64 tile per block of 256 threads, 4 x 4 outputs per thread, 16-deep shared-memory stages.
__global__ void __launch_bounds__(256) head_gemm_kernel(const float* __restrict__ A, long sai, long sak, const float* __restrict__ B,
                                                        long sbk, long sbj, int M, int Nn, int Kd, float* __restrict__ C) {
  __shared__ float As[16][68];
  __shared__ float Bs[16][68];
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  const int i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
  const int Z = gridDim.z, z = blockIdx.z;
  const int k_lo = (int)((long)Kd * z / Z), k_hi = (int)((long)Kd * (z + 1) / Z);
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
  for (int k0 = k_lo; k0 < k_hi; k0 += 16) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int e = t + 256 * r;
      // walk the tile along whichever index is contiguous in memory
      const int ai = sai == 1 ? e % 64 : e / 16, ak = sai == 1 ? e / 64 : e % 16;
      const int bj = sbj == 1 ? e % 64 : e / 16, bk = sbj == 1 ? e / 64 : e % 16;
      As[ak][ai] = (i0 + ai < M && k0 + ak < k_hi) ? A[(long)(i0 + ai) * sai + (long)(k0 + ak) * sak] : 0.f;
      Bs[bk][bj] = (j0 + bj < Nn && k0 + bk < k_hi) ? B[(long)(k0 + bk) * sbk + (long)(j0 + bj) * sbj] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        a[u] = As[kk][ty * 4 + u];
        b[u] = Bs[kk][tx * 4 + u];
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(a[u], b[v], acc[u][v]);
    }
    __syncthreads();
  }
  float* out = C + (size_t)z * M * Nn;
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int i = i0 + ty * 4 + u, j = j0 + tx * 4 + v;
      if (i < M && j < Nn) out[(size_t)i * Nn + j] = acc[u][v];
    }
}

// out[e] = (bias ? bias[e % Nn] : 0) + part[0][e] + part[1][e] + ... in range order
__global__ void head_finish_kernel(const float* __restrict__ part, int Z, size_t mn, int Nn, const float* __restrict__ bias,
                                   float* __restrict__ out) {
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= mn) return;
  float s = bias ? bias[e % Nn] : 0.f;
  for (int z = 0; z < Z; ++z) s += part[(size_t)z * mn + e];
  out[e] = s;
}

// One warp per sample: the loss of Eq. 3 on a row of logits, its derivative dlogits, the per-sample loss.
__global__ void __launch_bounds__(256) head_loss_rows_kernel(const float* __restrict__ logits, const int32_t* __restrict__ labels, int N,
                                                             int K, int loss_kind, float* __restrict__ dlogits,
                                                             float* __restrict__ lossn, int32_t* status, int n_scale) {
  const int n = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (n >= N) return;
  const float* l = logits + (size_t)n * K;
  float* g = dlogits + (size_t)n * K;
  int lab = labels[n];
  if (lab < 0 || lab >= K) {
    if (lane == 0) atomicOr(status, NF_ELABEL);
    lab = lab < 0 ? 0 : K - 1;
  }
  if (loss_kind == 1) {
    float se = 0.f;
    const float sc = 2.f / ((float)n_scale * (float)K);
    for (int k = lane; k < K; k += 32) {
      const float e = l[k] - (k == lab ? 1.f : 0.f);
      se = fmaf(e, e, se);
      g[k] = e * sc;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
    if (lane == 0) lossn[n] = se / (float)K;
    return;
  }
  float mx = -INFINITY;
  for (int k = lane; k < K; k += 32) mx = fmaxf(mx, l[k]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float se = 0.f;
  for (int k = lane; k < K; k += 32) se += expf(l[k] - mx);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
  const float lse = mx + logf(se);
  if (lane == 0) lossn[n] = lse - l[lab];
  const float invN = 1.f / (float)n_scale;
  for (int k = lane; k < K; k += 32) g[k] = (expf(l[k] - lse) - (k == lab ? 1.f : 0.f)) * invN;
}

// part[rb][k] = sum over the rb-th of gridDim.y row ranges of dlogits[n][k] (32 columns x 8 row lanes per block, lanes added in
// order; the ranges are added in range order by head_finish_kernel: with tens of thousands of rows and a few hundred columns
// a single block per 32 columns was the slowest kernel of the head).  Block (0, 0) also reduces the per-sample losses in
// fp64 (256 lanes, then a fixed tree).
__global__ void __launch_bounds__(256) head_colsum_loss_kernel(const float* __restrict__ dl, const float* __restrict__ lossn, int N, int K,
                                                               float* __restrict__ part, float* __restrict__ loss_out, int32_t* status,
                                                               int n_scale) {
  __shared__ float sm[8][33];
  __shared__ double sd[256];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int k = blockIdx.x * 32 + tx;
  const int n0 = (int)((long)N * blockIdx.y / gridDim.y), n1 = (int)((long)N * (blockIdx.y + 1) / gridDim.y);
  float s = 0.f;
  if (k < K)
    for (int n = n0 + ty; n < n1; n += 8) s += dl[(size_t)n * K + k];
  sm[ty][tx] = s;
  __syncthreads();
  if (ty == 0 && k < K) {
    float tsum = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) tsum += sm[j][tx];
    part[(size_t)blockIdx.y * K + k] = tsum;
  }
  if (blockIdx.x == 0 && blockIdx.y == 0) {
    double a = 0.0;
    for (int n = threadIdx.x; n < N; n += 256) a += (double)lossn[n];
    sd[threadIdx.x] = a;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
      if (threadIdx.x < o) sd[threadIdx.x] += sd[threadIdx.x + o];
      __syncthreads();
    }
    if (threadIdx.x == 0) {
      const float L = (float)(sd[0] / (double)n_scale);
      *loss_out = L;
      if (!isfinite(L)) atomicOr(status, NF_ENONFINITE);
    }
  }
}

// first arg-max of each row of logits, one warp per sample
__global__ void __launch_bounds__(256) head_argmax_rows_kernel(const float* __restrict__ logits, int N, int K, int32_t* __restrict__ pred) {
  const int n = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (n >= N) return;
  const float* l = logits + (size_t)n * K;
  float best = -INFINITY;
  int arg = 0x7fffffff;
  for (int k = lane; k < K; k += 32)
    if (l[k] > best) { best = l[k]; arg = k; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ob = __shfl_xor_sync(0xffffffffu, best, o);
    const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
    if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
  }
  if (lane == 0) pred[n] = arg;
}

int gemm(const float* A, long sai, long sak, const float* B, long sbk, long sbj, int M, int Nn, int Kd, int Z, float* C) {
  dim3 grid((Nn + 63) / 64, (M + 63) / 64, Z);
  head_gemm_kernel<<<grid, 256, 0, g_nf_stream>>>(A, sai, sak, B, sbk, sbj, M, Nn, Kd, C);
  NF_LAUNCHED();
  return NF_OK;
}

}  // namespace

bool nf_head_is_large(int N, int D, int K) { return (double)N * D * K >= (double)(1 << 24); }

int nf_head_logits(const float* p, int N, int D, int K, const float* Wf, const float* bf, float* logits, float* scratch) {
  // logits[n][k] = bf[k] + sum_d p[n][d] Wf[k][d]
  int rc = gemm(p, D, 1, Wf, 1, D, N, K, D, 1, scratch);
  if (rc != NF_OK) return rc;
  const size_t mn = (size_t)N * K;
  head_finish_kernel<<<(unsigned)((mn + 255) / 256), 256, 0, g_nf_stream>>>(scratch, 1, mn, K, bf, logits);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_head_predict(const float* logits, int N, int K, int32_t* pred) {
  head_argmax_rows_kernel<<<(N + 7) / 8, 256, 0, g_nf_stream>>>(logits, N, K, pred);
  NF_LAUNCHED();
  return NF_OK;
}

size_t nf_head_scratch_floats(int N, int D, int K) {
  const size_t a = (size_t)N * K, b = (size_t)K * D;  // logits before the bias; at least one range of gWf
  return a > b ? a : b;
}

int nf_head_step(const float* p, const int32_t* labels, int N, int D, int K, const float* Wf, const float* bf, float* logits,
                 float* dlogits, float* dp, float* lossn, int32_t* status, int loss_kind, float* gWf, float* gbf, float* loss_out,
                 float* scratch, size_t scratch_floats, int n_scale) {
  if (scratch_floats < nf_head_scratch_floats(N, D, K)) return NF_ENOWS;
  int rc = nf_head_logits(p, N, D, K, Wf, bf, logits, scratch);
  if (rc != NF_OK) return rc;
  head_loss_rows_kernel<<<(N + 7) / 8, 256, 0, g_nf_stream>>>(logits, labels, N, K, loss_kind, dlogits, lossn, status, n_scale);
  NF_LAUNCHED();
  // dp[n][d] = sum_k dlogits[n][k] Wf[k][d]
  if ((rc = gemm(dlogits, K, 1, Wf, D, 1, N, D, K, 1, dp)) != NF_OK) return rc;
  // gWf[k][d] = sum_n dlogits[n][k] p[n][d], the batch cut into Z ranges
  const size_t kd = (size_t)K * D;
  int Z = (int)std::min<size_t>(scratch_floats / kd, 64);
  const int tiles = ((D + 63) / 64) * ((K + 63) / 64);
  Z = std::min(Z, std::max(1, 592 / tiles));  // about four blocks per SM
  Z = std::min(Z, std::max(1, N / 256));
  if (Z < 1) Z = 1;
  if ((rc = gemm(dlogits, 1, K, p, D, 1, K, D, N, Z, scratch)) != NF_OK) return rc;
  head_finish_kernel<<<(unsigned)((kd + 255) / 256), 256, 0, g_nf_stream>>>(scratch, Z, kd, D, nullptr, gWf);
  NF_LAUNCHED();
  // gbf[k] = sum_n dlogits[n][k]: row ranges in parallel (the scratch is free again), then the ranges in order
  int RB = std::max(1, std::min(64, N / 128));
  if ((size_t)RB * K > scratch_floats) RB = 1;
  head_colsum_loss_kernel<<<dim3((K + 31) / 32, RB), 256, 0, g_nf_stream>>>(dlogits, lossn, N, K, scratch, loss_out, status, n_scale);
  NF_LAUNCHED();
  head_finish_kernel<<<(unsigned)((K + 255) / 256), 256, 0, g_nf_stream>>>(scratch, RB, (size_t)K, K, nullptr, gbf);
  NF_LAUNCHED();
  return NF_OK;
}
