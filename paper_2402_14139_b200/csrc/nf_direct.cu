// Generic CUDA-core kernels of the local-layer step: any shape, fp32 or bf16 storage, fp32
// accumulation, deterministic reductions (fixed-order partials, no floating-point atomics).
// They carry the fp32 configuration and every shape the tensor-core kernels do not cover.
#include "nf_internal.h"
#include "nf_ldst.cuh"

namespace {

// ------------------------------------------------------------------ direct 3x3 convolution, pad 1
// y[n,i,j,co] = act(bias[co] + sum_{kh,kw,ci} w(tap,co,ci) * x[n, i*s+kh-1, j*s+kw-1, ci]).
// Weight element (tap,co,ci) sits at w[t*ws_tap + co*ws_co + ci*ws_ci] with t = tap, or 8-tap when
// flip is set (flip + swapped strides turn the same kernel into the input-gradient convolution).
constexpr int CT_P = 16, CT_CO = 16, CT_CI = 32;

template <typename T>
__global__ void __launch_bounds__(256) conv_direct_kernel(const T* __restrict__ x, int N, int H, int W, int Ci,
                                                          const T* __restrict__ w, long ws_tap, long ws_co,
                                                          long ws_ci, int flip, const float* __restrict__ bias,
                                                          int relu, int s, int Co, int Ho, int Wo, T* __restrict__ y) {
  __shared__ float xs[3][CT_P * 2 + 2][CT_CI];
  __shared__ float wsm[9][CT_CO][CT_CI + 1];
  const int wt = (Wo + CT_P - 1) / CT_P, ct = (Co + CT_CO - 1) / CT_CO;
  long b = blockIdx.x;
  const int jt = b % wt; b /= wt;
  const int cot = b % ct; b /= ct;
  const int i = b % Ho;
  const int n = b / Ho;
  const int tid = threadIdx.x, co_l = tid % CT_CO, p_l = tid / CT_CO;
  const int j0 = jt * CT_P, co0 = cot * CT_CO;
  const int cols = (CT_P - 1) * s + 3;
  float acc = 0.f;
  for (int c0 = 0; c0 < Ci; c0 += CT_CI) {
    const int cn = min(CT_CI, Ci - c0);
    for (int e = tid; e < 3 * cols * CT_CI; e += 256) {
      const int c = e % CT_CI, col = (e / CT_CI) % cols, r = e / (CT_CI * cols);
      const int ii = i * s + r - 1, jj = j0 * s + col - 1;
      float v = 0.f;
      if (c < cn && ii >= 0 && ii < H && jj >= 0 && jj < W) v = ldf(x, (((size_t)n * H + ii) * W + jj) * Ci + c0 + c);
      xs[r][col][c] = v;
    }
    for (int e = tid; e < 9 * CT_CO * CT_CI; e += 256) {
      const int c = e % CT_CI, co = (e / CT_CI) % CT_CO, t = e / (CT_CI * CT_CO);
      float v = 0.f;
      if (c < cn && co0 + co < Co)
        v = ldf(w, (size_t)((flip ? 8 - t : t) * ws_tap + (co0 + co) * ws_co + (c0 + c) * ws_ci));
      wsm[t][co][c] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kh = 0; kh < 3; ++kh)
#pragma unroll
      for (int kw = 0; kw < 3; ++kw) {
        const float* xr = xs[kh][p_l * s + kw];
        const float* wr = wsm[kh * 3 + kw][co_l];
#pragma unroll 8
        for (int c = 0; c < CT_CI; ++c) acc = fmaf(xr[c], wr[c], acc);
      }
    __syncthreads();
  }
  const int j = j0 + p_l, co = co0 + co_l;
  if (j < Wo && co < Co) {
    if (bias) acc += bias[co];
    if (relu) acc = fmaxf(acc, 0.f);
    stf(y, (((size_t)n * Ho + i) * Wo + j) * Co + co, acc);
  }
}

// ------------------------------------------------------------------ direct weight gradient
// part[split][tap][co][ci] = sum over the split's (n,i) rows and all j of g[n,i,j,co] * x[n,i*s+kh-1,j*s+kw-1,ci]
constexpr int WG_J = 64;

template <typename T>
__global__ void __launch_bounds__(256) wgrad_direct_kernel(const T* __restrict__ x, int N, int H, int W, int Ci,
                                                           const T* __restrict__ g, int Co, int s, int Ho, int Wo,
                                                           int splits, float* __restrict__ part) {
  __shared__ float gs[WG_J][16];
  __shared__ float xs[3][WG_J * 2 + 2][16];
  const int cit = (Ci + 15) / 16, cot = (Co + 15) / 16;
  int b = blockIdx.x;
  const int ti = b % cit; b /= cit;
  const int to = b % cot; b /= cot;
  const int sp = b;
  const int tid = threadIdx.x, ci_l = tid % 16, co_l = tid / 16;
  const int ci0 = ti * 16, co0 = to * 16;
  const long rows = (long)N * Ho;
  const long r0 = rows * sp / splits, r1 = rows * (sp + 1) / splits;
  float acc[9];
#pragma unroll
  for (int t = 0; t < 9; ++t) acc[t] = 0.f;
  for (long r = r0; r < r1; ++r) {
    const int n = (int)(r / Ho), i = (int)(r % Ho);
    for (int j0 = 0; j0 < Wo; j0 += WG_J) {
      const int jn = min(WG_J, Wo - j0);
      const int cols = (jn - 1) * s + 3;
      for (int e = tid; e < jn * 16; e += 256) {
        const int c = e % 16, j = e / 16;
        gs[j][c] = (co0 + c < Co) ? ldf(g, (((size_t)n * Ho + i) * Wo + j0 + j) * Co + co0 + c) : 0.f;
      }
      for (int e = tid; e < 3 * cols * 16; e += 256) {
        const int c = e % 16, col = (e / 16) % cols, rr = e / (16 * cols);
        const int ii = i * s + rr - 1, jj = j0 * s + col - 1;
        float v = 0.f;
        if (ci0 + c < Ci && ii >= 0 && ii < H && jj >= 0 && jj < W)
          v = ldf(x, (((size_t)n * H + ii) * W + jj) * Ci + ci0 + c);
        xs[rr][col][c] = v;
      }
      __syncthreads();
      for (int j = 0; j < jn; ++j) {
        const float gv = gs[j][co_l];
#pragma unroll
        for (int kh = 0; kh < 3; ++kh)
#pragma unroll
          for (int kw = 0; kw < 3; ++kw) acc[kh * 3 + kw] = fmaf(gv, xs[kh][j * s + kw][ci_l], acc[kh * 3 + kw]);
      }
      __syncthreads();
    }
  }
  if (co0 + co_l < Co && ci0 + ci_l < Ci)
#pragma unroll
    for (int t = 0; t < 9; ++t) part[(((size_t)sp * 9 + t) * Co + co0 + co_l) * Ci + ci0 + ci_l] = acc[t];
}

// out[i] = sum over the splits of part[k][i]: 32 consecutive elements x 8 lanes over the splits per block; a lane adds its
// splits in index order with four loads in flight, the lane sums are added in lane order (fixed order, no atomics)
__global__ void __launch_bounds__(256) sum_splits_kernel(const float* __restrict__ part, int splits, size_t n, float* __restrict__ out) {
  __shared__ float sm[8][33];
  const size_t i = (size_t)blockIdx.x * 32 + threadIdx.x;
  float s = 0.f;
  if (i < n) {
    int k = threadIdx.y;
    for (; k + 3 * 8 < splits; k += 4 * 8) {
      const float a = part[(size_t)k * n + i], b = part[(size_t)(k + 8) * n + i], c = part[(size_t)(k + 16) * n + i],
                  d = part[(size_t)(k + 24) * n + i];
      s += a;
      s += b;
      s += c;
      s += d;
    }
    for (; k < splits; k += 8) s += part[(size_t)k * n + i];
  }
  sm[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0 && i < n) {
    float t = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) t += sm[j][threadIdx.x];
    out[i] = t;
  }
}


// ------------------------------------------------------------------ first-layer kernels (Cin <= 4)
// An RGB input gives a K dimension of only 27: too thin for the tensor cores and, with 6-byte pixels,
// not addressable by TMA.  One thread computes 16 output channels of one pixel from its 3x3xCin patch held
// in registers; weights sit in shared memory and are read as warp-wide broadcasts.
template <typename T> __device__ __forceinline__ void store16(T* dst, const float (&v)[16]);
template <> __device__ __forceinline__ void store16<float>(float* dst, const float (&v)[16]) {
#pragma unroll
  for (int k = 0; k < 4; ++k) reinterpret_cast<float4*>(dst)[k] = make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
}
template <> __device__ __forceinline__ void store16<bf16>(bf16* dst, const float (&v)[16]) {
  uint32_t w[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const __nv_bfloat162 b2 = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
    w[k] = *reinterpret_cast<const uint32_t*>(&b2);
  }
  reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
  reinterpret_cast<uint4*>(dst)[1] = make_uint4(w[4], w[5], w[6], w[7]);
}

template <typename T>
__global__ void __launch_bounds__(256) conv_smallc_kernel(const T* __restrict__ x, int N, int H, int W, int Ci,
                                                          const T* __restrict__ w, int s, int Co, int Ho, int Wo,
                                                          T* __restrict__ y) {
  extern __shared__ float wsm[];  // [tap][ci][co]
  for (int e = threadIdx.y * 32 + threadIdx.x; e < 9 * Ci * Co; e += blockDim.x * blockDim.y) {
    const int co = e % Co, ci = (e / Co) % Ci, t = e / (Co * Ci);
    wsm[e] = ldf(w, ((size_t)t * Co + co) * Ci + ci);
  }
  __syncthreads();
  const size_t P = (size_t)N * Ho * Wo;
  const int co0 = threadIdx.y * 16;
  for (size_t pix = (size_t)blockIdx.x * 32 + threadIdx.x; pix < P; pix += (size_t)gridDim.x * 32) {  // weights loaded once per block
    const int j = (int)(pix % Wo), i = (int)((pix / Wo) % Ho);
    const size_t n = pix / ((size_t)Wo * Ho);
    float patch[36];
#pragma unroll
    for (int t = 0; t < 9; ++t) {
      const int ii = i * s + t / 3 - 1, jj = j * s + t % 3 - 1;
      const bool in = ii >= 0 && ii < H && jj >= 0 && jj < W;
#pragma unroll
      for (int c = 0; c < 4; ++c) patch[t * 4 + c] = (in && c < Ci) ? ldf(x, ((n * H + ii) * W + jj) * Ci + c) : 0.f;
    }
    float acc[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) acc[k] = 0.f;
#pragma unroll
    for (int t = 0; t < 9; ++t)
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (c < Ci) {
          const float xv = patch[t * 4 + c];
          const float4* wr = reinterpret_cast<const float4*>(wsm + (t * Ci + c) * Co + co0);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float4 wv = wr[k];
            acc[4 * k] = fmaf(xv, wv.x, acc[4 * k]);
            acc[4 * k + 1] = fmaf(xv, wv.y, acc[4 * k + 1]);
            acc[4 * k + 2] = fmaf(xv, wv.z, acc[4 * k + 2]);
            acc[4 * k + 3] = fmaf(xv, wv.w, acc[4 * k + 3]);
          }
        }
    store16(y + pix * Co + co0, acc);
  }
}

// part[split][tap][co][ci]: thread (co, lane) sums its 9*Ci products over the pixels lane, lane+4, ... of the
// split's rows; the 3 input rows of an output row are staged in shared memory and read as broadcasts.
template <typename T>
__global__ void __launch_bounds__(512) wgrad_smallc_kernel(const T* __restrict__ x, int N, int H, int W, int Ci,
                                                           const T* __restrict__ g, int Co, int s, int Ho, int Wo,
                                                           int splits, float* __restrict__ part) {
  extern __shared__ float sm[];           // xrow[(R-1)*s + 3][W + 2][4]  then  red[4][Co][36]
  constexpr int R = 4;                    // output rows staged per synchronisation
  const int xr = (R - 1) * s + 3;
  float* xrow = sm;
  float* red = sm + xr * (W + 2) * 4;
  const int co = threadIdx.x, ln = threadIdx.y, tid = ln * blockDim.x + co, nthr = blockDim.x * 4;
  const long rows = (long)N * Ho;
  const long r0 = rows * blockIdx.x / splits, r1 = rows * (blockIdx.x + 1) / splits;
  float acc[36];
#pragma unroll
  for (int k = 0; k < 36; ++k) acc[k] = 0.f;
  for (long r = r0; r < r1;) {
    const int n = (int)(r / Ho), i = (int)(r % Ho);
    int nr = R;
    if (nr > r1 - r) nr = (int)(r1 - r);
    if (nr > Ho - i) nr = Ho - i;          // stay inside one image
    const int need = (nr - 1) * s + 3;
    __syncthreads();
    for (int e = tid; e < need * (W + 2) * 4; e += nthr) {
      const int c = e & 3, col = (e >> 2) % (W + 2), rr = (e >> 2) / (W + 2);
      const int ii = i * s + rr - 1, jj = col - 1;
      xrow[e] = (c < Ci && ii >= 0 && ii < H && jj >= 0 && jj < W) ? ldf(x, (((size_t)n * H + ii) * W + jj) * Ci + c) : 0.f;
    }
    __syncthreads();
    for (int q = 0; q < nr; ++q)
      for (int j = ln; j < Wo; j += 4) {
        const float gv = ldf(g, (((size_t)n * Ho + i + q) * Wo + j) * Co + co);
#pragma unroll
        for (int t = 0; t < 9; ++t) {
          const float4 xv = *reinterpret_cast<const float4*>(xrow + ((q * s + t / 3) * (W + 2) + j * s + t % 3) * 4);
          acc[t * 4 + 0] = fmaf(gv, xv.x, acc[t * 4 + 0]);
          acc[t * 4 + 1] = fmaf(gv, xv.y, acc[t * 4 + 1]);
          acc[t * 4 + 2] = fmaf(gv, xv.z, acc[t * 4 + 2]);
          acc[t * 4 + 3] = fmaf(gv, xv.w, acc[t * 4 + 3]);
        }
      }
    r += nr;
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < 36; ++k) red[(ln * Co + co) * 36 + k] = acc[k];
  __syncthreads();
  if (ln == 0)
    for (int t = 0; t < 9; ++t)
      for (int c = 0; c < Ci; ++c) {
        float v = 0.f;
        for (int q = 0; q < 4; ++q) v += red[(q * Co + co) * 36 + t * 4 + c];
        part[(((size_t)blockIdx.x * 9 + t) * Co + co) * Ci + c] = v;
      }
}

inline bool smallc_ok(int Ci, int Co, int W) { return Ci <= 4 && Co % 16 == 0 && Co <= 128 && W <= 512; }

}  // namespace

int nf_k_conv(int dtype, const void* x, int N, int H, int W, int Ci, const void* w, long ws_tap, long ws_co,
                long ws_ci, int flip, const float* bias, int relu, int stride, int Co, void* y) {
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
  if (smallc_ok(Ci, Co, W) && !flip && !bias && !relu && ws_ci == 1 && ws_co == Ci && ws_tap == (long)Co * Ci) {
    const size_t P = (size_t)N * Ho * Wo;
    const dim3 blk(32, Co / 16);
    const size_t sm = (size_t)9 * Ci * Co * sizeof(float);
    size_t nblk_ = (P + 31) / 32;
    if (nblk_ > 148 * 16) nblk_ = 148 * 16;
    const unsigned grid = (unsigned)nblk_;
    if (dtype == NF_F32)
      conv_smallc_kernel<float><<<grid, blk, sm, g_nf_stream>>>((const float*)x, N, H, W, Ci, (const float*)w,
                                                                                   stride, Co, Ho, Wo, (float*)y);
    else
      conv_smallc_kernel<bf16><<<grid, blk, sm, g_nf_stream>>>((const bf16*)x, N, H, W, Ci, (const bf16*)w,
                                                                                  stride, Co, Ho, Wo, (bf16*)y);
    NF_LAUNCHED();
    return NF_OK;
  }
  const long blocks = (long)N * Ho * ((Wo + CT_P - 1) / CT_P) * ((Co + CT_CO - 1) / CT_CO);
  if (blocks <= 0 || blocks > 0x7fffffffL) return NF_EUNSUPPORTED;
  if (dtype == NF_F32)
    conv_direct_kernel<float><<<(unsigned)blocks, 256, 0, g_nf_stream>>>(
        (const float*)x, N, H, W, Ci, (const float*)w, ws_tap, ws_co, ws_ci, flip, bias, relu, stride, Co, Ho, Wo, (float*)y);
  else
    conv_direct_kernel<bf16><<<(unsigned)blocks, 256, 0, g_nf_stream>>>(
        (const bf16*)x, N, H, W, Ci, (const bf16*)w, ws_tap, ws_co, ws_ci, flip, bias, relu, stride, Co, Ho, Wo, (bf16*)y);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_k_wgrad_splits(int N, int Ho, int Ci, int Co) {
  if (Ci <= 4 && Co % 16 == 0 && Co <= 128) {  // first-layer kernel: one block per slice of rows
    long sp = (long)N * Ho;
    return (int)(sp > 1184 ? 1184 : sp);
  }
  const long tiles = (long)((Ci + 15) / 16) * ((Co + 15) / 16);
  long s = 2368 / tiles;
  if (s < 1) s = 1;
  if (s > (long)N * Ho) s = (long)N * Ho;
  return (int)s;
}

int nf_k_wgrad(int dtype, const void* x, int N, int H, int W, int Ci, const void* g, int Co, int stride,
                 float* part, size_t part_floats, float* dw) {
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
  const int splits = nf_k_wgrad_splits(N, Ho, Ci, Co);
  const size_t n = (size_t)9 * Co * Ci;
  if ((size_t)splits * n > part_floats) return NF_ENOWS;
  if (smallc_ok(Ci, Co, W)) {
    const dim3 blk(Co, 4);
    const size_t sm = ((size_t)(3 * stride + 3) * (W + 2) * 4 + (size_t)4 * Co * 36) * sizeof(float);
    static bool attr_done = false;
    if (!attr_done) {
      NF_CUDA(cudaFuncSetAttribute(wgrad_smallc_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024));
      NF_CUDA(cudaFuncSetAttribute(wgrad_smallc_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024));
      attr_done = true;
    }
    if (dtype == NF_F32)
      wgrad_smallc_kernel<float><<<splits, blk, sm, g_nf_stream>>>((const float*)x, N, H, W, Ci, (const float*)g, Co, stride, Ho, Wo,
                                                                 splits, part);
    else
      wgrad_smallc_kernel<bf16><<<splits, blk, sm, g_nf_stream>>>((const bf16*)x, N, H, W, Ci, (const bf16*)g, Co, stride, Ho, Wo,
                                                                splits, part);
    NF_LAUNCHED();
    sum_splits_kernel<<<(unsigned)((n + 31) / 32), dim3(32, 8), 0, g_nf_stream>>>(part, splits, n, dw);
    NF_LAUNCHED();
    return NF_OK;
  }
  const unsigned blocks = (unsigned)(((Ci + 15) / 16) * ((Co + 15) / 16) * splits);
  if (dtype == NF_F32)
    wgrad_direct_kernel<float><<<blocks, 256, 0, g_nf_stream>>>((const float*)x, N, H, W, Ci, (const float*)g, Co,
                                                                stride, Ho, Wo, splits, part);
  else
    wgrad_direct_kernel<bf16><<<blocks, 256, 0, g_nf_stream>>>((const bf16*)x, N, H, W, Ci, (const bf16*)g, Co,
                                                               stride, Ho, Wo, splits, part);
  NF_LAUNCHED();
  sum_splits_kernel<<<(unsigned)((n + 31) / 32), dim3(32, 8), 0, g_nf_stream>>>(part, splits, n, dw);
  NF_LAUNCHED();
  return NF_OK;
}
