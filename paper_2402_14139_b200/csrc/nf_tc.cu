// Tensor-core convolution kernels for sm_100a: implicit GEMM on tcgen05.mma with accumulators in
// tensor memory, operands staged in shared memory by TMA, warp-specialised persistent CTAs.
//
// Forward (Eq. 1's theta_n x_n, stride 1, Cin and Cout multiples of 64):
//   GEMM view  D[pixel, co] = sum_{tap, ci} X[pixel shifted by tap, ci] * W[tap][co][ci]
//   M tile = 128 output pixels = a BW x BH patch of one image, N tile = BN output channels,
//   K loop  = (Cin/64 channel chunks) x (3 column taps kw); for each such step ONE TMA box of
//   (BH+2) rows x BW pixels x 64 channels lands in shared memory (zero fill outside the image is
//   the padding) and serves the three row taps kh = 0,1,2 by advancing the operand descriptor by
//   kh rows, so the input is fetched 3(BH+2)/BH times from L2 instead of 9 times.
//   Epilogue: TMEM -> registers -> bf16 -> swizzled shared tile -> TMA store of y; the per-channel
//   sum and sum of squares of the stored (rounded) values are accumulated per CTA for BatchNorm.
#include <cuda.h>

#include "nf_ptx.cuh"
#include "nf_tc.h"

namespace {

constexpr int kThreads = 192;  // warp 0: TMA producer, warp 1: MMA issuer + TMEM owner, warps 2-5: epilogue
constexpr int kMaxStages = 8;
// normalisation threads of the fused BatchNorm + aux forward: two groups of 128 that take the stages in turn.  A single group
// was the slowest role of the kernel (busy 2350 of every 2450 cycles per tile while the issuer waited 520 on it: one warp per
// scheduler cannot hide the latency of its load - arithmetic - store - fence chain).  Splitting the ten rows of ONE box over
// two groups had measured slower (0.25 -> 0.27 ms); alternating whole stages gives each group twice the time per box.  Three
// groups measured slower again (aux forward 0.637 -> 0.681 ms over the c4 block): the tensor-core instructions stretch with
// every warp that works on shared memory.
constexpr int kXfGroups = 2;
constexpr int kXfThreads = 128 * kXfGroups;
constexpr int kFoldThreads = 320;  // folded-tap forward: producer, MMA issuer and two epilogue groups of four warps
// Tiles of y2 (the conv output read beside the input gradient, stats >= 2) in flight per CTA.  A slot turns over once per
// load latency plus epilogue time, so with the earlier two slots per epilogue group the kernel ran at the pace of these loads
// (about four tiles per HBM round trip) whatever else it did; with five the loads run as far ahead as the operand stages.
constexpr int kYSlots = 5;

struct FwdParams {
  int N, H, W, Cin, Cout;
  int BW, BH, tiles_w, tiles_h, n_tiles, total_tiles, kchunks, stages;
  int stride, BI;     // PT mode: conv stride and images per tile (BW*BH*BI = 128)
  int stats;
  float* red;         // [grid * parts][2][Cout] channel partials (pre-zeroed)
  int32_t* status;    // device status word
  const float* bias;  // EPI 1: per-channel bias added before the ReLU
  bf16* out;          // EPI 1: destination [N][H][W][Cout], written straight from registers
  // stats == 2 (EPI 0): the output is the gradient da at a BatchNorm+ReLU output of the same shape; the partial sums are
  // (dz, dz * xhat) with dz = da * 1[y2*scale+shift > 0], and the tiles of y2 come through tm_y2
  const float *bn_scale, *bn_shift, *bn_mu, *bn_invstd;
  CUtensorMap tm_y2;
};

struct TcPlan {
  int ok, BW, BH, BI, PT, BN, KC, RW, stages, grid, parts;
  size_t smem;
};

// EPI 0: y in bf16 through a TMA store plus BatchNorm partial sums (BN = 64 or 128).
// EPI 1: bias + ReLU, channels [0, Cout) of a BN-wide tile written directly (aux conv; Cout <= BN <= 64,
//        weight rows beyond Cout are zero-filled by TMA).
// KC  : channels per K chunk of the activation box (64, or 16/32 for the narrow dh tensor of the aux
//       input gradient; rows of 2*KC bytes with the matching TMA swizzle).
// BMN : 0 = weights [tap][co][ci] read K-major (forward); 1 = weights [tap][f][c] read MN-major with the
//       taps mirrored, which makes the same kernel the input-gradient convolution da = dh (*) Wa^T.
// PT  : 1 = one TMA box per tap: stride-2 convolutions (the box is gathered with element stride 2, so the
//       three row taps cannot share a box) and feature maps smaller than a tile, where a tile spans BI whole
//       images (8x8x2, 4x4x8, 2x2x32); p.H, p.W are the OUTPUT sizes.
// RW  : 1 = all nine weight tiles of the CTA's channel tile stay resident in shared memory for the whole
//       kernel (single 64-channel K chunk, 9*BN*128 bytes); the pipeline then carries activations only.
template <int BN, int EPI, int KC = 64, int BMN = 0, int PT = 0, int RW = 0>
__global__ void __launch_bounds__(kThreads, 1)
conv_fwd_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                   const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ FwdParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int kARow = KC * 2;  // bytes of one pixel row of the activation box
  constexpr uint32_t kALayout = KC == 64 ? 2 : KC == 32 ? 4 : 6;
  const int a_bytes = PT ? 128 * kARow : (p.BH + 2) * p.BW * kARow;
  const int a_stride = (a_bytes + 1023) & ~1023;  // keeps the weight tiles 1024-byte aligned
  constexpr int b_bytes = RW ? 0 : PT ? (BMN ? (BN / 64) * KC * 128 : BN * 128) : BMN ? (BN / 64) * 3 * KC * 128 : 3 * BN * 128;
  constexpr int w_bytes = RW ? 9 * BN * 128 : 0;  // resident weights [kw][kh][BN][64]
  const int stage_bytes = a_stride + b_bytes;
  constexpr int kSub = EPI == 0 ? BN / 64 : 0;  // 64-channel sub-tiles of the output staging
  uint8_t* wres = smem + (size_t)p.stages * stage_bytes;
  uint8_t* stg = wres + w_bytes;
  uint8_t* ybuf = stg + kSub * 16384;  // stats 2: the y2 tile of the tile in the epilogue (kSub sub-tiles)
  uint64_t* bars = reinterpret_cast<uint64_t*>(stg + (p.stats == 2 ? 2 : 1) * kSub * 16384);
  uint64_t* full = bars;
  uint64_t* empty = bars + kMaxStages;
  uint64_t* tfull = bars + 2 * kMaxStages;
  uint64_t* tempty = tfull + 2;
  uint64_t* wfull = tempty + 2;
  uint64_t* yfull = wfull + 1;
  uint64_t* yempty = yfull + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(yempty + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* epi_go = reinterpret_cast<volatile int*>(tmem_slot + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ksteps = (PT ? 9 : 3) * p.kchunks;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&tfull[a], 1);
      ptx::mbar_init(&tempty[a], 128);
    }
    ptx::mbar_init(wfull, 1);
    ptx::mbar_init(yfull, 1);
    ptx::mbar_init(yempty, 128);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tm_x);
    ptx::prefetch_tmap(&tm_w);
    ptx::prefetch_tmap(&tm_y);
  }
  constexpr uint32_t kTmemCols = 2 * BN < 32 ? 32 : 2 * BN;
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- producer: one TMA box of activations + three weight tiles per k-step
    uint32_t it = 0;
    bool ok = true;
    if constexpr (RW) {
      if (lane == 0 && blockIdx.x < p.total_tiles) {
        ptx::mbar_expect_tx(wfull, (uint32_t)w_bytes);
#pragma unroll
        for (int kw = 0; kw < 3; ++kw) ptx::tma_load_4d(wres + kw * 3 * BN * 128, &tm_w, wfull, 0, (blockIdx.x % p.n_tiles) * BN, kw, 0);
      }
      __syncwarp();
    }
    uint32_t ptl = 0;
    for (int t = blockIdx.x; ok && t < p.total_tiles; t += gridDim.x, ++ptl) {
      const int nt = t % p.n_tiles, m = t / p.n_tiles;
      const int w0 = (m % p.tiles_w) * p.BW, h0 = ((m / p.tiles_w) % p.tiles_h) * p.BH, n = (m / (p.tiles_w * p.tiles_h)) * p.BI;
      for (int ks = 0; ks < ksteps; ++ks, ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(&empty[s], ph ^ 1, abort_flag))) { ok = false; break; }
        if (lane == 0) {
          uint8_t* a_s = smem + (size_t)s * stage_bytes;
          ptx::mbar_expect_tx(&full[s], (uint32_t)(a_bytes + b_bytes));
          if constexpr (PT) {
            const int tap = ks % 9, ck = ks / 9, kh = tap / 3, kw = tap % 3;
            ptx::tma_load_4d(a_s, &tm_x, &full[s], ck * KC, p.stride * w0 + kw - 1, p.stride * h0 + kh - 1, n);
            if constexpr (BMN) {
#pragma unroll
              for (int hf = 0; hf < BN / 64; ++hf)  // [half][KC rows of f][64 channels], both taps mirrored
                ptx::tma_load_4d(a_s + a_stride + hf * KC * 128, &tm_w, &full[s], nt * BN + hf * 64, 0, 2 - kw, 2 - kh);
            } else {
              ptx::tma_load_4d(a_s + a_stride, &tm_w, &full[s], ck * 64, nt * BN, kw, kh);
            }
          } else {
            const int kw = ks % 3, ck = ks / 3;
            ptx::tma_load_4d(a_s, &tm_x, &full[s], ck * KC, w0 + kw - 1, h0 - 1, n);
            if constexpr (BMN) {
#pragma unroll
              for (int hf = 0; hf < BN / 64; ++hf)  // [half][kh][KC rows of f][64 channels], mirrored column tap
                ptx::tma_load_4d(a_s + a_stride + hf * 3 * KC * 128, &tm_w, &full[s], nt * BN + hf * 64, 0, 2 - kw, 0);
            } else if constexpr (!RW) {
              ptx::tma_load_4d(a_s + a_stride, &tm_w, &full[s], ck * 64, nt * BN, kw, 0);
            }
          }
        }
        __syncwarp();
      }
      if constexpr (EPI == 0) {
        // the y2 tile of this output tile goes out after its operand loads: the single buffer is free once the epilogue
        // has finished the statistics of the previous tile, which it does while this tile is being multiplied
        if (ok && p.stats == 2) {
          if (!__all_sync(0xffffffffu, ptx::mbar_wait(yempty, (ptl & 1) ^ 1, abort_flag))) break;
          if (lane == 0) {
            ptx::mbar_expect_tx(yfull, (uint32_t)(kSub * 16384));
#pragma unroll
            for (int sb = 0; sb < kSub; ++sb) ptx::tma_load_4d(ybuf + sb * 16384, &p.tm_y2, yfull, nt * BN + sb * 64, w0, h0, n);
          }
          __syncwarp();
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    constexpr uint32_t idesc = ptx::idesc_bf16(128, BN, 0, BMN);
    uint32_t it = 0, tl = 0;
    bool ok = true;
    // descriptors differ only in their 14-bit address field: constant upper parts, address added per use
    const uint64_t a_hi = ptx::sdesc(0, 16, 8 * kARow, kALayout);
    const uint64_t b_hi = BMN ? ptx::sdesc(0, (PT ? 1 : 3) * KC * 128, 1024, 2) : ptx::sdesc(0, 16, 1024, 2);
    const uint32_t a_row16 = (uint32_t)(p.BW * kARow) >> 4;  // one image row of the box, in 16-byte units
    if constexpr (RW) {
      if (blockIdx.x < p.total_tiles) ok = __all_sync(0xffffffffu, ptx::mbar_wait(wfull, 0, abort_flag));
    }
    for (int t = blockIdx.x; ok && t < p.total_tiles; t += gridDim.x, ++tl) {
      const uint32_t acc = tl & 1, aph = (tl >> 1) & 1;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&tempty[acc], aph ^ 1, abort_flag))) break;
      ptx::tc_fence_after();
      const uint32_t d = tmem_base + acc * BN;
      for (int ks = 0; ks < ksteps; ++ks, ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(&full[s], ph, abort_flag))) { ok = false; break; }
        ptx::tc_fence_after();
        if (lane == 0) {
          const uint32_t a_base = ptx::smem_u32(smem + (size_t)s * stage_bytes);
          const uint32_t a16 = a_base >> 4;
          const uint32_t b16 = RW ? (ptx::smem_u32(wres) + (ks % 3) * 3 * BN * 128) >> 4 : (a_base + a_stride) >> 4;
#pragma unroll
          for (int kh = 0; kh < (PT ? 1 : 3); ++kh)
#pragma unroll
            for (int k = 0; k < KC / 16; ++k) {
              const uint64_t ad = a_hi | (uint64_t)(a16 + kh * a_row16 + k * 2);
              const uint64_t bd = b_hi | (uint64_t)(BMN ? b16 + (((PT ? 0 : (2 - kh) * KC * 128) + k * 16 * 128) >> 4)
                                                        : b16 + ((kh * BN * 128 + k * 32) >> 4));
              ptx::mma_f16(d, ad, bd, idesc, (ks | kh | k) != 0);
            }
          ptx::mma_commit(&empty[s]);
        }
        __syncwarp();
      }
      if (ok && lane == 0) ptx::mma_commit(&tfull[acc]);
      __syncwarp();
    }
  } else {
    // ---------------- epilogue: 128 threads, thread <-> output pixel (TMEM lane)
    if constexpr (EPI == 0) {
    const int et = threadIdx.x - 64;
    const int lg = warp & 3;          // TMEM lane group this warp may read
    const int r = lg * 32 + lane;     // row of the tile = pixel (r % BW, r / BW)
    constexpr int kRowsPer = BN >= 128 ? 128 : 64;  // rows each thread sums for its channel
    const int sc = et % BN, shalf = et / BN;        // stats: channel and row half of this thread
    float ssum = 0.f, ssq = 0.f;
    float ssum2 = 0.f, ssq2 = 0.f;                  // BN = 256: the thread's second channel, sc + 128
    uint32_t tl = 0;
    int my_nt = blockIdx.x % p.n_tiles;
    float bsc = 0.f, bsh = 0.f, bsc2 = 0.f, bsh2 = 0.f;  // stats 2: BatchNorm scale / shift of the thread's channel(s)
    if (p.stats == 2) {
      const int ch = my_nt * BN + sc;
      bsc = p.bn_scale[ch];
      bsh = p.bn_shift[ch];
      if constexpr (BN == 256) {
        bsc2 = p.bn_scale[ch + 128];
        bsh2 = p.bn_shift[ch + 128];
      }
    }
    for (int t = blockIdx.x; t < p.total_tiles; t += gridDim.x, ++tl) {
      const int nt = t % p.n_tiles, m = t / p.n_tiles;
      const int w0 = (m % p.tiles_w) * p.BW, h0 = ((m / p.tiles_w) % p.tiles_h) * p.BH, n = (m / (p.tiles_w * p.tiles_h)) * p.BI;
      const uint32_t acc = tl & 1, aph = (tl >> 1) & 1;
      ptx::mbar_wait(&tfull[acc], aph, abort_flag);  // sets the abort flag itself when it gives up
      ptx::tc_fence_after();
      if (et == 0) {
        ptx::tma_store_wait_read();  // the previous tile's store has finished reading the staging tile
        *epi_go = *abort_flag ? 0 : 1;  // one thread decides for all 128, so nobody is left alone at a barrier
      }
      ptx::named_barrier(1, 128);
      if (!*epi_go) break;
#pragma unroll
      for (int j = 0; j < BN / 32; ++j) {
        uint32_t v[32];
        ptx::tmem_ld32(tmem_base + ((uint32_t)(lg * 32) << 16) + acc * BN + j * 32, v);
        ptx::tmem_ld_wait();
        uint8_t* sub = stg + ((j * 32) / 64) * 16384 + r * 128;
        const int u0 = ((j * 32) % 64) / 8;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float o0 = __uint_as_float(v[q * 8 + 2 * e]), o1 = __uint_as_float(v[q * 8 + 2 * e + 1]);
            if (p.bias) {  // wide aux forward: bias and ReLU before the value is rounded for storage
              const float* bch = p.bias + nt * BN + j * 32 + q * 8 + 2 * e;
              o0 = fmaxf(o0 + __ldg(bch), 0.f);
              o1 = fmaxf(o1 + __ldg(bch + 1), 0.f);
            }
            const __nv_bfloat162 b2 = __floats2bfloat162_rn(o0, o1);
            w[e] = *reinterpret_cast<const uint32_t*>(&b2);
          }
          *reinterpret_cast<uint4*>(sub + (((u0 + q) ^ (r & 7)) * 16)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&tempty[acc]);
      ptx::fence_async_smem();
      ptx::named_barrier(1, 128);
      if (et == 0) {
#pragma unroll
        for (int sb = 0; sb < kSub; ++sb) ptx::tma_store_4d(&tm_y, stg + sb * 16384, nt * BN + sb * 64, w0, h0, n);
        ptx::tma_store_commit();
      }
      if (p.stats == 2) {
        // sums of dz and dz*y2 (the last step turns them into sum dz*xhat = invstd * (sum dz*y2 - mu * sum dz))
        ptx::mbar_wait(yfull, tl & 1, abort_flag);
        const int coff = (sc / 64) * 16384 + (sc % 8) * 2;
        const int u = (sc % 64) / 8;
        const int rb = shalf * kRowsPer;
#pragma unroll 8
        for (int rr = 0; rr < kRowsPer; ++rr) {
          const int row = rb + rr;
          const int off = coff + row * 128 + ((u ^ (row & 7)) * 16);
          const float d = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(stg + off));
          const float yv = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(ybuf + off));
          const float dz = fmaf(yv, bsc, bsh) > 0.f ? d : 0.f;
          ssum += dz;
          ssq = fmaf(dz, yv, ssq);
          if constexpr (BN == 256) {
            const float d2 = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(stg + 2 * 16384 + off));
            const float y2 = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(ybuf + 2 * 16384 + off));
            const float dz2 = fmaf(y2, bsc2, bsh2) > 0.f ? d2 : 0.f;
            ssum2 += dz2;
            ssq2 = fmaf(dz2, y2, ssq2);
          }
        }
        ptx::mbar_arrive(yempty);
      } else if (p.stats) {
        const uint8_t* col = stg + (sc / 64) * 16384 + (sc % 8) * 2;
        const int u = (sc % 64) / 8;
        const int rb = shalf * kRowsPer;
#pragma unroll 8
        for (int rr = 0; rr < kRowsPer; ++rr) {
          const int row = rb + rr;
          const float v = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(col + row * 128 + ((u ^ (row & 7)) * 16)));
          ssum += v;
          ssq = fmaf(v, v, ssq);
          if constexpr (BN == 256) {
            const float v2 = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(col + 2 * 16384 + row * 128 + ((u ^ (row & 7)) * 16)));
            ssum2 += v2;
            ssq2 = fmaf(v2, v2, ssq2);
          }
        }
      }
    }
    if (et == 0) ptx::tma_store_wait_all();
    if (p.stats) {
      constexpr int parts = 128 / BN > 0 ? 128 / BN : 1;
      const size_t b = (size_t)blockIdx.x * parts + shalf;
      if (p.stats == 2) {
        const int ch = my_nt * BN + sc;
        ssq = (float)((double)p.bn_invstd[ch] * ((double)ssq - (double)p.bn_mu[ch] * (double)ssum));
        if constexpr (BN == 256) ssq2 = (float)((double)p.bn_invstd[ch + 128] * ((double)ssq2 - (double)p.bn_mu[ch + 128] * (double)ssum2));
      }
      p.red[(b * 2 + 0) * p.Cout + my_nt * BN + sc] = ssum;
      p.red[(b * 2 + 1) * p.Cout + my_nt * BN + sc] = ssq;
      if constexpr (BN == 256) {
        p.red[(b * 2 + 0) * p.Cout + my_nt * BN + 128 + sc] = ssum2;
        p.red[(b * 2 + 1) * p.Cout + my_nt * BN + 128 + sc] = ssq2;
      }
    }
    } else {
      const int et = threadIdx.x - 64;
      const int lg = warp & 3;
      const int r = lg * 32 + lane;
      uint32_t tl = 0;
      for (int t = blockIdx.x; t < p.total_tiles; t += gridDim.x, ++tl) {
        const int m = t / p.n_tiles;
        const int w0 = (m % p.tiles_w) * p.BW, h0 = ((m / p.tiles_w) % p.tiles_h) * p.BH, n = (m / (p.tiles_w * p.tiles_h)) * p.BI;
        const uint32_t acc = tl & 1, aph = (tl >> 1) & 1;
        ptx::mbar_wait(&tfull[acc], aph, abort_flag);
        ptx::tc_fence_after();
        if (et == 0) *epi_go = *abort_flag ? 0 : 1;
        ptx::named_barrier(1, 128);
        if (!*epi_go) break;
        const int img = r / (p.BW * p.BH);  // image of this pixel inside a multi-image tile
        const bool img_ok = n + img < p.N;
        bf16* dst = p.out + (((size_t)(n + img) * p.H + h0 + (r / p.BW) % p.BH) * p.W + w0 + r % p.BW) * p.Cout;
#pragma unroll
        for (int j = 0; j < BN / 16; ++j) {
          uint32_t v[16];
          ptx::tmem_ld16(tmem_base + ((uint32_t)(lg * 32) << 16) + acc * BN + j * 16, v);
          ptx::tmem_ld_wait();
          if (j * 16 < p.Cout && img_ok) {
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int c = j * 16 + 2 * e;
              const float a0 = c < p.Cout ? fmaxf(__uint_as_float(v[2 * e]) + p.bias[c], 0.f) : 0.f;
              const float a1 = c + 1 < p.Cout ? fmaxf(__uint_as_float(v[2 * e + 1]) + p.bias[c + 1], 0.f) : 0.f;
              const __nv_bfloat162 b2 = __floats2bfloat162_rn(a0, a1);
              w[e] = *reinterpret_cast<const uint32_t*>(&b2);
            }
            const int c0 = j * 16;
            if ((p.Cout & 7) == 0) {
              *reinterpret_cast<uint4*>(dst + c0) = make_uint4(w[0], w[1], w[2], w[3]);
              if (c0 + 8 < p.Cout) *reinterpret_cast<uint4*>(dst + c0 + 8) = make_uint4(w[4], w[5], w[6], w[7]);
            } else if ((p.Cout & 3) == 0) {
#pragma unroll
              for (int g4 = 0; g4 < 4; ++g4)
                if (c0 + 4 * g4 < p.Cout) *reinterpret_cast<uint2*>(dst + c0 + 4 * g4) = make_uint2(w[2 * g4], w[2 * g4 + 1]);
            } else {
              for (int e = 0; e < 16 && c0 + e < p.Cout; ++e)
                dst[c0 + e] = __ushort_as_bfloat16((unsigned short)((w[e >> 1] >> ((e & 1) * 16)) & 0xffffu));
            }
          }
        }
        ptx::tc_fence_before();
        ptx::mbar_arrive(&tempty[acc]);
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, NF_ETIMEOUT);
    // give copies still in flight time to land before the shared memory is released
    const unsigned long long t0 = ptx::globaltimer();
    while (ptx::globaltimer() - t0 < 2000000ull) __nanosleep(1000);
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 2 * BN);
  }
}


// ---------------------------------------------------------------- forward, 64 -> 64 channels, column taps folded into N
// With a 64-wide N tile an MMA is bound by the bytes of its operands, not by its arithmetic.  This
// variant widens N to 192: D'[pixel, (kw, co)] = sum_{kh, ci} X[pixel shifted by kh rows, ci] * W[kh][kw][co][ci],
// i.e. the three column taps become three 64-column groups of one accumulator and only the three row
// taps remain in the K loop (12 instructions of N = 192 per tile instead of 36 of N = 64, one
// activation box per tile instead of three).  The output is the shift-add
//   y[h, w, co] = D'[(h, w-1), kw=0, co] + D'[(h, w), kw=1, co] + D'[(h, w+1), kw=2, co],
// done in the epilogue with warp shuffles: a tile is 16 columns x 8 rows of pixels of which the outer
// two columns are halo, so the left/right neighbours of every output pixel are adjacent TMEM lanes of the
// same warp.  14 x 8 output pixels per tile; needs W % 14 == 0 and H % 8 == 0.
// Per-channel partial sums of one epilogue group (128 threads = 4 warps; a thread holds 8 channels, lane & 7 selects which):
// shuffles add the lanes of a warp, the warps are added through `scratch` (2 KB of shared memory the group owns) in warp order,
// and lanes 0..7 of the group's first warp write the 64 channel totals: red[0][c0 + ..] the first sums, red[1][..] the second
// (bn_second: turned into sum(dz * xhat) = invstd * (sum(dz * y) - mu * sum(dz)) in fp64).
__device__ __forceinline__ void fold_group_partial(float (&s1)[8], float (&s2)[8], float* scratch, int grp, int lg, int lane,
                                                   bool bn_second, const float* mu, const float* invstd, int c0, float* red, int C) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    s1[i] += __shfl_xor_sync(0xffffffffu, s1[i], 8);
    s2[i] += __shfl_xor_sync(0xffffffffu, s2[i], 8);
    s1[i] += __shfl_xor_sync(0xffffffffu, s1[i], 16);
    s2[i] += __shfl_xor_sync(0xffffffffu, s2[i], 16);
  }
  ptx::named_barrier(1 + grp, 128);  // the group's last TMA store has read the staging tile (its issuer waited before this)
  if (lane < 8) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      scratch[(lg * 2 + 0) * 64 + lane * 8 + i] = s1[i];
      scratch[(lg * 2 + 1) * 64 + lane * 8 + i] = s2[i];
    }
  }
  ptx::named_barrier(1 + grp, 128);
  if (lg == 0 && lane < 8) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int c = lane * 8 + i;
      const float a = ((scratch[0 * 64 + c] + scratch[2 * 64 + c]) + scratch[4 * 64 + c]) + scratch[6 * 64 + c];
      float b = ((scratch[1 * 64 + c] + scratch[3 * 64 + c]) + scratch[5 * 64 + c]) + scratch[7 * 64 + c];
      if (bn_second) b = (float)((double)invstd[c0 + c] * ((double)b - (double)mu[c0 + c] * (double)a));
      red[c0 + c] = a;
      red[C + c0 + c] = b;
    }
  }
}

struct FoldParams {
  int N, H, W, Cout, kchunks, n_tiles, tiles_w, tiles_h, total_tiles, stages, stats;
  float* red;         // EPI 0, stats != 0: [grid / n_tiles * 8][2][Cout]
  int32_t* status;
  const float *bn_scale, *bn_shift, *bn_mu, *bn_invstd;  // stats >= 2
  const float *bn_sdz, *bn_sdzx;                         // stats == 4: the reduced sums of the whole batch
  float inv_m;                                           // stats == 4: 1 / (elements per channel)
  const float* bias;  // EPI 1
  bf16* out;          // EPI 1: [N][H][W][Cout]
  // XF: the input map is the conv output y; a = ReLU(y*scale + shift) is formed in shared memory and written to xf_a
  const float *xf_scale, *xf_shift;
  bf16* xf_a;         // [N][H][W][64 * kchunks]
  // EPI 1 with pool_part != nullptr: h itself is not written.  What the rest of the step needs of it leaves the epilogue
  // directly: per tile and epilogue warp the per-channel sums of h over the warp's pixels (the average pool to 2 x 2 adds
  // them up; a tile never straddles a quadrant: H/2 % 8 == 0, W/2 % 14 == 0), and one bit per element, h > 0.
  float* pool_part;   // [total_tiles][4][Cout]
  uint8_t* mask;      // [N][H][W][Cout / 8], bit f % 8 of byte f / 8
};

// G   : width of one column-tap group of the accumulator (N = 3*G): 64 for the main conv, 16/32/64 for the
//       aux conv with F <= G filters (weight rows beyond F are zero-filled by TMA).
// EPI : 0 = y in bf16 through a TMA store + BatchNorm partial sums (G = 64, Cout = 64);
//       1 = bias + ReLU, F channels written straight from registers (aux conv forward).
// Cin = 64 * kchunks; all 9 * kchunks weight tiles stay resident in shared memory.
// stats (EPI 0): 1 = per-channel sums of (y, y^2) of the stored values (BatchNorm forward statistics);
//       2 = the output is the gradient da at a BatchNorm+ReLU output of the same shape: per-channel sums of
//       (dz, dz * xhat) with dz = da * 1[y2*scale+shift > 0], xhat = (y2 - mu) * invstd, where the tile of the
//       pre-normalisation values y2 is fetched through tm_y2 (BatchNorm backward reduction fused into the producer of da);
//       3 = the same sums, but da is not written at all; 4 = the second pass of that pair: da is formed again, turned
//       into dy = scale * (dz - sum(dz)/M - xhat * sum(dz*xhat)/M) in the staging tile with the sums of pass 3, and dy is
//       what the TMA store writes.  Passes 3 + 4 replace "write da; read y and da; write dy" by one more read of the
//       narrow dh tensor: da never reaches memory.
// KC / MIR: KC = channels of the activation box (64; 16 or 32 for the aux input gradient whose input dh has F
// channels), MIR = 1 reads the weights [tap][f][c] MN-major with both taps mirrored (input-gradient convolution;
// the CTA's 64-channel output tile is blockIdx.x % n_tiles).
// UF = 1 (input gradient with KC <= 32 only): the column taps are NOT folded.  With so few input channels a tile needs
// only nine instructions (one per tap, N = 64) even unfolded, and the epilogue is what bounds the kernel: three
// column-shifted activation boxes per stage replace the shift-add, the accumulator is 64 columns wide and all 16 x 8
// pixels of a tile are outputs (W % 16 == 0).
// XF = 1 (aux forward only): BatchNorm + ReLU of the layer are applied on the way in.  The boxes are loaded from the
// conv output y; four more warps turn each box into a = ReLU(y*scale + shift) in place (zero outside the image, as the
// padding of a must be), write the tile's own 14 x 8 pixels of a to global memory (the layer's output activation) and
// only then hand the stage to the issuer.  The separate normalisation pass (read y, write a) and this kernel's read of
// a disappear; the halo pixels are normalised by both neighbours.
template <int G, int EPI, int KC = 64, int MIR = 0, int UF = 0, int XF = 0>
__global__ void __launch_bounds__(kFoldThreads + kXfThreads * XF, 1)
conv_fwd_fold_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                     const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_y2, const FoldParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int kARow = KC * 2;               // bytes of one pixel of the activation box
  constexpr uint32_t kALayout = KC == 64 ? 2 : KC == 32 ? 4 : 6;
  static_assert(!UF || (MIR && EPI == 0 && G == 64 && KC <= 32), "unfolded form: input gradient with few input channels");
  static_assert(!XF || (EPI == 1 && KC == 64 && !MIR && !UF), "fused normalisation: aux forward only");
  // UF = 2: tiles of 8 columns x 16 rows fed by ONE box of 10 x 18 pixels.  An image row of the tile is then exactly one
  // 8-row group of the operand, so the nine taps are nine start addresses (kh * 10 + kw pixels into the box) with a constant
  // pitch of 10 pixels between groups: a third of the TMA rows of the three-box form, whose narrow 32-byte rows made the
  // producer the slowest role of the kernel.  The shared-memory swizzle is a function of the address, so TMA and the tensor
  // core agree wherever a tap starts.
  constexpr int kBox = UF == 2 ? 18 * 10 * kARow : 10 * 16 * kARow;  // (8+2) rows x 16 pixels x KC channels
  constexpr int kABytes = UF == 2 ? (kBox + 1023) / 1024 * 1024 : (UF ? 3 : 1) * kBox;  // UF 1: one box per column tap
  constexpr int kTW = UF == 2 ? 8 : UF ? 16 : 14;  // output columns of a tile
  constexpr int kTH = UF == 2 ? 16 : 8;            // output rows of a tile
  constexpr int kStatIters = UF ? 8 : 7;           // 16-row slices of the staged tile (128 or 112 pixels)
  constexpr int kWTile = MIR ? 3 * KC * 128 : 3 * G * 128;  // one kernel row: [kw*G + co][64 ci], or mirrored [kw][f][64 c]
  const int w_bytes = 3 * p.kchunks * kWTile; // [chunk][kh][kw*G + co][64 ci]
  uint8_t* wres = smem + (size_t)p.stages * kABytes;
  uint8_t* stg = wres + w_bytes;              // EPI 0: 112 (UF: 128) output pixels x 128 bytes
  uint8_t* ybuf = stg + 2 * 16384;            // EPI 0, stats >= 2: kYSlots tiles of y2, taken in turn by the CTA's tiles
  constexpr int kAStg = 112 * 128;            // XF: one 14 x 8-pixel tile of a on its way to global memory (three in rotation per group)
  // one staging tile per epilogue group (EPI 0), or the three tiles of a (XF)
  uint64_t* bars = reinterpret_cast<uint64_t*>(stg + (EPI == 0 ? (p.stats >= 2 ? 2 + kYSlots : 2) * 16384 : XF ? 3 * kXfGroups * kAStg : 0));
  uint64_t* full = bars;
  uint64_t* empty = bars + kMaxStages;
  uint64_t* tfull = bars + 2 * kMaxStages;
  uint64_t* tempty = tfull + 4;
  uint64_t* wfull = tempty + 4;
  uint64_t* yfull = wfull + 1;
  uint64_t* yempty = yfull + kYSlots;
  uint64_t* xfull = yempty + kYSlots;  // XF: stage normalised, ready for the issuer
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(xfull + kMaxStages);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* epi_go = reinterpret_cast<volatile int*>(tmem_slot + 2);  // [2], one per epilogue group
  volatile int* xf_go = reinterpret_cast<volatile int*>(tmem_slot + 4);   // [2 per group], alternating between a group's iterations
  // Accumulators in tensor memory.  The unfolded form needs 64 columns each and keeps four, so that the issuer can run two
  // tiles ahead of each epilogue group (group g takes the tiles tl = g, g + 2, ... and so alternates between two of them);
  // the folded forms need up to 192 columns each and keep two, one per group.
  constexpr uint32_t kAccs = UF ? 4 : 2;
  constexpr uint32_t kAccStride = UF ? 128 : G == 64 ? 256 : 128;  // columns between two accumulators
  constexpr uint32_t kTmemCols = kAccs * kAccStride;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
      ptx::mbar_init(&xfull[s], 128);
    }
    for (int a = 0; a < (int)kAccs; ++a) {
      ptx::mbar_init(&tfull[a], 1);
      ptx::mbar_init(&tempty[a], 128);
    }
    for (int a = 0; a < kYSlots; ++a) {
      ptx::mbar_init(&yfull[a], 1);
      ptx::mbar_init(&yempty[a], 128);
    }
    ptx::mbar_init(wfull, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tm_x);
    ptx::prefetch_tmap(&tm_w);
    ptx::prefetch_tmap(&tm_y);
    ptx::prefetch_tmap(&tm_y2);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0 && blockIdx.x < p.total_tiles) {
      ptx::mbar_expect_tx(wfull, (uint32_t)w_bytes);
      for (int ck = 0; ck < p.kchunks; ++ck)
#pragma unroll
        for (int kh = 0; kh < 3; ++kh)
          ptx::tma_load_4d(wres + (ck * 3 + kh) * kWTile, &tm_w, wfull, MIR ? (int)(blockIdx.x % p.n_tiles) * 64 : ck * 64, 0, 0, kh);
    }
    __syncwarp();
    uint32_t it = 0, tl = 0;
    bool ok = true;
    for (int t = blockIdx.x; ok && t < p.total_tiles; t += gridDim.x, ++tl) {
      const int m = t / p.n_tiles;
      const int w0 = (m % p.tiles_w) * kTW, h0 = ((m / p.tiles_w) % p.tiles_h) * kTH, n = m / (p.tiles_w * p.tiles_h);
      for (int ck = 0; ck < p.kchunks; ++ck, ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(&empty[s], ph ^ 1, abort_flag))) { ok = false; break; }
        if (lane == 0) {
          ptx::mbar_expect_tx(&full[s], (uint32_t)(UF == 2 ? kBox : kABytes));
          if constexpr (UF == 2) {
            ptx::tma_load_4d(smem + (size_t)s * kABytes, &tm_x, &full[s], ck * KC, w0 - 1, h0 - 1, n);
          } else if constexpr (UF) {
#pragma unroll
            for (int kw = 0; kw < 3; ++kw)
              ptx::tma_load_4d(smem + (size_t)s * kABytes + kw * kBox, &tm_x, &full[s], ck * KC, w0 - 1 + kw, h0 - 1, n);
          } else {
            ptx::tma_load_4d(smem + (size_t)s * kABytes, &tm_x, &full[s], ck * KC, w0 - 1, h0 - 1, n);
          }
        }
        __syncwarp();
      }
      if constexpr (EPI == 0) {
        if (ok && p.stats >= 2) {  // the y2 tile of this output tile, for the epilogue group that owns it
          const uint32_t slot = tl % kYSlots;
          if (!__all_sync(0xffffffffu, ptx::mbar_wait(&yempty[slot], ((tl / kYSlots) & 1) ^ 1, abort_flag))) break;
          if (lane == 0) {
            ptx::mbar_expect_tx(&yfull[slot], kTW * kTH * 128);
            ptx::tma_load_4d(ybuf + slot * 16384, &tm_y2, &yfull[slot], (t % p.n_tiles) * 64, w0, h0, n);
          }
          __syncwarp();
        }
      }
    }
  } else if (warp == 1) {
    constexpr uint32_t idesc = ptx::idesc_bf16(128, UF ? G : 3 * G, 0, MIR);
    const uint64_t a_hi = ptx::sdesc(0, 16, (UF == 2 ? 10 : 8) * kARow, kALayout);  // UF 2: next 8-pixel group = next box row
    const uint64_t b_hi = MIR ? ptx::sdesc(0, KC * 128, 1024, 2) : ptx::sdesc(0, 16, 1024, 2);
    const uint32_t w16 = ptx::smem_u32(wres) >> 4;
    uint32_t it = 0, tl = 0;
    bool ok = blockIdx.x >= p.total_tiles || __all_sync(0xffffffffu, ptx::mbar_wait(wfull, 0, abort_flag));
    for (int t = blockIdx.x; ok && t < p.total_tiles; t += gridDim.x, ++tl) {
      const uint32_t acc = tl % kAccs, aph = (tl / kAccs) & 1;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&tempty[acc], aph ^ 1, abort_flag))) break;
      ptx::tc_fence_after();
      const uint32_t d = tmem_base + acc * kAccStride;
      for (int ck = 0; ck < p.kchunks; ++ck, ++it) {
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(XF ? &xfull[s] : &full[s], ph, abort_flag))) { ok = false; break; }
        ptx::tc_fence_after();
        if (lane == 0) {
          const uint32_t a16 = ptx::smem_u32(smem + (size_t)s * kABytes) >> 4;
          if constexpr (UF) {  // one instruction per tap and 16 input channels; tap (kh, kw) reads the mirrored weight tile
#pragma unroll
            for (int kh = 0; kh < 3; ++kh)
#pragma unroll
              for (int kw = 0; kw < 3; ++kw)
#pragma unroll
                for (int k = 0; k < KC / 16; ++k) {
                  const uint64_t ad = UF == 2 ? a_hi | (uint64_t)(a16 + ((kh * 10 + kw) * kARow >> 4) + k * 2)
                                              : a_hi | (uint64_t)(a16 + kw * (kBox >> 4) + kh * (16 * kARow >> 4) + k * 2);
                  const uint64_t bd = b_hi | (uint64_t)(w16 + (2 - kh) * (kWTile >> 4) + (2 - kw) * (KC * 128 >> 4) + k * 128);
                  ptx::mma_f16(d, ad, bd, idesc, (kh | kw | k) != 0);
                }
          } else
#pragma unroll
          for (int kh = 0; kh < 3; ++kh)
#pragma unroll
            for (int k = 0; k < KC / 16; ++k) {
              const uint64_t ad = a_hi | (uint64_t)(a16 + kh * (16 * kARow >> 4) + k * 2);
              const uint64_t bd = MIR ? b_hi | (uint64_t)(w16 + (2 - kh) * (kWTile >> 4) + k * 128)   // mirrored row tap, 16 f rows on
                                      : b_hi | (uint64_t)(w16 + (ck * 3 + kh) * (kWTile >> 4) + k * 2);
              ptx::mma_f16(d, ad, bd, idesc, (ck | kh | k) != 0);
            }
          ptx::mma_commit(&empty[s]);
        }
        __syncwarp();
      }
      if (ok && lane == 0) ptx::mma_commit(&tfull[acc]);
      __syncwarp();
    }
  } else if (XF && warp >= kFoldThreads / 32) {
    // normalisation warps: a thread owns one 16-byte channel chunk (8 channels) of one box column and walks the 10 rows.
    // The tile's own 14 x 8 pixels of a leave through a TMA store: the threads copy them from registers into a dense staging
    // tile (three in rotation) and one thread issues the store, so no global store instruction runs in these warps.
    const int xt = (threadIdx.x - kFoldThreads) & 127, xgrp = (threadIdx.x - kFoldThreads) >> 7;  // group xgrp takes the stages it % kXfGroups == xgrp
    constexpr int kXg = 1, kRows = 10, xg = 0;
    uint8_t* const stg_x = stg + xgrp * 3 * kAStg;
    const int j = xt & 7, col = xt >> 3;                   // logical chunk, box column (0..15)
    const uint32_t off0 = (uint32_t)col * 128 + (uint32_t)((j ^ (col & 7)) * 16);  // 128-byte swizzle: the row's low bits are col's
    uint32_t it = 0;
    float sc[8], sh[8];
    int coef_ck = -1;  // channel chunk whose coefficients the registers hold
    bool go = true;
    for (int t = blockIdx.x; go && t < p.total_tiles; t += gridDim.x) {
      const int m = t / p.n_tiles;
      const int w0 = (m % p.tiles_w) * 14, h0 = ((m / p.tiles_w) % p.tiles_h) * 8, n = m / (p.tiles_w * p.tiles_h);
      const int w = w0 - 1 + col;
      const bool w_in = w >= 0 && w < p.W, w_own = col >= 1 && col <= 14;
      for (int ck = 0; ck < p.kchunks; ++ck, ++it) {
        if ((int)(it % kXfGroups) != xgrp) continue;
        const uint32_t jt = it / kXfGroups;  // this group's iteration count
        const int s = it % p.stages;
        const uint32_t ph = (it / p.stages) & 1;
        if (ck != coef_ck) {
          coef_ck = ck;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            sc[i] = __ldg(p.xf_scale + ck * 64 + j * 8 + i);
            sh[i] = __ldg(p.xf_shift + ck * 64 + j * 8 + i);
          }
        }
        const bool ok = ptx::mbar_wait(&full[s], ph, abort_flag);
        const uint32_t astg = ptx::smem_u32(stg_x) + (jt % 3) * kAStg;
        if (ok) {
          const uint32_t box = ptx::smem_u32(smem + (size_t)s * kABytes) + off0 + xg * 2048;
          // all rows are loaded first, then normalised, then stored: the loads overlap instead of queueing behind stores
          uint4 q[kRows];
#pragma unroll
          for (int i = 0; i < kRows; ++i) q[i] = ptx::lds128(box + i * kXg * 2048);
#pragma unroll
          for (int i = 0; i < kRows; ++i) {
            const int h = h0 - 1 + i * kXg + xg;
            const uint32_t qw[4] = {q[i].x, q[i].y, q[i].z, q[i].w};
            uint32_t ow[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float a0 = fmaxf(fmaf(__uint_as_float(qw[e] << 16), sc[2 * e], sh[2 * e]), 0.f);
              const float a1 = fmaxf(fmaf(__uint_as_float(qw[e] & 0xffff0000u), sc[2 * e + 1], sh[2 * e + 1]), 0.f);
              const __nv_bfloat162 b2 = __floats2bfloat162_rn(a0, a1);
              ow[e] = *reinterpret_cast<const uint32_t*>(&b2);
            }
            const bool in = w_in && h >= 0 && h < p.H;
            q[i] = in ? make_uint4(ow[0], ow[1], ow[2], ow[3]) : make_uint4(0u, 0u, 0u, 0u);
            ptx::sts128(box + i * kXg * 2048, q[i]);
          }
          if (w_own) {  // box rows 1..8 x columns 1..14 are the tile's own pixels: dense rows of the staging tile, same swizzle
#pragma unroll
            for (int i = 1; i <= 8; ++i) {
              const uint32_t orow = (uint32_t)((i - 1) * 14 + col - 1);
              ptx::sts128(astg + orow * 128 + ((j ^ (orow & 7)) * 16), q[i]);
            }
          }
          ptx::fence_async_smem();  // the tensor core and the TMA store read shared memory through the async proxy
          ptx::mbar_arrive(&xfull[s]);
        }
        // one thread decides for all 128 whether to go on, so nobody is left alone at the barrier
        if (xt == 0) xf_go[xgrp * 2 + (jt & 1)] = ok && !*abort_flag ? 1 : 0;
        ptx::named_barrier(3 + xgrp, 128);
        if (!xf_go[xgrp * 2 + (jt & 1)]) { go = false; break; }
        if (xt == 0) {
          ptx::tma_store_4d(&tm_y, reinterpret_cast<const void*>(stg_x + (jt % 3) * kAStg), ck * 64, w0, h0, n);
          ptx::tma_store_commit();
          ptx::tma_store_wait_read_but_one();  // the store before this one has read its tile: the tile after next may be written
        }
      }
    }
    if (xt == 0) ptx::tma_store_wait_all();
  } else {
    // two epilogue groups of 128 threads; group g owns accumulator g and takes every second tile of the CTA
    const int grp = (threadIdx.x - 64) >> 7;
    const int et = (threadIdx.x - 64) & 127;
    uint8_t* const stg_g = stg + grp * 16384;
    const int lg = warp & 3;
    const int r = lg * 32 + lane;            // TMEM lane = extended-tile pixel (we = r % 16, h = r / 16)
    const int we = r & 15, hh = r >> 4;
    const bool valid = UF || (we >= 1 && we <= 14);
    const int orow = UF ? r : (we - 1) + 14 * hh;  // row of the output staging tile
    // statistics: a thread owns 8 channels (one 16-byte chunk of a pixel row) and the 7 rows rg, rg+16, ...
    const int schunk = et & 7, srg = et >> 3;
    float s1[8], s2[8], bsc[8], bsh[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) s1[i] = s2[i] = bsc[i] = bsh[i] = 0.f;
    if constexpr (EPI == 0) {
      if (p.stats >= 2) {
        const int ch = (int)(blockIdx.x % p.n_tiles) * 64 + schunk * 8;
#pragma unroll
        for (int i = 0; i < 8; ++i) { bsc[i] = p.bn_scale[ch + i]; bsh[i] = p.bn_shift[ch + i]; }
        if (p.stats == 4) {  // s1, s2 hold the per-channel constants of dy = scale*dz + s1*y + s2 instead of running sums
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float sc = bsc[i], m1 = p.bn_sdz[ch + i] * p.inv_m, m2 = p.bn_sdzx[ch + i] * p.inv_m, is = p.bn_invstd[ch + i];
            s1[i] = -sc * m2 * is;
            s2[i] = sc * (m2 * is * p.bn_mu[ch + i] - m1);
          }
        }
      }
    }
    uint32_t tl = grp;
    // 32-bit tile arithmetic (the host keeps total_tiles below 2^30): 64-bit divisions here cost about a quarter of the tile time
    for (int t = blockIdx.x + grp * gridDim.x; t < p.total_tiles; t += 2 * gridDim.x, tl += 2) {
      const int nt = t % p.n_tiles;
      const int m = t / p.n_tiles;
      const int w0 = (m % p.tiles_w) * kTW, h0 = ((m / p.tiles_w) % p.tiles_h) * kTH, n = m / (p.tiles_w * p.tiles_h);
      const uint32_t acc = tl % kAccs, aph = (tl / kAccs) & 1;
      ptx::mbar_wait(&tfull[acc], aph, abort_flag);
      ptx::tc_fence_after();
      if (et == 0) {
        if constexpr (EPI == 0) ptx::tma_store_wait_read();
        epi_go[grp] = *abort_flag ? 0 : 1;
      }
      ptx::named_barrier(1 + grp, 128);
      if (!epi_go[grp]) break;
      // a last tile column may reach beyond the image (widths that are not multiples of 14): those pixels are stored as
      // zeros in the staging tile (they add nothing to the statistics; the TMA store clips them) and never written directly
      const bool vcol = valid && (UF || w0 + we - 1 < p.W);
      const uint32_t tbase = tmem_base + ((uint32_t)(lg * 32) << 16) + acc * kAccStride;
      bf16* gdst = EPI == 1 ? p.out + (((size_t)n * p.H + h0 + hh) * p.W + w0 + we - 1) * p.Cout : nullptr;
#pragma unroll
      for (int q = 0; q < G / 16; ++q) {     // 16 output channels at a time
        uint32_t v0[16], v1[16], v2[16];
        uint32_t w[8];
        if constexpr (UF) {
          ptx::tmem_ld16(tbase + q * 16, v1);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(v1[2 * e]), __uint_as_float(v1[2 * e + 1]));
            w[e] = *reinterpret_cast<const uint32_t*>(&b2);
          }
        } else {
        ptx::tmem_ld16(tbase + (MIR ? 2 * G : 0) + q * 16, v0);  // group feeding the pixel on the left
        ptx::tmem_ld16(tbase + G + q * 16, v1);
        ptx::tmem_ld16(tbase + (MIR ? 0 : 2 * G) + q * 16, v2);  // group feeding the pixel on the right
        ptx::tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          float o[2];
#pragma unroll
          for (int h2 = 0; h2 < 2; ++h2) {
            const int c = 2 * e + h2;
            const float left = __shfl_up_sync(0xffffffffu, __uint_as_float(v0[c]), 1);     // kw = 0 term of pixel w-1
            const float right = __shfl_down_sync(0xffffffffu, __uint_as_float(v2[c]), 1);  // kw = 2 term of pixel w+1
            o[h2] = left + __uint_as_float(v1[c]) + right;
            if constexpr (EPI == 1) {
              const int ch = q * 16 + c;
              o[h2] = ch < p.Cout ? fmaxf(o[h2] + p.bias[ch], 0.f) : 0.f;
            } else {
              if (p.bias) o[h2] = fmaxf(o[h2] + __ldg(p.bias + nt * 64 + q * 16 + c), 0.f);
            }
          }
          const __nv_bfloat162 b2 = __floats2bfloat162_rn(o[0], o[1]);
          w[e] = *reinterpret_cast<const uint32_t*>(&b2);
        }
        }
        if constexpr (EPI == 0) {
          if (valid) {
            uint8_t* dst = stg_g + orow * 128;
            *reinterpret_cast<uint4*>(dst + (((2 * q) ^ (orow & 7)) * 16)) = vcol ? make_uint4(w[0], w[1], w[2], w[3]) : make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(dst + (((2 * q + 1) ^ (orow & 7)) * 16)) = vcol ? make_uint4(w[4], w[5], w[6], w[7]) : make_uint4(0u, 0u, 0u, 0u);
          }
        } else if (p.pool_part) {
          // h stays in registers: its sign bits go to the mask, its sum over the warp's 32 pixels (halo pixels count as
          // zero) to the pooling partials.  The 16 channel sums are formed by a reduce-scatter over the lanes: each step
          // halves the channels a lane carries and doubles the pixels its sums cover (16 shuffles for 16 channels); the
          // lane pair (2j, 2j+1) ends with the sum of channel j's bit pattern below.
          const int c0 = q * 16;
          float ov[16];
          uint32_t bits = 0;
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float lo = __uint_as_float(w[e] << 16), hi = __uint_as_float(w[e] & 0xffff0000u);
            ov[2 * e] = vcol ? lo : 0.f;
            ov[2 * e + 1] = vcol ? hi : 0.f;
            bits |= (lo > 0.f ? 1u : 0u) << (2 * e);
            bits |= (hi > 0.f ? 1u : 0u) << (2 * e + 1);
          }
          if (vcol && c0 < p.Cout) {
            uint8_t* mdst = p.mask + ((((size_t)n * p.H + h0 + hh) * p.W + w0 + we - 1) * (size_t)(p.Cout >> 3)) + (c0 >> 3);
            mdst[0] = (uint8_t)(bits & 0xffu);
            if (c0 + 8 < p.Cout) mdst[1] = (uint8_t)(bits >> 8);
          }
          float r8[8], r4[4], r2[2];
          const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4, b1 = lane & 2;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float send = b4 ? ov[i] : ov[8 + i], keep = b4 ? ov[8 + i] : ov[i];
            r8[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float send = b3 ? r8[i] : r8[4 + i], keep = b3 ? r8[4 + i] : r8[i];
            r4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
          }
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const float send = b2 ? r4[i] : r4[2 + i], keep = b2 ? r4[2 + i] : r4[i];
            r2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
          }
          float r1 = (b1 ? r2[1] : r2[0]) + __shfl_xor_sync(0xffffffffu, b1 ? r2[0] : r2[1], 2);
          r1 += __shfl_xor_sync(0xffffffffu, r1, 1);
          const int ch = c0 + (b4 ? 8 : 0) + (b3 ? 4 : 0) + (b2 ? 2 : 0) + (b1 ? 1 : 0);
          if ((lane & 1) == 0 && ch < p.Cout) p.pool_part[((size_t)t * 4 + lg) * p.Cout + ch] = r1;
        } else {
          const int c0 = q * 16;             // Cout is a multiple of 8 here
          if (vcol && c0 < p.Cout) {
            *reinterpret_cast<uint4*>(gdst + c0) = make_uint4(w[0], w[1], w[2], w[3]);
            if (c0 + 8 < p.Cout) *reinterpret_cast<uint4*>(gdst + c0 + 8) = make_uint4(w[4], w[5], w[6], w[7]);
          }
        }
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&tempty[acc]);
      if constexpr (EPI == 0) {
        ptx::fence_async_smem();
        ptx::named_barrier(1 + grp, 128);
        if (p.stats == 4) {
          // second pass: the staged da tile becomes dy in place (thread <-> 8 channels x 7 or 8 rows, as for the sums)
          const uint32_t slot = tl % kYSlots;
          ptx::mbar_wait(&yfull[slot], (tl / kYSlots) & 1, abort_flag);
          const uint8_t* yb = ybuf + slot * 16384;
#pragma unroll
          for (int rr = 0; rr < kStatIters; ++rr) {
            const int row = srg + 16 * rr;
            const int off = row * 128 + ((schunk ^ (row & 7)) * 16);
            const uint4 dq = *reinterpret_cast<const uint4*>(stg_g + off);
            const uint4 yq = *reinterpret_cast<const uint4*>(yb + off);
            const uint32_t dw[4] = {dq.x, dq.y, dq.z, dq.w}, yw[4] = {yq.x, yq.y, yq.z, yq.w};
            uint32_t ow[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float d0 = __uint_as_float(dw[e] << 16), d1 = __uint_as_float(dw[e] & 0xffff0000u);
              const float y0 = __uint_as_float(yw[e] << 16), y1 = __uint_as_float(yw[e] & 0xffff0000u);
              const float z0 = fmaf(y0, bsc[2 * e], bsh[2 * e]) > 0.f ? d0 : 0.f;
              const float z1 = fmaf(y1, bsc[2 * e + 1], bsh[2 * e + 1]) > 0.f ? d1 : 0.f;
              const float o0 = fmaf(bsc[2 * e], z0, fmaf(s1[2 * e], y0, s2[2 * e]));
              const float o1 = fmaf(bsc[2 * e + 1], z1, fmaf(s1[2 * e + 1], y1, s2[2 * e + 1]));
              const __nv_bfloat162 b2 = __floats2bfloat162_rn(o0, o1);
              ow[e] = *reinterpret_cast<const uint32_t*>(&b2);
            }
            *reinterpret_cast<uint4*>(stg_g + off) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
          }
          ptx::mbar_arrive(&yempty[slot]);
          ptx::fence_async_smem();
          ptx::named_barrier(1 + grp, 128);
        }
        if (et == 0 && p.stats != 3) {
          ptx::tma_store_4d(&tm_y, stg_g, nt * 64, w0, h0, n);
          ptx::tma_store_commit();
        }
        if (p.stats == 2 || p.stats == 3) {
          // sums of dz and dz*y2 (the caller of the kernel gets sum dz*xhat = invstd * (sum dz*y2 - mu * sum dz))
          const uint32_t slot = tl % kYSlots;
          ptx::mbar_wait(&yfull[slot], (tl / kYSlots) & 1, abort_flag);
          const uint8_t* yb = ybuf + slot * 16384;
#pragma unroll
          for (int rr = 0; rr < kStatIters; ++rr) {
            const int row = srg + 16 * rr;
            const int off = row * 128 + ((schunk ^ (row & 7)) * 16);
            const uint4 dq = *reinterpret_cast<const uint4*>(stg_g + off);
            const uint4 yq = *reinterpret_cast<const uint4*>(yb + off);
            const uint32_t dw[4] = {dq.x, dq.y, dq.z, dq.w}, yw[4] = {yq.x, yq.y, yq.z, yq.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float d0 = __uint_as_float(dw[e] << 16), d1 = __uint_as_float(dw[e] & 0xffff0000u);
              const float y0 = __uint_as_float(yw[e] << 16), y1 = __uint_as_float(yw[e] & 0xffff0000u);
              const float z0 = fmaf(y0, bsc[2 * e], bsh[2 * e]) > 0.f ? d0 : 0.f;
              const float z1 = fmaf(y1, bsc[2 * e + 1], bsh[2 * e + 1]) > 0.f ? d1 : 0.f;
              s1[2 * e] += z0;
              s1[2 * e + 1] += z1;
              s2[2 * e] = fmaf(z0, y0, s2[2 * e]);
              s2[2 * e + 1] = fmaf(z1, y1, s2[2 * e + 1]);
            }
          }
          ptx::mbar_arrive(&yempty[slot]);
        } else if (p.stats == 1) {
#pragma unroll
          for (int rr = 0; rr < kStatIters; ++rr) {
            const int row = srg + 16 * rr;
            const uint4 vq = *reinterpret_cast<const uint4*>(stg_g + row * 128 + ((schunk ^ (row & 7)) * 16));
            const uint32_t vw[4] = {vq.x, vq.y, vq.z, vq.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float v0 = __uint_as_float(vw[e] << 16), v1 = __uint_as_float(vw[e] & 0xffff0000u);
              s1[2 * e] += v0;
              s1[2 * e + 1] += v1;
              s2[2 * e] = fmaf(v0, v0, s2[2 * e]);
              s2[2 * e + 1] = fmaf(v1, v1, s2[2 * e + 1]);
            }
          }
        }
      }
    }
    if constexpr (EPI == 0) {
      if (et == 0) ptx::tma_store_wait_all();
      if (p.stats && p.stats != 4) {
        // one partial per epilogue group: lanes with the same chunk (lane & 7) are added by shuffles, the group's four warps
        // through the (now idle) staging tile, all in a fixed order
        fold_group_partial(s1, s2, reinterpret_cast<float*>(stg_g), grp, lg, lane, p.stats >= 2, p.bn_mu, p.bn_invstd,
                           (int)(blockIdx.x % p.n_tiles) * 64, p.red + ((size_t)(blockIdx.x / p.n_tiles) * 2 + grp) * 2 * p.Cout, p.Cout);
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, NF_ETIMEOUT);
    const unsigned long long t0 = ptx::globaltimer();
    while (ptx::globaltimer() - t0 < 2000000ull) __nanosleep(1000);
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------- aux input gradient, 256 pixels per instruction
// The narrow input gradient da = dh (*) Wa^T (K = F <= 32 per tap) is bound by the NUMBER of its K = 16 instructions, each of
// which holds the tensor pipe for about the same time whatever its shape.  With the pixels on the M side an instruction covers
// 128 of them; here the operands are swapped: A = the mirrored weight tile of a tap, [64 output channels] x [16 f] (M = 64,
// MN-major as stored), B = 256 pixels x [16 f] of the dh box (N = 256, K-major), so the nine taps of a 256-pixel tile are nine
// instructions instead of eighteen.  A tile is 8 columns x 32 rows; ONE 10 x 34-pixel box feeds all taps (a tap is a start
// address kh * 10 + kw pixels into the box, an image row of the tile is one 8-row group, pitch 10 pixels: the swizzle is a
// function of the address).  The accumulator holds D[channel][pixel]: with M = 64, channel c sits in lane 32 * (c / 16) + c % 16,
// so warp q of an epilogue group reads channels 16q .. 16q+15 in lanes 0..15 of its quadrant as accumulator fragments and
// transposes them into the pixel-major staging tile with transposing matrix stores (16 bytes = 8 channels per pixel and store row).
// From there on everything is as in the folded kernel: BatchNorm-backward sums (stats 2, 3), the second pass that turns the
// tile into dy (stats 4), TMA store (not for stats 3).  Needs W % 8 == 0 and H % 16 == 0 (a last tile row of 16 image rows: the
// box rows below the image load as zeros, the store is clipped, the sums skip them); one 64-channel output tile per CTA.
constexpr int kWideThreads = 320;
constexpr int kWideYSlots = 3;

template <int KC>
__global__ void __launch_bounds__(kWideThreads, 1)
aux_dgrad_wide_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                      const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_y2, const FoldParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int kARow = KC * 2;                                    // bytes of one pixel of the dh box
  constexpr uint32_t kALayout = KC == 32 ? 4 : 6;
  constexpr int kBox = 34 * 10 * kARow;                            // (32+2) rows x (8+2) pixels
  constexpr int kStage = (kBox + 1023) / 1024 * 1024;
  constexpr int kWTile = 3 * KC * 128;                             // one kernel row: [kw][f][64 c]
  constexpr int kTile = 256 * 128;                                 // 256 pixels x 64 channels bf16
  uint8_t* wres = smem + (size_t)p.stages * kStage;
  uint8_t* stg = wres + 3 * kWTile;                                // one staging tile per epilogue group
  uint8_t* ybuf = stg + 2 * kTile;                                 // stats >= 2: kWideYSlots tiles of y2
  uint64_t* bars = reinterpret_cast<uint64_t*>(ybuf + (p.stats >= 2 ? kWideYSlots : 0) * kTile);
  uint64_t* full = bars;
  uint64_t* empty = bars + kMaxStages;
  uint64_t* tfull = bars + 2 * kMaxStages;
  uint64_t* tempty = tfull + 2;
  uint64_t* wfull = tempty + 2;
  uint64_t* yfull = wfull + 1;
  uint64_t* yempty = yfull + kWideYSlots;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(yempty + kWideYSlots);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* epi_go = reinterpret_cast<volatile int*>(tmem_slot + 2);
  constexpr uint32_t kTmemCols = 512;                              // two accumulators of 256 columns

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&tfull[a], 1);
      ptx::mbar_init(&tempty[a], 128);
    }
    for (int a = 0; a < kWideYSlots; ++a) {
      ptx::mbar_init(&yfull[a], 1);
      ptx::mbar_init(&yempty[a], 128);
    }
    ptx::mbar_init(wfull, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tm_x);
    ptx::prefetch_tmap(&tm_w);
    ptx::prefetch_tmap(&tm_y);
    ptx::prefetch_tmap(&tm_y2);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- producer: the CTA's weights once, then per tile one dh box and (stats >= 2) the y2 tile
    if (lane == 0 && blockIdx.x < p.total_tiles) {
      ptx::mbar_expect_tx(wfull, (uint32_t)(3 * kWTile));
#pragma unroll
      for (int kh = 0; kh < 3; ++kh) ptx::tma_load_4d(wres + kh * kWTile, &tm_w, wfull, (int)(blockIdx.x % p.n_tiles) * 64, 0, 0, kh);
    }
    __syncwarp();
    uint32_t tl = 0;
    for (int t = blockIdx.x; t < p.total_tiles; t += gridDim.x, ++tl) {
      const int m = t / p.n_tiles;
      const int w0 = (m % p.tiles_w) * 8, h0 = ((m / p.tiles_w) % p.tiles_h) * 32, n = m / (p.tiles_w * p.tiles_h);
      const int s = tl % p.stages;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&empty[s], ((tl / p.stages) & 1) ^ 1, abort_flag))) break;
      if (lane == 0) {
        ptx::mbar_expect_tx(&full[s], (uint32_t)kBox);
        ptx::tma_load_4d(smem + (size_t)s * kStage, &tm_x, &full[s], 0, w0 - 1, h0 - 1, n);
      }
      __syncwarp();
      if (p.stats >= 2) {
        const uint32_t slot = tl % kWideYSlots;
        if (!__all_sync(0xffffffffu, ptx::mbar_wait(&yempty[slot], ((tl / kWideYSlots) & 1) ^ 1, abort_flag))) break;
        if (lane == 0) {
          ptx::mbar_expect_tx(&yfull[slot], (uint32_t)kTile);
          ptx::tma_load_4d(ybuf + slot * kTile, &tm_y2, &yfull[slot], (t % p.n_tiles) * 64, w0, h0, n);
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ---------------- issuer: nine instructions per tile, D[channel][pixel] += Wa_mirrored(tap)[channel][f] * dh[pixel + tap][f]
    constexpr uint32_t idesc = ptx::idesc_bf16(64, 256, 1, 0);
    const uint64_t a_hi = ptx::sdesc(0, KC * 128, 1024, 2);          // weight tile of a tap: [f][64 c], MN-major
    const uint64_t b_hi = ptx::sdesc(0, 16, 10 * kARow, kALayout);   // pixels: next 8-pixel group = next box row
    const uint32_t w16 = ptx::smem_u32(wres) >> 4;
    uint32_t tl = 0;
    bool ok = blockIdx.x >= p.total_tiles || __all_sync(0xffffffffu, ptx::mbar_wait(wfull, 0, abort_flag));
    for (int t = blockIdx.x; ok && t < p.total_tiles; t += gridDim.x, ++tl) {
      const uint32_t acc = tl & 1, aph = (tl >> 1) & 1;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&tempty[acc], aph ^ 1, abort_flag))) break;
      ptx::tc_fence_after();
      const int s = tl % p.stages;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&full[s], (tl / p.stages) & 1, abort_flag))) break;
      ptx::tc_fence_after();
      if (lane == 0) {
        const uint32_t d = tmem_base + acc * 256;
        const uint32_t x16 = ptx::smem_u32(smem + (size_t)s * kStage) >> 4;
#pragma unroll
        for (int kh = 0; kh < 3; ++kh)
#pragma unroll
          for (int kw = 0; kw < 3; ++kw)
#pragma unroll
            for (int k = 0; k < KC / 16; ++k) {
              const uint64_t ad = a_hi | (uint64_t)(w16 + (2 - kh) * (kWTile >> 4) + (2 - kw) * (KC * 128 >> 4) + k * 128);
              const uint64_t bd = b_hi | (uint64_t)(x16 + ((kh * 10 + kw) * kARow >> 4) + k * 2);
              ptx::mma_f16(d, ad, bd, idesc, (kh | kw | k) != 0);
            }
        ptx::mma_commit(&empty[s]);
        ptx::mma_commit(&tfull[acc]);
      }
      __syncwarp();
    }
  } else {
    // ---------------- two epilogue groups of 128 threads; group g takes the tiles tl = g, g + 2, ... (accumulator g)
    const int grp = (threadIdx.x - 64) >> 7;
    const int et = (threadIdx.x - 64) & 127;
    uint8_t* const stg_g = stg + grp * kTile;
    const int lg = warp & 3;                     // lane quadrant of tensor memory: channels 16*lg .. 16*lg + 15 in lanes 0..15
    // sums / second pass: a thread owns 8 channels (one 16-byte chunk) and the 16 rows srg, srg + 16, ... of the 256
    const int schunk = et & 7, srg = et >> 3;
    float s1[8], s2[8], bsc[8], bsh[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) s1[i] = s2[i] = bsc[i] = bsh[i] = 0.f;
    if (p.stats >= 2) {
      const int c0 = (int)(blockIdx.x % p.n_tiles) * 64 + schunk * 8;
#pragma unroll
      for (int i = 0; i < 8; ++i) { bsc[i] = p.bn_scale[c0 + i]; bsh[i] = p.bn_shift[c0 + i]; }
      if (p.stats == 4) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float sc = bsc[i], m1 = p.bn_sdz[c0 + i] * p.inv_m, m2 = p.bn_sdzx[c0 + i] * p.inv_m, is = p.bn_invstd[c0 + i];
          s1[i] = -sc * m2 * is;
          s2[i] = sc * (m2 * is * p.bn_mu[c0 + i] - m1);
        }
      }
    }
    uint32_t tl = grp;
    for (int t = blockIdx.x + grp * gridDim.x; t < p.total_tiles; t += 2 * gridDim.x, tl += 2) {
      const int nt = t % p.n_tiles;
      const int m = t / p.n_tiles;
      const int w0 = (m % p.tiles_w) * 8, h0 = ((m / p.tiles_w) % p.tiles_h) * 32, n = m / (p.tiles_w * p.tiles_h);
      const uint32_t acc = grp, aph = (tl >> 1) & 1;
      ptx::mbar_wait(&tfull[acc], aph, abort_flag);
      ptx::tc_fence_after();
      if (et == 0) {
        ptx::tma_store_wait_read();              // the previous store of this group has read the staging tile
        epi_go[grp] = *abort_flag ? 0 : 1;
      }
      ptx::named_barrier(1 + grp, 128);
      if (!epi_go[grp]) break;
      const uint32_t tbase = tmem_base + ((uint32_t)(lg * 32) << 16) + acc * 256;
      // Transpose through the matrix-store instruction: a fragment load hands thread i channel i / 4 (and i / 4 + 8) of the
      // warp's 16 with two neighbouring pixels; as bfloat16 pairs these are the column fragments of 8 x 8 matrices whose
      // transposed store writes, per pixel, the 8 channels of a chunk as 16 contiguous bytes of the pixel-major tile.
      const uint32_t sbase = ptx::smem_u32(stg_g);
      const int mrow = lane & 7, mat = lane >> 3;                       // this thread addresses row mrow of matrix mat
      const uint32_t mchunk = (uint32_t)(2 * lg + (mat & 1));           // matrices 0, 2: channels 16 lg + 0..7; 1, 3: + 8..15
#pragma unroll 4
      for (int j = 0; j < 16; ++j) {             // 16 pixels at a time
        uint32_t v[8];
        ptx::tmem_ld_16x256b_x2(tbase + j * 16, v);
        ptx::tmem_ld_wait();
        uint32_t r[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {            // r[0]: ch 0-7, px 0-7; r[1]: ch 8-15, px 0-7; r[2], r[3]: px 8-15
          const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(v[2 * q]), __uint_as_float(v[2 * q + 1]));
          r[q] = *reinterpret_cast<const uint32_t*>(&b2);
        }
        const uint32_t px = (uint32_t)(j * 16 + (mat >> 1) * 8 + mrow);
        ptx::stmatrix_x4_trans(sbase + px * 128 + ((mchunk ^ (px & 7)) * 16), r[0], r[1], r[2], r[3]);
      }
      ptx::tc_fence_before();
      ptx::mbar_arrive(&tempty[acc]);
      ptx::fence_async_smem();
      ptx::named_barrier(1 + grp, 128);
      const uint32_t slot = tl % kWideYSlots;
      if (p.stats == 4) {
        ptx::mbar_wait(&yfull[slot], (tl / kWideYSlots) & 1, abort_flag);
        const uint8_t* yb = ybuf + slot * kTile;
#pragma unroll 4
        for (int rr = 0; rr < 16; ++rr) {
          const int row = srg + 16 * rr;
          const int off = row * 128 + ((schunk ^ (row & 7)) * 16);
          const uint4 dq = *reinterpret_cast<const uint4*>(stg_g + off);
          const uint4 yq = *reinterpret_cast<const uint4*>(yb + off);
          const uint32_t dw[4] = {dq.x, dq.y, dq.z, dq.w}, yw[4] = {yq.x, yq.y, yq.z, yq.w};
          uint32_t ow[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float d0 = __uint_as_float(dw[e] << 16), d1 = __uint_as_float(dw[e] & 0xffff0000u);
            const float y0 = __uint_as_float(yw[e] << 16), y1 = __uint_as_float(yw[e] & 0xffff0000u);
            const float z0 = fmaf(y0, bsc[2 * e], bsh[2 * e]) > 0.f ? d0 : 0.f;
            const float z1 = fmaf(y1, bsc[2 * e + 1], bsh[2 * e + 1]) > 0.f ? d1 : 0.f;
            const float o0 = fmaf(bsc[2 * e], z0, fmaf(s1[2 * e], y0, s2[2 * e]));
            const float o1 = fmaf(bsc[2 * e + 1], z1, fmaf(s1[2 * e + 1], y1, s2[2 * e + 1]));
            const __nv_bfloat162 b2 = __floats2bfloat162_rn(o0, o1);
            ow[e] = *reinterpret_cast<const uint32_t*>(&b2);
          }
          *reinterpret_cast<uint4*>(stg_g + off) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
        }
        ptx::mbar_arrive(&yempty[slot]);
        ptx::fence_async_smem();
        ptx::named_barrier(1 + grp, 128);
      }
      if (et == 0 && p.stats != 3) {
        ptx::tma_store_4d(&tm_y, stg_g, nt * 64, w0, h0, n);
        ptx::tma_store_commit();
      }
      if (p.stats == 2 || p.stats == 3) {
        ptx::mbar_wait(&yfull[slot], (tl / kWideYSlots) & 1, abort_flag);
        const uint8_t* yb = ybuf + slot * kTile;
#pragma unroll 4
        for (int rr = 0; rr < 16; ++rr) {
          const int row = srg + 16 * rr;
          const bool rv = h0 + (row >> 3) < p.H;  // a last tile row may reach below the image: those pixels count for nothing
          const int off = row * 128 + ((schunk ^ (row & 7)) * 16);
          const uint4 dq = *reinterpret_cast<const uint4*>(stg_g + off);
          const uint4 yq = *reinterpret_cast<const uint4*>(yb + off);
          const uint32_t dw[4] = {dq.x, dq.y, dq.z, dq.w}, yw[4] = {yq.x, yq.y, yq.z, yq.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float d0 = __uint_as_float(dw[e] << 16), d1 = __uint_as_float(dw[e] & 0xffff0000u);
            const float y0 = __uint_as_float(yw[e] << 16), y1 = __uint_as_float(yw[e] & 0xffff0000u);
            const float z0 = rv && fmaf(y0, bsc[2 * e], bsh[2 * e]) > 0.f ? d0 : 0.f;
            const float z1 = rv && fmaf(y1, bsc[2 * e + 1], bsh[2 * e + 1]) > 0.f ? d1 : 0.f;
            s1[2 * e] += z0;
            s1[2 * e + 1] += z1;
            s2[2 * e] = fmaf(z0, y0, s2[2 * e]);
            s2[2 * e + 1] = fmaf(z1, y1, s2[2 * e + 1]);
          }
        }
        ptx::mbar_arrive(&yempty[slot]);
      }
    }
    if (et == 0) ptx::tma_store_wait_all();
    if (p.stats == 2 || p.stats == 3)  // one partial per epilogue group, as in the folded kernel
      fold_group_partial(s1, s2, reinterpret_cast<float*>(stg_g), grp, lg, lane, true, p.bn_mu, p.bn_invstd,
                         (int)(blockIdx.x % p.n_tiles) * 64, p.red + ((size_t)(blockIdx.x / p.n_tiles) * 2 + grp) * 2 * p.Cout, p.Cout);
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, NF_ETIMEOUT);
    const unsigned long long t0 = ptx::globaltimer();
    while (ptx::globaltimer() - t0 < 2000000ull) __nanosleep(1000);
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------- weight gradient
// dW[tap][co][ci] = sum over pixels of dy[pixel, co] * x[pixel shifted by tap, ci].  The K dimension of the
// GEMM is the pixel index, so both operands are MN-major in shared memory exactly as TMA delivers the
// channels-last tiles.  Work is split over (64-input-channel chunk, output-channel chunk) pairs and over
// the pixel tiles (split-K): accumulators stay in tensor memory over a CTA's whole pixel range and are
// written as per-CTA partials that a second kernel sums in a fixed order.  Two kernels: the per-tap form
// below (stride 2 and small feature maps) and conv_wgrad_kw_kernel (stride 1).
struct WgParams {
  int N, H, W, Cin, Cout;
  int BW, BH, tiles_w, tiles_h, pix_tiles, ci_chunks, co_chunks, splits, stages, stride, BI;
  float* part;      // [splits][9][Cout][Cin]
  int32_t* status;
};

// NB = width of the output-gradient tile in channels (64: main conv, one 64-channel chunk per CTA;
// 16/32/64: aux conv with F <= NB filters, rows of 2*NB bytes with the matching TMA swizzle).
// Per-tap form (S2 is always 1): stride-2 convolutions, and feature maps smaller than a tile where a tile
// spans BI whole images.  The shifted activation tiles are gathered by TMA, with element stride 2 for
// stride 2, one 128-pixel tile per tap; a CTA then owns one kernel row kh (grid dimension) with its three column
// taps: taps (kh,0) and (kh,1) stacked in one instruction, tap (kh,2) in a second, half-empty one.
template <int NB, int S2>
__global__ void __launch_bounds__(kThreads, 1)
conv_wgrad_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_dy, const WgParams p) {
  constexpr int kAtoms = NB > 64 ? NB / 64 : 1;                // 64-channel atoms of the dy tile (NB = 128, 256: main conv only)
  constexpr int kBRow = (NB > 64 ? 64 : NB) * 2;               // bytes of one pixel row of one atom
  constexpr uint32_t kBLayout = NB >= 64 ? 2 : NB == 32 ? 4 : 6;  // swizzle of that tile
  constexpr int kBTile = 128 * kBRow;                          // one atom
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  static_assert(S2 == 1, "stride 1 on tileable maps uses conv_wgrad_kw_kernel");
  constexpr int kStages = NB > 64 ? 2 : 3;
  constexpr int kJobs = 2;  // instructions (accumulators) per 16 pixels
  constexpr int copy_bytes = 16384;  // one 128-pixel tap tile
  const int stage_bytes = 3 * copy_bytes + kAtoms * 16384;  // a dy atom always gets 16 KB so the unused rows read by the
                                                            // half-empty last instruction stay inside the stage
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)kStages * stage_bytes);
  uint64_t* full = bars;
  uint64_t* empty = bars + kStages;
  uint64_t* done = bars + 2 * kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(done + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  constexpr uint32_t kNeed = kJobs * NB;
  constexpr uint32_t kCols = kNeed <= 32 ? 32 : kNeed <= 64 ? 64 : kNeed <= 128 ? 128 : kNeed <= 256 ? 256 : 512;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blocks = p.ci_chunks * p.co_chunks;
  const int blk = blockIdx.x % blocks;
  const int rest = blockIdx.x / blocks;
  const int khg = rest % 3;  // kernel row owned by this CTA
  const int sp = rest / 3;
  const int cic = blk % p.ci_chunks, coc = blk / p.ci_chunks;
  const int t0 = (int)((long)p.pix_tiles * sp / p.splits), t1 = (int)((long)p.pix_tiles * (sp + 1) / p.splits);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
    }
    ptx::mbar_init(done, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tm_x);
    ptx::prefetch_tmap(&tm_dy);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    uint32_t it = 0;
    for (int t = t0; t < t1; ++t, ++it) {
      const int s = it % kStages;
      const uint32_t ph = (it / kStages) & 1;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&empty[s], ph ^ 1, abort_flag))) break;
      if (lane == 0) {
        const int w0 = (t % p.tiles_w) * p.BW, h0 = ((t / p.tiles_w) % p.tiles_h) * p.BH, n = (t / (p.tiles_w * p.tiles_h)) * p.BI;
        uint8_t* st = smem + (size_t)s * stage_bytes;
        ptx::mbar_expect_tx(&full[s], (uint32_t)(3 * copy_bytes + kAtoms * kBTile));
#pragma unroll
        for (int kw = 0; kw < 3; ++kw)
          ptx::tma_load_4d(st + kw * copy_bytes, &tm_x, &full[s], cic * 64, p.stride * w0 + kw - 1, p.stride * h0 + khg - 1, n);
#pragma unroll
        for (int a = 0; a < kAtoms; ++a)
          ptx::tma_load_4d(st + 3 * copy_bytes + a * 16384, &tm_dy, &full[s], coc * NB + a * 64, w0, h0, n);
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    constexpr uint32_t idesc = ptx::idesc_bf16(128, NB, 1, 1);
    uint32_t it = 0;
    bool ok = true;
    for (int t = t0; t < t1; ++t, ++it) {
      const int s = it % kStages;
      const uint32_t ph = (it / kStages) & 1;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&full[s], ph, abort_flag))) { ok = false; break; }
      ptx::tc_fence_after();
      if (lane == 0) {
        const uint32_t xb = ptx::smem_u32(smem + (size_t)s * stage_bytes);
        const uint32_t x16 = xb >> 4, g16 = (xb + 3 * copy_bytes) >> 4;
        const uint32_t copy16 = (uint32_t)copy_bytes >> 4;
        // descriptors differ only in the address field; the second stacked chunk sits one tap tile further
        const uint64_t a_copy_hi = ptx::sdesc(0, copy_bytes, 1024, 2);
        const uint64_t b_hi = ptx::sdesc(0, 16384, 8 * kBRow, kBLayout);  // next 64-channel atom: 16 KB further
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t k16 = k * 128;  // 16 pixels x 128 bytes, in 16-byte units
          const uint64_t bd = b_hi | (uint64_t)(g16 + k * kBRow);
          const uint32_t acc = (it | k) != 0;
          // taps (kh,0) and (kh,1): second chunk one tile further; tap (kh,2): rows 64..127 unused
          ptx::mma_f16(tmem_base, a_copy_hi | (uint64_t)(x16 + k16), bd, idesc, acc);
          ptx::mma_f16(tmem_base + NB, a_copy_hi | (uint64_t)(x16 + 2 * copy16 + k16), bd, idesc, acc);
        }
        ptx::mma_commit(&empty[s]);
      }
      __syncwarp();
    }
    if (ok && lane == 0) ptx::mma_commit(done);
    __syncwarp();
  } else {
    // epilogue: after the last MMA, lane m of tensor memory = row m of the stacked (tap, ci) chunks
    const int lg = warp & 3, m = lg * 32 + lane;
    if (ptx::mbar_wait(done, 0, abort_flag) && t1 > t0) {
      ptx::tc_fence_after();
      const size_t plane = (size_t)p.Cout * p.Cin;
      float* base = p.part + (size_t)sp * 9 * plane + (size_t)(coc * NB) * p.Cin + cic * 64 + (m & 63);
      const int co_left = p.Cout - coc * NB;  // output channels of this chunk that exist (aux: F may be < NB)
#pragma unroll 1
      for (int j = 0; j < kJobs; ++j) {
        // taps of accumulator j: rows 0..63 -> tapA, rows 64..127 -> tapB (kh*3+kw)
        const int tapA = khg * 3 + (j == 0 ? 0 : 2);
        const int tapB = j == 0 ? khg * 3 + 1 : -1;
        const int tap = m < 64 ? tapA : tapB;
#pragma unroll 2
        for (int q = 0; q < NB / 16; ++q) {  // not fully unrolled: 16 column blocks of address arithmetic spill at NB = 256
          uint32_t v[16];
          ptx::tmem_ld16(tmem_base + ((uint32_t)(lg * 32) << 16) + j * NB + q * 16, v);
          ptx::tmem_ld_wait();
          if (tap >= 0) {
            float* dst = base + (size_t)tap * plane + (size_t)(q * 16) * p.Cin;
#pragma unroll
            for (int e = 0; e < 16; ++e)
              if (q * 16 + e < co_left) dst[(size_t)e * p.Cin] = __uint_as_float(v[e]);
          }
        }
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, NF_ETIMEOUT);
    const unsigned long long tt = ptx::globaltimer();
    while (ptx::globaltimer() - tt < 2000000ull) __nanosleep(1000);
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kCols);
  }
}

// ---------------------------------------------------------------- weight gradient, stride 1, column shift on the gradient
// dW[kh,kw][co][ci] = sum_{i,j} dy[i,j,co] * x[i+kh-1, j+kw-1, ci].  With j' = j+kw-1 this is
//   sum over the pixels (i,j') of the x grid of  x[i+kh-1, j', ci] * dy[i, j'-kw+1, co]   (dy = 0 outside),
// so the column tap can sit on the gradient operand: ONE activation box (BH+2 rows, no column copies)
// and three column-shifted gradient tiles per stage.  Per 16 pixels two instructions:
//   A (M = 128) = rows kh=0 and kh=1 of the box stacked (second one half empty: kh=2 + unused rows),
//   B (N = 3*NB) = the three shifted gradient tiles side by side (MN-major atoms one tile apart).
// Fewer operand bytes per useful FLOP than stacking all nine taps on the activation side.
template <int NB>
__global__ void __launch_bounds__(kThreads, 1)
conv_wgrad_kw_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_dy, const WgParams p) {
  constexpr int kBRow = NB * 2;
  constexpr uint32_t kBLayout = NB == 64 ? 2 : NB == 32 ? 4 : 6;
  constexpr int kBTile = 128 * kBRow;                 // one shifted gradient tile
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int box_bytes = (p.BH + 2) * p.BW * 128;
  const int g_region = 3 * kBTile < 4096 ? 4096 : 3 * kBTile;  // >= 32 rows after the box for the unused operand rows
  const int stage_bytes = box_bytes + g_region;
  const int stages = p.stages;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)stages * stage_bytes);
  uint64_t* full = bars;
  uint64_t* empty = bars + kMaxStages;
  uint64_t* done = bars + 2 * kMaxStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(done + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  constexpr uint32_t kAcc = NB == 64 ? 256 : 3 * NB <= 64 ? 64 : 128;  // columns reserved per accumulator
  constexpr uint32_t kCols = 2 * kAcc;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blocks = p.ci_chunks * p.co_chunks;
  const int blk = blockIdx.x % blocks, sp = blockIdx.x / blocks;
  const int cic = blk % p.ci_chunks, coc = blk / p.ci_chunks;
  const int t0 = (int)((long)p.pix_tiles * sp / p.splits), t1 = (int)((long)p.pix_tiles * (sp + 1) / p.splits);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
    }
    ptx::mbar_init(done, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tm_x);
    ptx::prefetch_tmap(&tm_dy);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    uint32_t it = 0;
    for (int t = t0; t < t1; ++t, ++it) {
      const int s = it % stages;
      const uint32_t ph = (it / stages) & 1;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&empty[s], ph ^ 1, abort_flag))) break;
      if (lane == 0) {
        const int w0 = (t % p.tiles_w) * p.BW, h0 = ((t / p.tiles_w) % p.tiles_h) * p.BH, n = t / (p.tiles_w * p.tiles_h);
        uint8_t* st = smem + (size_t)s * stage_bytes;
        ptx::mbar_expect_tx(&full[s], (uint32_t)(box_bytes + 3 * kBTile));
        ptx::tma_load_4d(st, &tm_x, &full[s], cic * 64, w0, h0 - 1, n);
#pragma unroll
        for (int kw = 0; kw < 3; ++kw)  // gradient column j = j' - kw + 1
          ptx::tma_load_4d(st + box_bytes + kw * kBTile, &tm_dy, &full[s], coc * NB, w0 - kw + 1, h0, n);
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    constexpr uint32_t idesc = ptx::idesc_bf16(128, 3 * NB, 1, 1);
    const uint64_t a_hi = ptx::sdesc(0, p.BW * 128, 1024, 2);      // second 64 rows: one image row further
    const uint64_t b_hi = ptx::sdesc(0, kBTile, 8 * kBRow, kBLayout);  // next N atom: next shifted tile
    const uint32_t row16 = (uint32_t)(p.BW * 128) >> 4;
    uint32_t it = 0;
    bool ok = true;
    for (int t = t0; t < t1; ++t, ++it) {
      const int s = it % stages;
      const uint32_t ph = (it / stages) & 1;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&full[s], ph, abort_flag))) { ok = false; break; }
      ptx::tc_fence_after();
      if (lane == 0) {
        const uint32_t xb = ptx::smem_u32(smem + (size_t)s * stage_bytes);
        const uint32_t x16 = xb >> 4, g16 = (xb + box_bytes) >> 4;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint64_t bd = b_hi | (uint64_t)(g16 + k * kBRow);   // 16 pixels x kBRow bytes = k * kBRow sixteen-byte units
          const uint32_t acc = (it | k) != 0;
          ptx::mma_f16(tmem_base, a_hi | (uint64_t)(x16 + k * 128), bd, idesc, acc);                      // kh = 0 | 1
          ptx::mma_f16(tmem_base + kAcc, a_hi | (uint64_t)(x16 + 2 * row16 + k * 128), bd, idesc, acc);  // kh = 2 | unused
        }
        ptx::mma_commit(&empty[s]);
      }
      __syncwarp();
    }
    if (ok && lane == 0) ptx::mma_commit(done);
    __syncwarp();
  } else {
    const int lg = warp & 3, m = lg * 32 + lane;
    if (ptx::mbar_wait(done, 0, abort_flag) && t1 > t0) {
      ptx::tc_fence_after();
      const size_t plane = (size_t)p.Cout * p.Cin;
      float* base = p.part + (size_t)sp * 9 * plane + (size_t)(coc * NB) * p.Cin + cic * 64 + (m & 63);
      const int co_left = p.Cout - coc * NB;
#pragma unroll 1
      for (int j = 0; j < 2; ++j) {
        const int kh = j == 0 ? (m < 64 ? 0 : 1) : (m < 64 ? 2 : -1);
#pragma unroll 1
        for (int kw = 0; kw < 3; ++kw)
#pragma unroll
          for (int q = 0; q < NB / 16; ++q) {
            uint32_t v[16];
            ptx::tmem_ld16(tmem_base + ((uint32_t)(lg * 32) << 16) + j * kAcc + kw * NB + q * 16, v);
            ptx::tmem_ld_wait();
            if (kh >= 0) {
              float* dst = base + (size_t)(kh * 3 + kw) * plane + (size_t)(q * 16) * p.Cin;
#pragma unroll
              for (int e = 0; e < 16; ++e)
                if (q * 16 + e < co_left) dst[(size_t)e * p.Cin] = __uint_as_float(v[e]);
            }
          }
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, NF_ETIMEOUT);
    const unsigned long long tt = ptx::globaltimer();
    while (ptx::globaltimer() - tt < 2000000ull) __nanosleep(1000);
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kCols);
  }
}

// ---------------------------------------------------------------- weight gradient, stride 1, few filters: gradient on the M side
// An instruction holds the tensor pipe for about the same time whatever its shape, so for the auxiliary conv
// (F <= 32 filters) the fewest instructions win.  Here the roles of conv_wgrad_kw_kernel are swapped:
//   A (M = 4 * NB rows) = the three column-shifted gradient tiles as consecutive MN-major atoms (kw, f) plus one unused atom,
//   B (N = 192)         = the three row taps of the activation box as consecutive 64-channel atoms (kh, ci),
// so ONE instruction per 16 pixels produces all nine taps: D[(kw, f), (kh, ci)].  NB = 16 uses the 64-row shape
// (row r in TMEM lane 32 * (r / 16) + r % 16), NB = 32 the 128-row shape (row r in lane r); in both, the warp of
// lane quadrant q holds column tap kw = q and lane l holds filter f = l.
template <int NB>
__global__ void __launch_bounds__(kThreads, 1)
conv_wgrad_gx_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_dy, const WgParams p) {
  constexpr int kBRow = NB * 2;
  constexpr uint32_t kGLayout = NB == 32 ? 4 : 6;
  constexpr int kGTile = 128 * kBRow;                 // one shifted gradient tile
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int box_bytes = (p.BH + 2) * p.BW * 128;
  const int stage_bytes = box_bytes + 4 * kGTile;     // the fourth atom is never loaded: its accumulator rows are not read
  const int stages = p.stages;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)stages * stage_bytes);
  uint64_t* full = bars;
  uint64_t* empty = bars + kMaxStages;
  uint64_t* done = bars + 2 * kMaxStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(done + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  constexpr uint32_t kCols = 256;                     // 192 accumulator columns

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cic = blockIdx.x % p.ci_chunks, sp = blockIdx.x / p.ci_chunks;
  const int t0 = (int)((long)p.pix_tiles * sp / p.splits), t1 = (int)((long)p.pix_tiles * (sp + 1) / p.splits);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
    }
    ptx::mbar_init(done, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tm_x);
    ptx::prefetch_tmap(&tm_dy);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    uint32_t it = 0;
    for (int t = t0; t < t1; ++t, ++it) {
      const int s = it % stages;
      const uint32_t ph = (it / stages) & 1;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&empty[s], ph ^ 1, abort_flag))) break;
      if (lane == 0) {
        const int w0 = (t % p.tiles_w) * p.BW, h0 = ((t / p.tiles_w) % p.tiles_h) * p.BH, n = t / (p.tiles_w * p.tiles_h);
        uint8_t* st = smem + (size_t)s * stage_bytes;
        ptx::mbar_expect_tx(&full[s], (uint32_t)(box_bytes + 3 * kGTile));
        ptx::tma_load_4d(st, &tm_x, &full[s], cic * 64, w0, h0 - 1, n);
#pragma unroll
        for (int kw = 0; kw < 3; ++kw)  // gradient column j = j' - kw + 1
          ptx::tma_load_4d(st + box_bytes + kw * kGTile, &tm_dy, &full[s], 0, w0 - kw + 1, h0, n);
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    constexpr uint32_t idesc = ptx::idesc_bf16(4 * NB, 192, 1, 1);
    const uint64_t a_hi = ptx::sdesc(0, kGTile, 8 * kBRow, kGLayout);  // next M atom: next shifted tile
    const uint64_t b_hi = ptx::sdesc(0, p.BW * 128, 1024, 2);          // next N atom: one image row further (next kh)
    uint32_t it = 0;
    bool ok = true;
    for (int t = t0; t < t1; ++t, ++it) {
      const int s = it % stages;
      const uint32_t ph = (it / stages) & 1;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&full[s], ph, abort_flag))) { ok = false; break; }
      ptx::tc_fence_after();
      if (lane == 0) {
        const uint32_t xb = ptx::smem_u32(smem + (size_t)s * stage_bytes);
        const uint32_t x16 = xb >> 4, g16 = (xb + box_bytes) >> 4;
#pragma unroll
        for (int k = 0; k < 8; ++k)
          ptx::mma_f16(tmem_base, a_hi | (uint64_t)(g16 + k * kBRow), b_hi | (uint64_t)(x16 + k * 128), idesc, (it | k) != 0);
        ptx::mma_commit(&empty[s]);
      }
      __syncwarp();
    }
    if (ok && lane == 0) ptx::mma_commit(done);
    __syncwarp();
  } else {
    const int lg = warp & 3;  // = column tap kw of this warp's rows
    if (ptx::mbar_wait(done, 0, abort_flag) && t1 > t0) {
      ptx::tc_fence_after();
      const size_t plane = (size_t)p.Cout * p.Cin;
      const bool mine = lg < 3 && lane < NB && lane < p.Cout;
      float* base = p.part + (size_t)sp * 9 * plane + (size_t)lg * plane + (size_t)lane * p.Cin + cic * 64;
#pragma unroll 1
      for (int kh = 0; kh < 3; ++kh)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t v[16];
          ptx::tmem_ld16(tmem_base + ((uint32_t)(lg * 32) << 16) + kh * 64 + q * 16, v);
          ptx::tmem_ld_wait();
          if (mine) {
            float4* dst = reinterpret_cast<float4*>(base + (size_t)(kh * 3) * plane + q * 16);
#pragma unroll
            for (int e = 0; e < 4; ++e)
              dst[e] = make_float4(__uint_as_float(v[4 * e]), __uint_as_float(v[4 * e + 1]), __uint_as_float(v[4 * e + 2]),
                                   __uint_as_float(v[4 * e + 3]));
          }
        }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, NF_ETIMEOUT);
    const unsigned long long tt = ptx::globaltimer();
    while (ptx::globaltimer() - tt < 2000000ull) __nanosleep(1000);
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kCols);
  }
}

__global__ void __launch_bounds__(256) sum_parts_kernel(const float* __restrict__ part, int splits, size_t n, float* __restrict__ out) {
  // 32 consecutive elements x 8 lanes over the splits; each lane adds its splits in index order, lane sums are added in lane order
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

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor, 4 dims (innermost first), zero fill outside; the swizzle span equals the inner box (32/64/128 bytes)
int make_map4(CUtensorMap* m, const void* base, const uint64_t dims[4], const uint32_t box[4], int spatial_stride = 1) {
  const CUtensorMapSwizzle sw = box[0] * 2 >= 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                : box[0] * 2 == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
  EncodeTiledFn fn = encode_fn();
  if (!fn) return NF_ECUDA;
  cuuint64_t gdim[4] = {dims[0], dims[1], dims[2], dims[3]};
  cuuint64_t gstr[3] = {dims[0] * 2, dims[0] * dims[1] * 2, dims[0] * dims[1] * dims[2] * 2};
  // with an element stride s along w and h the box spans s*box elements and keeps every s-th one
  const cuuint32_t ss = (cuuint32_t)spatial_stride;
  cuuint32_t bx[4] = {box[0], box[1] * ss, box[2] * ss, box[3]};
  cuuint32_t es[4] = {1, ss, ss, 1};
  const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), gdim, gstr, bx, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? NF_OK : nf_cuda_check(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
}

// Per-process caches (kernel attributes, SM count, symbol addresses) are kept per device: a process may use several.
constexpr int kMaxDevices = 64;
int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
  return dev;
}

int sm_count() {
  static int n_dev[kMaxDevices];
  const int dev = current_device();
  int& n = n_dev[dev];
  if (!n) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
  }
  return n;
}

// mode 0: main forward (y + statistics), 1: aux forward (bias + ReLU, Cout = F), 2: aux input gradient
// (Cin = F <= 64 and a multiple of 8, Cout a multiple of 64, mirrored MN-major weights).
// H, W: OUTPUT size (equal to the input size for stride 1).
// Pixel tile of 128 output pixels: a BW x BH patch of one image, or (per-tap mode only) BI whole images
// of a small feature map.  Returns false when the size does not tile.
bool pick_tile(int H, int W, bool allow_multi, int* BW, int* BH, int* BI) {
  const int cand[3][2] = {{16, 8}, {32, 4}, {8, 16}};
  for (auto& c : cand)
    if (W % c[0] == 0 && H % c[1] == 0) {
      *BW = c[0]; *BH = c[1]; *BI = 1;
      return true;
    }
  if (allow_multi && W * H <= 64 && 128 % (W * H) == 0 && (W & (W - 1)) == 0) {  // 8x8, 4x4, 2x2, 8x4, 1x1 ...
    *BW = W; *BH = H; *BI = 128 / (W * H);
    return true;
  }
  return false;
}

// ybuf = 1 reserves the y2 tile of the fused BatchNorm-backward sums (as large as the output staging)
TcPlan plan_fwd(int H, int W, int Cin, int Cout, int N, int epi = 0, int stride = 1, int ybuf = 0) {
  TcPlan pl{};
  if (stride == 2 && (epi != 0 || Cin % 64)) return pl;
  if (epi == 2 ? (Cin > 64 || Cin % 8 || Cout % 64) : (Cin % 64 != 0)) return pl;
  if (epi == 0 ? (Cout % 64 != 0) : epi == 1 ? (Cout > 64) : false) return pl;
  if (!pick_tile(H, W, true, &pl.BW, &pl.BH, &pl.BI)) return pl;
  pl.PT = (stride == 2 || pl.BI > 1) ? 1 : 0;
  if (epi == 0 && Cout % 256 == 0) pl.PT = 1;  // 256-wide instructions need the per-tap form (one tap of weights per stage)
  pl.BN = epi != 1 ? (Cout % 128 == 0 ? 128 : 64) : (Cout <= 16 ? 16 : Cout <= 32 ? 32 : 64);
  if (epi == 0 && pl.PT && Cout % 256 == 0) pl.BN = 256;  // per-tap form: weights of one tap and 256 channels are 32 KB a stage
  pl.KC = epi == 2 ? (Cin <= 16 ? 16 : Cin <= 32 ? 32 : 64) : 64;
  const size_t a_stride = pl.PT ? (size_t)128 * pl.KC * 2 : ((size_t)(pl.BH + 2) * pl.BW * pl.KC * 2 + 1023) & ~(size_t)1023;
  pl.RW = (!pl.PT && epi != 2 && Cin == 64 && pl.BN <= 64) ? 1 : 0;  // weights resident in shared memory
  const size_t b_stage = pl.RW ? 0 : pl.PT ? (epi == 2 ? (size_t)(pl.BN / 64) * pl.KC * 128 : (size_t)pl.BN * 128)
                                           : epi == 2 ? (size_t)(pl.BN / 64) * 3 * pl.KC * 128 : (size_t)3 * pl.BN * 128;
  const size_t stage = ((a_stride + 1023) & ~(size_t)1023) + b_stage;
  const size_t fixed = (size_t)(epi != 1 ? pl.BN / 64 : 0) * 16384 * (ybuf ? 2 : 1) + (pl.RW ? (size_t)9 * pl.BN * 128 : 0) + 1024 + 1024;
  int st = (int)((232448 - fixed) / stage);
  if (st > kMaxStages) st = kMaxStages;
  if (st < 2) return pl;
  pl.stages = st;
  pl.smem = (size_t)st * stage + fixed;
  pl.parts = pl.BN >= 128 ? 1 : 128 / pl.BN;
  const int n_tiles = epi != 1 ? Cout / pl.BN : 1;
  const long total = (long)((N + pl.BI - 1) / pl.BI) * (H / pl.BH) * (W / pl.BW) * n_tiles;
  long g = sm_count();
  g -= g % n_tiles;  // every CTA keeps one channel tile for its whole life
  if (g < n_tiles) g = n_tiles;
  if (g > total) g = total;
  pl.grid = (int)g;
  pl.ok = 1;
  return pl;
}

template <int BN, int EPI, int KC = 64, int BMN = 0, int PT = 0, int RW = 0>
int launch_fwd(const TcPlan& pl, const CUtensorMap& mx, const CUtensorMap& mw, const CUtensorMap& my, const FwdParams& p) {
  static bool attr_done_dev[kMaxDevices];  // function attributes belong to a device's context: set once per device
  bool& attr_done = attr_done_dev[current_device()];
  if (!attr_done) {
    NF_CUDA(cudaFuncSetAttribute(conv_fwd_tc_kernel<BN, EPI, KC, BMN, PT, RW>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448));
    attr_done = true;
  }
  conv_fwd_tc_kernel<BN, EPI, KC, BMN, PT, RW><<<pl.grid, kThreads, pl.smem, g_nf_stream>>>(mx, mw, my, p);
  NF_LAUNCHED();
  return NF_OK;
}

// The folded-tap kernel covers, when W % 14 == 0 and H % 8 == 0: the main forward 64 -> 64 (epi 0), the aux
// forward with F <= 64, F % 8 == 0 (epi 1) if all weight tiles fit in shared memory beside >= 3 activation
// stages, and the aux input gradient F -> Cout (epi 2; F <= 32, F % 8 == 0, Cout % 64 == 0).  The input gradient
// also takes widths that tile by 16 instead of 14 (its unfolded form): always with the fused BatchNorm-backward
// sums (stats 2) or 64 output channels; without the sums a wider layer is faster on the generic kernel's
// 128-channel tiles (measured).
int fold_group(int Cout, int epi) { return epi != 1 ? 64 : (Cout <= 16 ? 16 : Cout <= 32 ? 32 : 64); }
// widths the 14-column tiles of the folded forward cover: multiples of 14, and wider maps whose ragged last tile column wastes
// at most a third (32, 48, 64, ...: the zero-filled loads and clipped stores of TMA make the overhang harmless)
bool fold_width_ok(int W) { return W % 14 == 0 || (W >= 28 && ((W + 13) / 14) * 14 * 3 <= W * 4); }

bool fold_ok(int H, int W, int Cin, int Cout, int epi, int stride, int stats = 0, size_t extra_smem = 0) {
  if (stride != 1 || H % 8) return false;
  if (epi == 2 && W % 14 && W % 16 == 0 && (stats >= 2 || Cout == 64)) return Cin <= 32 && Cin % 8 == 0 && Cout % 64 == 0;
  if (epi == 2 ? W % 14 != 0 : !fold_width_ok(W)) return false;
  // the plain aux forward (no fused normalisation: extra_smem == 0) stays on the generic kernel for ragged widths: with 64
  // filters at 32 columns the folded form measured slower there (0.33 vs 0.25 ms), the fused form faster everywhere
  if (epi == 1 && W % 14 != 0 && extra_smem == 0) return false;
  if (epi == 2) return Cin <= 32 && Cin % 8 == 0 && Cout % 64 == 0;
  if (Cin % 64) return false;
  if (epi == 0 ? (Cin != 64 || Cout != 64) : (Cout > 64 || Cout % 8)) return false;
  const size_t wbytes = (size_t)9 * (Cin / 64) * fold_group(Cout, epi) * 128;
  return wbytes + (epi == 0 ? 2 * 16384 : 0) + extra_smem + 2048 + 3 * 20480 <= 232448;
}

template <int G, int EPI, int KC = 64, int MIR = 0, int UF = 0, int XF = 0>
int launch_fold(int grid, size_t smem, const CUtensorMap& mx, const CUtensorMap& mw, const CUtensorMap& my, const CUtensorMap& my2,
                const FoldParams& p) {
  static bool attr_done_dev[kMaxDevices];  // function attributes belong to a device's context: set once per device
  bool& attr_done = attr_done_dev[current_device()];
  if (!attr_done) {
    NF_CUDA(cudaFuncSetAttribute(conv_fwd_fold_kernel<G, EPI, KC, MIR, UF, XF>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448));
    attr_done = true;
  }
  conv_fwd_fold_kernel<G, EPI, KC, MIR, UF, XF><<<grid, kFoldThreads + kXfThreads * XF, smem, g_nf_stream>>>(mx, mw, my, my2, p);
  NF_LAUNCHED();
  return NF_OK;
}

// BatchNorm-backward inputs of the fused reduction (stats 2): y2 has the shape of the output
struct BnBwdIn {
  const void* y2;
  const float *scale, *shift, *mu, *invstd;
  const float *sdz = nullptr, *sdzx = nullptr;  // second pass (stats 4): the reduced sums and 1 / (elements per channel)
  float inv_m = 0.f;
};

// Normalisation fused into the aux forward (epi 1): x is then the conv output and a = ReLU(x*scale + shift) is written to a
struct XfIn {
  const float *scale, *shift;
  void* a;
  float* pool_part;  // non-null: pooling partials and sign mask instead of h (see FoldParams)
  uint8_t* mask;
};

int run_fold(int N, int H, int W, int Cin, int Cout, const void* x, const void* w, void* y, int stats, float* red,
             size_t red_floats, int32_t* status, int* nb, int epi, const float* bias, const BnBwdIn* bn = nullptr,
             const XfIn* xf = nullptr) {
  const int G = fold_group(Cout, epi);
  const int KC = epi == 2 ? (Cin <= 16 ? 16 : 32) : 64;
  // input gradient on widths that also tile by 16: the unfolded form (three shifted boxes, no shift-add in the epilogue);
  // where the map tiles by 8 x 16 as well: its single-box form
  const bool uf = epi == 2 && W % 16 == 0;
  const bool uf2 = uf && H % 16 == 0;
  // ... and by 8 x 32 with 16 channels of dh: the form with 256 pixels per instruction
  const bool wide = uf2 && KC == 16;  // H % 16 == 0: the last tile row may be half a tile
  const int TW = uf2 ? 8 : uf ? 16 : 14, TH = wide ? 32 : uf2 ? 16 : 8;
  CUtensorMap mx, mw, my, my2;
  const uint64_t dx[4] = {(uint64_t)Cin, (uint64_t)W, (uint64_t)H, (uint64_t)N};
  const uint32_t bx[4] = {(uint32_t)KC, (uint32_t)(uf2 ? 10 : 16), (uint32_t)(wide ? 34 : uf2 ? 18 : 10), 1};
  // forward: weights [kh][kw][Cout][Cin], box = G rows of co x 64 ci for the three kw of one kh;
  // input gradient: weights [kh][kw][F][Cout], box = KC rows of f x 64 c for the three kw of one kh
  const uint64_t dw[4] = {(uint64_t)(epi == 2 ? Cout : Cin), (uint64_t)(epi == 2 ? Cin : Cout), 3, 3};
  const uint32_t bw[4] = {64, (uint32_t)(epi == 2 ? KC : G), 3, 1};
  const uint64_t dy[4] = {(uint64_t)Cout, (uint64_t)W, (uint64_t)H, (uint64_t)N};
  const uint32_t by[4] = {64, (uint32_t)TW, (uint32_t)TH, 1};
  int rc;
  if ((rc = make_map4(&mx, x, dx, bx)) != NF_OK) return rc;
  if ((rc = make_map4(&mw, w, dw, bw)) != NF_OK) return rc;
  if (epi != 1) {
    if ((rc = make_map4(&my, y, dy, by)) != NF_OK) return rc;
  } else {
    my = mx;
  }
  if (xf) {  // the normalised activation leaves the aux forward through TMA stores of 14 x 8-pixel tiles, 64 channels each
    const uint32_t ba[4] = {64, 14, 8, 1};
    if ((rc = make_map4(&my, xf->a, dx, ba)) != NF_OK) return rc;
  }
  my2 = my;
  if (stats >= 2) {
    if (epi != 2 || !bn || (stats == 4 && (!bn->sdz || !bn->sdzx))) return NF_EINVAL;
    if ((rc = make_map4(&my2, bn->y2, dy, by)) != NF_OK) return rc;
  }
  FoldParams p{};
  if (bn) {
    p.bn_scale = bn->scale; p.bn_shift = bn->shift; p.bn_mu = bn->mu; p.bn_invstd = bn->invstd;
    p.bn_sdz = bn->sdz; p.bn_sdzx = bn->sdzx; p.inv_m = bn->inv_m;
  }
  p.N = N; p.H = H; p.W = W; p.Cout = Cout; p.kchunks = epi == 2 ? 1 : Cin / 64; p.n_tiles = epi == 2 ? Cout / 64 : 1;
  p.tiles_w = (W + TW - 1) / TW; p.tiles_h = (H + TH - 1) / TH; p.total_tiles = N * p.tiles_w * p.tiles_h * p.n_tiles;
  if ((long long)N * p.tiles_w * p.tiles_h * p.n_tiles > (1ll << 30)) return NF_EUNSUPPORTED;
  p.stats = stats; p.red = red; p.status = status; p.bias = bias; p.out = (bf16*)y;
  const size_t a_bytes = wide ? ((size_t)34 * 10 * KC * 2 + 1023) / 1024 * 1024
                         : uf2 ? ((size_t)18 * 10 * KC * 2 + 1023) / 1024 * 1024 : (size_t)(uf ? 3 : 1) * 10 * 16 * KC * 2;
  const size_t wbytes = epi == 2 ? (size_t)9 * KC * 128 : (size_t)9 * p.kchunks * G * 128;
  const size_t fixed = wide ? wbytes + (size_t)(stats >= 2 ? 2 + kWideYSlots : 2) * 32768 + 1024 + 1024
                            : wbytes + (epi != 1 ? (stats >= 2 ? 2 + kYSlots : 2) * 16384 : xf ? 3 * kXfGroups * 112 * 128 : 0) + 1024 + 1024;
  int st = (int)((232448 - fixed) / a_bytes);
  if (st > kMaxStages) st = kMaxStages;
  p.stages = st;
  const size_t smem = (size_t)st * a_bytes + fixed;
  int grid = sm_count();
  grid -= grid % p.n_tiles;  // a CTA keeps one output-channel tile (and its resident weights) for its whole life
  if (grid < p.n_tiles) grid = p.n_tiles;
  if (grid > p.total_tiles) grid = p.total_tiles;
  if (stats && stats != 4) {
    const size_t need = (size_t)(grid / p.n_tiles) * 2 * 2 * Cout;  // every CTA writes its two partials (one per epilogue group)
    if (need > red_floats) return NF_ENOWS;
    *nb = grid / p.n_tiles * 2;
  }
  if (xf) {
    if (epi != 1) return NF_EINVAL;
    p.xf_scale = xf->scale; p.xf_shift = xf->shift; p.xf_a = (bf16*)xf->a;
    p.pool_part = xf->pool_part; p.mask = xf->mask;
    return G == 16 ? launch_fold<16, 1, 64, 0, 0, 1>(grid, smem, mx, mw, my, my2, p)
                   : G == 32 ? launch_fold<32, 1, 64, 0, 0, 1>(grid, smem, mx, mw, my, my2, p)
                             : launch_fold<64, 1, 64, 0, 0, 1>(grid, smem, mx, mw, my, my2, p);
  }
  if (epi == 0) return launch_fold<64, 0>(grid, smem, mx, mw, my, my2, p);
  if (wide) {
    static bool attr_done_dev[kMaxDevices];
    bool& attr_done = attr_done_dev[current_device()];
    if (!attr_done) {
      NF_CUDA(cudaFuncSetAttribute(aux_dgrad_wide_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448));
      attr_done = true;
    }
    aux_dgrad_wide_kernel<16><<<grid, kWideThreads, smem, g_nf_stream>>>(mx, mw, my, my2, p);
    NF_LAUNCHED();
    return NF_OK;
  }
  if (epi == 2 && uf2)
    return KC == 16 ? launch_fold<64, 0, 16, 1, 2>(grid, smem, mx, mw, my, my2, p) : launch_fold<64, 0, 32, 1, 2>(grid, smem, mx, mw, my, my2, p);
  if (epi == 2 && uf)
    return KC == 16 ? launch_fold<64, 0, 16, 1, 1>(grid, smem, mx, mw, my, my2, p) : launch_fold<64, 0, 32, 1, 1>(grid, smem, mx, mw, my, my2, p);
  if (epi == 2)
    return KC == 16 ? launch_fold<64, 0, 16, 1>(grid, smem, mx, mw, my, my2, p) : launch_fold<64, 0, 32, 1>(grid, smem, mx, mw, my, my2, p);
  return G == 16 ? launch_fold<16, 1>(grid, smem, mx, mw, my, my2, p)
                 : G == 32 ? launch_fold<32, 1>(grid, smem, mx, mw, my, my2, p) : launch_fold<64, 1>(grid, smem, mx, mw, my, my2, p);
}

// epi 0: y through TMA + optional statistics.  epi 1: out = ReLU(conv + bias) written directly (y unused).
// H, W are the INPUT size; stride 2 halves them (rounding up) for the output.
int run_fwd(int N, int Hin, int Win, int Cin, int Cout, const void* x, const void* w, void* y, int stats, float* red,
            size_t red_floats, int32_t* status, int* nb, int epi = 0, const float* bias = nullptr, int stride = 1,
            const BnBwdIn* bn = nullptr) {
  const int H = (Hin - 1) / stride + 1, W = (Win - 1) / stride + 1;
  if (fold_ok(H, W, Cin, Cout, epi, stride, stats))
    return run_fold(N, H, W, Cin, Cout, x, w, y, stats, red, red_floats, status, nb, epi, bias, bn);
  if (stats > 2) return NF_EUNSUPPORTED;  // the two-pass input gradient exists in the folded kernel only
  if (stats == 2 && (!bn || epi == 1)) return NF_EINVAL;
  const TcPlan pl = plan_fwd(H, W, Cin, Cout, N, epi, stride, stats == 2);
  if (!pl.ok) return NF_EUNSUPPORTED;
  CUtensorMap mx, mw, my;
  const uint64_t dx[4] = {(uint64_t)Cin, (uint64_t)Win, (uint64_t)Hin, (uint64_t)N};
  const uint32_t bx[4] = {(uint32_t)pl.KC, (uint32_t)pl.BW, (uint32_t)(pl.PT ? pl.BH : pl.BH + 2), (uint32_t)pl.BI};
  // forward: weights [kh][kw][Cout][Cin] -> box of BN rows x 64 ci for three kh; input gradient: weights
  // [kh][kw][F][Cout] -> box of KC rows of f x 64 c for three kh
  const uint64_t dw[4] = {(uint64_t)(epi == 2 ? Cout : Cin), (uint64_t)(epi == 2 ? Cin : Cout), 3, 3};
  const uint32_t bw[4] = {64, (uint32_t)(epi == 2 ? pl.KC : pl.BN), 1, (uint32_t)(pl.PT ? 1 : 3)};
  const uint64_t dy[4] = {(uint64_t)Cout, (uint64_t)W, (uint64_t)H, (uint64_t)N};
  const uint32_t by[4] = {64, (uint32_t)pl.BW, (uint32_t)pl.BH, (uint32_t)pl.BI};
  int rc;
  if ((rc = make_map4(&mx, x, dx, bx, stride)) != NF_OK) return rc;
  if ((rc = make_map4(&mw, w, dw, bw)) != NF_OK) return rc;
  if (epi != 1) {
    if ((rc = make_map4(&my, y, dy, by)) != NF_OK) return rc;
  } else {
    my = mx;  // not used by this epilogue
  }
  FwdParams p{};
  p.N = N; p.H = H; p.W = W; p.Cin = Cin; p.Cout = Cout;
  p.BW = pl.BW; p.BH = pl.BH; p.tiles_w = W / pl.BW; p.tiles_h = H / pl.BH; p.n_tiles = epi != 1 ? Cout / pl.BN : 1;
  p.bias = bias; p.out = (bf16*)y;
  p.total_tiles = ((N + pl.BI - 1) / pl.BI) * p.tiles_h * p.tiles_w * p.n_tiles;
  p.stride = stride; p.BI = pl.BI;
  p.kchunks = epi == 2 ? 1 : Cin / 64; p.stages = pl.stages; p.stats = stats; p.red = red; p.status = status;
  p.tm_y2 = my;
  if (stats == 2) {
    if ((rc = make_map4(&p.tm_y2, bn->y2, dy, by)) != NF_OK) return rc;
    p.bn_scale = bn->scale; p.bn_shift = bn->shift; p.bn_mu = bn->mu; p.bn_invstd = bn->invstd;
  }
  if (stats) {
    const size_t need = (size_t)pl.grid * pl.parts * 2 * Cout;
    if (need > red_floats) return NF_ENOWS;
    NF_CUDA(cudaMemsetAsync(red, 0, need * sizeof(float), g_nf_stream));
    *nb = pl.grid * pl.parts;
  }
  if (pl.PT) {  // per-tap boxes: stride 2, or several small images per tile
    if (epi == 0)
      return pl.BN == 256 ? launch_fwd<256, 0, 64, 0, 1>(pl, mx, mw, my, p)
                          : pl.BN == 128 ? launch_fwd<128, 0, 64, 0, 1>(pl, mx, mw, my, p) : launch_fwd<64, 0, 64, 0, 1>(pl, mx, mw, my, p);
    if (epi == 1)
      return pl.BN == 16 ? launch_fwd<16, 1, 64, 0, 1>(pl, mx, mw, my, p)
                         : pl.BN == 32 ? launch_fwd<32, 1, 64, 0, 1>(pl, mx, mw, my, p) : launch_fwd<64, 1, 64, 0, 1>(pl, mx, mw, my, p);
    if (pl.BN == 128)
      return pl.KC == 16 ? launch_fwd<128, 0, 16, 1, 1>(pl, mx, mw, my, p)
                         : pl.KC == 32 ? launch_fwd<128, 0, 32, 1, 1>(pl, mx, mw, my, p) : launch_fwd<128, 0, 64, 1, 1>(pl, mx, mw, my, p);
    return pl.KC == 16 ? launch_fwd<64, 0, 16, 1, 1>(pl, mx, mw, my, p)
                       : pl.KC == 32 ? launch_fwd<64, 0, 32, 1, 1>(pl, mx, mw, my, p) : launch_fwd<64, 0, 64, 1, 1>(pl, mx, mw, my, p);
  }
  if (epi == 0 && pl.RW) return launch_fwd<64, 0, 64, 0, 0, 1>(pl, mx, mw, my, p);
  if (epi == 0) return pl.BN == 128 ? launch_fwd<128, 0>(pl, mx, mw, my, p) : launch_fwd<64, 0>(pl, mx, mw, my, p);
  if (epi == 1 && pl.RW)
    return pl.BN == 16 ? launch_fwd<16, 1, 64, 0, 0, 1>(pl, mx, mw, my, p)
                       : pl.BN == 32 ? launch_fwd<32, 1, 64, 0, 0, 1>(pl, mx, mw, my, p) : launch_fwd<64, 1, 64, 0, 0, 1>(pl, mx, mw, my, p);
  if (epi == 2) {
    if (pl.BN == 128)
      return pl.KC == 16 ? launch_fwd<128, 0, 16, 1>(pl, mx, mw, my, p)
                         : pl.KC == 32 ? launch_fwd<128, 0, 32, 1>(pl, mx, mw, my, p) : launch_fwd<128, 0, 64, 1>(pl, mx, mw, my, p);
    return pl.KC == 16 ? launch_fwd<64, 0, 16, 1>(pl, mx, mw, my, p)
                       : pl.KC == 32 ? launch_fwd<64, 0, 32, 1>(pl, mx, mw, my, p) : launch_fwd<64, 0, 64, 1>(pl, mx, mw, my, p);
  }
  return pl.BN == 16 ? launch_fwd<16, 1>(pl, mx, mw, my, p)
                     : pl.BN == 32 ? launch_fwd<32, 1>(pl, mx, mw, my, p) : launch_fwd<64, 1>(pl, mx, mw, my, p);
}

struct WgPlan {
  int ok, BW, BH, BI, PT, NB, GX, splits, grid, stages;
  size_t smem, part_floats;
};

// aux = 0: main conv (Cout a multiple of 64).  aux = 1: aux conv (Cout = F <= 64, a multiple of 8).
// H, W: size of the gradient tensor (the conv OUTPUT; equals the input size for stride 1).
WgPlan plan_wgrad(int H, int W, int Cin, int Cout, int N, int aux = 0, int stride = 1) {
  WgPlan pl{};
  if (Cin % 64 || (stride == 2 && aux)) return pl;
  if (aux ? (Cout > 64 || Cout % 8) : (Cout % 64 != 0)) return pl;
  if (!pick_tile(H, W, true, &pl.BW, &pl.BH, &pl.BI)) return pl;
  pl.PT = (stride == 2 || pl.BI > 1) ? 1 : 0;
  pl.NB = aux ? (Cout <= 16 ? 16 : Cout <= 32 ? 32 : 64) : 64;
  if (!aux && pl.PT) pl.NB = Cout % 256 == 0 ? 256 : Cout % 128 == 0 ? 128 : 64;  // per-tap form: as wide an instruction as Cout allows
  pl.GX = (aux && !pl.PT && pl.NB <= 32) ? 1 : 0;  // few filters: one instruction per 16 pixels with the gradient on the M side
  size_t g_region = (size_t)(pl.GX ? 4 : 3) * 128 * pl.NB * 2;
  if (g_region < 4096) g_region = 4096;
  const size_t stage = pl.PT ? (size_t)49152 + (pl.NB > 64 ? pl.NB / 64 : 1) * 16384 : (size_t)(pl.BH + 2) * pl.BW * 128 + g_region;
  pl.stages = pl.PT ? (pl.NB > 64 ? 2 : 3) : (int)((232448 - 2048) / stage);
  if (pl.stages > kMaxStages) pl.stages = kMaxStages;
  if (pl.stages < 2) return pl;
  pl.smem = (size_t)pl.stages * stage + 1024 + 1024;
  if (pl.smem > 232448) return pl;
  const int blocks = (Cin / 64) * (aux ? 1 : Cout / pl.NB);
  const long pix_tiles = (long)((N + pl.BI - 1) / pl.BI) * (H / pl.BH) * (W / pl.BW);
  const int groups = pl.PT ? 3 : 1;  // kernel rows handled by separate CTAs
  // pixel splits per (chunk pair, kernel-row group): the count whose CTAs fill whole waves of SMs best (smallest on ties),
  // e.g. 512 -> 512 channels with three row groups: 192 units -> 3 splits = 576 CTAs = 3.9 waves instead of 1.3
  const int units = blocks * groups, sms = sm_count();
  long base = sms / units;
  if (base < 1) base = 1;
  long sp = base;
  double best = 0.0;
  for (long c = 1; c <= (base * 2 > 16 ? base * 2 : 16) && c <= pix_tiles; ++c) {
    const long total = c * units, waves = (total + sms - 1) / sms;
    const double eff = (double)total / (double)(waves * sms);
    if (eff > best + 1e-9) {
      best = eff;
      sp = c;
    }
  }
  if (sp > pix_tiles) sp = pix_tiles;
  pl.splits = (int)sp;
  pl.grid = (int)(sp * blocks * groups);
  pl.part_floats = (size_t)sp * 9 * Cout * Cin;
  pl.ok = 1;
  return pl;
}

template <int NB>
int launch_wgrad_kw(const WgPlan& pl, const CUtensorMap& mx, const CUtensorMap& mg, const WgParams& p) {
  static bool attr_done_dev[kMaxDevices];  // function attributes belong to a device's context: set once per device
  bool& attr_done = attr_done_dev[current_device()];
  if (!attr_done) {
    NF_CUDA(cudaFuncSetAttribute(conv_wgrad_kw_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448));
    attr_done = true;
  }
  conv_wgrad_kw_kernel<NB><<<pl.grid, kThreads, pl.smem, g_nf_stream>>>(mx, mg, p);
  NF_LAUNCHED();
  return NF_OK;
}

template <int NB>
int launch_wgrad_gx(const WgPlan& pl, const CUtensorMap& mx, const CUtensorMap& mg, const WgParams& p) {
  static bool attr_done_dev[kMaxDevices];  // function attributes belong to a device's context: set once per device
  bool& attr_done = attr_done_dev[current_device()];
  if (!attr_done) {
    NF_CUDA(cudaFuncSetAttribute(conv_wgrad_gx_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448));
    attr_done = true;
  }
  conv_wgrad_gx_kernel<NB><<<pl.grid, kThreads, pl.smem, g_nf_stream>>>(mx, mg, p);
  NF_LAUNCHED();
  return NF_OK;
}

template <int NB, int S2 = 0>
int launch_wgrad(const WgPlan& pl, const CUtensorMap& mx, const CUtensorMap& mg, const WgParams& p) {
  static bool attr_done_dev[kMaxDevices];  // function attributes belong to a device's context: set once per device
  bool& attr_done = attr_done_dev[current_device()];
  if (!attr_done) {
    NF_CUDA(cudaFuncSetAttribute(conv_wgrad_tc_kernel<NB, S2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448));
    attr_done = true;
  }
  conv_wgrad_tc_kernel<NB, S2><<<pl.grid, kThreads, pl.smem, g_nf_stream>>>(mx, mg, p);
  NF_LAUNCHED();
  return NF_OK;
}

// Hin, Win: INPUT size; the gradient tensor has the strided output size.
int run_wgrad(int N, int Hin, int Win, int Cin, int Cout, const void* x, const void* dy, float* part, size_t part_floats,
              float* dw, int32_t* status, int aux = 0, int stride = 1) {
  const int H = (Hin - 1) / stride + 1, W = (Win - 1) / stride + 1;
  const WgPlan pl = plan_wgrad(H, W, Cin, Cout, N, aux, stride);
  if (!pl.ok) return NF_EUNSUPPORTED;
  if (pl.part_floats > part_floats) return NF_ENOWS;
  CUtensorMap mx, mg;
  const uint64_t dx[4] = {(uint64_t)Cin, (uint64_t)Win, (uint64_t)Hin, (uint64_t)N};
  const uint32_t bx[4] = {64, (uint32_t)pl.BW, (uint32_t)(pl.PT ? pl.BH : pl.BH + 2), (uint32_t)pl.BI};
  const uint64_t dg[4] = {(uint64_t)Cout, (uint64_t)W, (uint64_t)H, (uint64_t)N};
  const uint32_t bg[4] = {(uint32_t)(pl.NB > 64 ? 64 : pl.NB), (uint32_t)pl.BW, (uint32_t)pl.BH, (uint32_t)pl.BI};
  int rc;
  if ((rc = make_map4(&mx, x, dx, bx, stride)) != NF_OK) return rc;
  if ((rc = make_map4(&mg, dy, dg, bg)) != NF_OK) return rc;
  WgParams p{};
  p.N = N; p.H = H; p.W = W; p.Cin = Cin; p.Cout = Cout; p.BW = pl.BW; p.BH = pl.BH;
  p.tiles_w = W / pl.BW; p.tiles_h = H / pl.BH; p.pix_tiles = ((N + pl.BI - 1) / pl.BI) * p.tiles_h * p.tiles_w;
  p.stride = stride; p.BI = pl.BI;
  p.ci_chunks = Cin / 64; p.co_chunks = aux ? 1 : Cout / pl.NB; p.splits = pl.splits; p.part = part; p.status = status;
  p.stages = pl.stages;
  if (pl.GX)
    rc = pl.NB == 32 ? launch_wgrad_gx<32>(pl, mx, mg, p) : launch_wgrad_gx<16>(pl, mx, mg, p);
  else if (pl.PT)
    rc = pl.NB == 256 ? launch_wgrad<256, 1>(pl, mx, mg, p) : pl.NB == 128 ? launch_wgrad<128, 1>(pl, mx, mg, p)
       : pl.NB == 64 ? launch_wgrad<64, 1>(pl, mx, mg, p) : pl.NB == 32 ? launch_wgrad<32, 1>(pl, mx, mg, p) : launch_wgrad<16, 1>(pl, mx, mg, p);
  else
    rc = pl.NB == 64 ? launch_wgrad_kw<64>(pl, mx, mg, p)
                     : pl.NB == 32 ? launch_wgrad_kw<32>(pl, mx, mg, p) : launch_wgrad_kw<16>(pl, mx, mg, p);
  if (rc != NF_OK) return rc;
  const size_t n = (size_t)9 * Cout * Cin;
  sum_parts_kernel<<<(unsigned)((n + 31) / 32), dim3(32, 8), 0, g_nf_stream>>>(part, pl.splits, n, dw);
  NF_LAUNCHED();
  return NF_OK;
}

}  // namespace

// The classic local-learning setting (256 auxiliary filters) and the paper's own rule for late layers give F > 64.
// Then the aux conv is as wide as a main conv and uses the same three kernels: forward (bias and ReLU in its epilogue),
// weight gradient, and the input gradient written as a forward conv over a mirrored, transposed weight copy.
static bool wide_aux(const nf_layer* L) { return L->F > 64 && L->F % 64 == 0; }

void nf_tc_select(nf_layer* L) {
  L->fam[0] = L->fam[1] = L->fam[2] = L->fam[3] = 0;
  L->cin_pad = 0;
  if (L->o.dtype != NF_BF16) return;
  // A first layer with a handful of input channels (RGB) is far too thin a contraction for useful tensor-core work (K = 27),
  // but its CUDA-core kernels reach under a tenth of the memory bandwidth, and the tensor cores are idle anyway: the input
  // batch is copied once per step into a 64-channel zero-padded tensor (as large as the layer's output) and the main conv
  // then runs on the ordinary 64-channel kernels.  21 times the arithmetic, a third of the time (VGG first layer at 64 x 64,
  // 1260 images: forward + weight gradient 2.6 ms -> 0.9 ms including the copy).
  if (L->Cin <= 8 && plan_fwd(L->Ho, L->Wo, 64, L->Cout, L->o.N, 0, L->o.stride).ok &&
      plan_wgrad(L->Ho, L->Wo, 64, L->Cout, L->o.N, 0, L->o.stride).ok)
    L->cin_pad = 64;
  const int Cin = L->cin_pad ? L->cin_pad : L->Cin;
  if (plan_fwd(L->Ho, L->Wo, Cin, L->Cout, L->o.N, 0, L->o.stride).ok) L->fam[0] = 1;
  if (plan_wgrad(L->Ho, L->Wo, Cin, L->Cout, L->o.N, 0, L->o.stride).ok) L->fam[1] = 1;
  if (wide_aux(L)) {  // more than 64 filters: the aux conv runs on the kernels of the main conv
    if (plan_fwd(L->Ha, L->Wa, L->Cout, L->F, L->o.N, 0).ok) L->fam[2] = 1;
    if (plan_wgrad(L->Ha, L->Wa, L->Cout, L->F, L->o.N, 0).ok && plan_fwd(L->Ha, L->Wa, L->F, L->Cout, L->o.N, 0).ok) L->fam[3] = 1;
    return;
  }
  if (plan_fwd(L->Ha, L->Wa, L->Cout, L->F, L->o.N, 1).ok) L->fam[2] = 1;
  if (plan_wgrad(L->Ha, L->Wa, L->Cout, L->F, L->o.N, 1).ok && plan_fwd(L->Ha, L->Wa, L->F, L->Cout, L->o.N, 2).ok) L->fam[3] = 1;
}

size_t nf_tc_scratch_floats(const nf_layer* L) {
  const size_t a = L->fam[1] ? plan_wgrad(L->Ho, L->Wo, L->cin_pad ? L->cin_pad : L->Cin, L->Cout, L->o.N, 0, L->o.stride).part_floats : 0;
  const size_t b = L->fam[3] ? plan_wgrad(L->Ha, L->Wa, L->Cout, L->F, L->o.N, wide_aux(L) ? 0 : 1).part_floats : 0;
  return a > b ? a : b;
}

size_t nf_tc_red_floats(const nf_layer* L) {
  size_t need = 0;
  if (L->fam[3]) need = (size_t)sm_count() * 8 * 2 * L->Cout;  // input-gradient kernel with the fused BatchNorm-backward sums
  if (!L->fam[0]) return need;
  const TcPlan pl = plan_fwd(L->Ho, L->Wo, L->cin_pad ? L->cin_pad : L->Cin, L->Cout, L->o.N, 0, L->o.stride);
  const size_t fwd = (size_t)sm_count() * (pl.parts < 8 ? 8 : pl.parts) * 2 * L->Cout;  // the folded kernel writes 8 partials per CTA
  return fwd > need ? fwd : need;
}

// input and operand weights of the main conv: the caller's, or their 64-channel zero-padded copies (refreshed here)
static int main_conv_operands(nf_layer* L, const void* x, int count, const void** xin, const void** win, int* Cin) {
  *xin = x;
  *win = L->shadow + L->off[NF_P_W];
  *Cin = L->Cin;
  if (!L->cin_pad) return NF_OK;
  int rc = nf_k_pad_channels(x, (size_t)count * L->H * L->W, L->Cin, L->cin_pad, L->xpad);
  if (rc != NF_OK) return rc;
  if ((rc = nf_k_pad_weights(L->shadow + L->off[NF_P_W], (size_t)9 * L->Cout, L->Cin, L->cin_pad, L->wpad)) != NF_OK) return rc;
  *xin = L->xpad;
  *win = L->wpad;
  *Cin = L->cin_pad;
  return NF_OK;
}

int nf_tc_conv_fwd(nf_layer* L, const void* x, int& nb) {
  if (L->cin_pad) {
    const void *xin, *win;
    int Cin;
    const int rc = main_conv_operands(L, x, L->o.N, &xin, &win, &Cin);
    if (rc != NF_OK) return rc;
    return run_fwd(L->o.N, L->H, L->W, Cin, L->Cout, xin, win, L->y, 1, L->red, L->red_floats, L->status, &nb, 0, nullptr, L->o.stride);
  }
  return run_fwd(L->o.N, L->H, L->W, L->Cin, L->Cout, x, L->shadow + L->off[NF_P_W], L->y, 1, L->red, L->red_floats,
                 L->status, &nb, 0, nullptr, L->o.stride);
}

int nf_tc_conv_fwd_eval(nf_layer* L, const void* x, int count) {
  int nb = 0;
  if (L->cin_pad) {
    const void *xin, *win;
    int Cin;
    const int rc = main_conv_operands(L, x, count, &xin, &win, &Cin);
    if (rc != NF_OK) return rc;
    return run_fwd(count, L->H, L->W, Cin, L->Cout, xin, win, L->y, 0, nullptr, 0, L->status, &nb, 0, nullptr, L->o.stride);
  }
  return run_fwd(count, L->H, L->W, L->Cin, L->Cout, x, L->shadow + L->off[NF_P_W], L->y, 0, nullptr, 0, L->status, &nb, 0,
                 nullptr, L->o.stride);
}

int nf_tc_aux_fwd(nf_layer* L, const void* a, int count) {
  int nb = 0;
  if (wide_aux(L)) {
    return run_fwd(count, L->Ha, L->Wa, L->Cout, L->F, a, L->shadow + L->off[NF_P_WA], L->h, 0, nullptr, 0, L->status, &nb, 0,
                   L->val + L->off[NF_P_BA]);
  }
  return run_fwd(count, L->Ha, L->Wa, L->Cout, L->F, a, L->shadow + L->off[NF_P_WA], L->h, 0, nullptr, 0, L->status, &nb, 1,
                 L->val + L->off[NF_P_BA]);
}

bool nf_tc_bn_aux_fused(const nf_layer* L) {
  // beside the weights and three activation stages the kernel then also holds three staging tiles of a.  On widths that are
  // no multiple of 14 (ragged last tile column) only for up to 32 filters: with 64 the wide shift-add epilogue ate the gain
  // (32 x 32 maps, 64 filters: aux forward + normalisation 0.174 ms separate, 0.197 ms fused).
  if (L->Wa % 14 != 0 && L->F > 32) return false;
  return L->fam[2] && !wide_aux(L) && !L->o.maxpool && fold_ok(L->Ha, L->Wa, L->Cout, L->F, 1, 1, 0, 3 * kXfGroups * 112 * 128);
}

// The fused aux forward can also keep h out of memory when the head pools by averaging and no tile straddles a pooling
// quadrant (14 x 8-pixel tiles: Ha/2 a multiple of 8, Wa/2 of 14): the epilogue then emits pooling partials and a sign mask.
bool nf_tc_aux_pool_fused(const nf_layer* L) {
  return nf_tc_bn_aux_fused(L) && L->o.aux_pool == NF_POOL_AVG && (L->Ha / 2) % 8 == 0 && (L->Wa / 2) % 14 == 0 && L->Ha % 2 == 0 &&
         L->Wa % 2 == 0 && (size_t)L->o.N * L->Ha * L->Wa < ((size_t)1 << 31);
}

size_t nf_tc_pool_part_floats(const nf_layer* L) {
  return (size_t)L->o.N * (L->Wa / 14) * (L->Ha / 8) * 4 * L->F;
}

int nf_tc_bn_aux_fwd(nf_layer* L, void* act_out) {
  if (!nf_tc_bn_aux_fused(L) || L->skip) return NF_EUNSUPPORTED;
  int nb = 0;
  const bool pooled = nf_tc_aux_pool_fused(L);
  // the partials live in the split-K scratch (free until the weight gradients), the mask in the unused h buffer
  const XfIn xf{L->scale, L->shift, act_out, pooled ? L->wpart : nullptr, pooled ? (uint8_t*)L->h : nullptr};
  return run_fold(L->o.N, L->Ha, L->Wa, L->Cout, L->F, L->y, L->shadow + L->off[NF_P_WA], L->h, 0, nullptr, 0, L->status, &nb, 1,
                  L->val + L->off[NF_P_BA], nullptr, &xf);
}

int nf_tc_wgrad(nf_layer* L, const void* x) {
  if (L->cin_pad) {  // the padded copy of this step's input is still in place (the forward made it); x itself is not read again
    const int rc = run_wgrad(L->o.N, L->H, L->W, L->cin_pad, L->Cout, L->xpad, L->dy, L->wpart, L->wpart_floats, L->gwpad, L->status, 0,
                             L->o.stride);
    if (rc != NF_OK) return rc;
    return nf_k_unpad_grad(L->gwpad, (size_t)9 * L->Cout, L->Cin, L->cin_pad, L->grad + L->off[NF_P_W]);
  }
  return run_wgrad(L->o.N, L->H, L->W, L->Cin, L->Cout, x, L->dy, L->wpart, L->wpart_floats, L->grad + L->off[NF_P_W],
                   L->status, 0, L->o.stride);
}

// Two-pass form of the input gradient (folded kernel, no pool, no shortcut, fewer than 64 aux filters): the first pass only
// reduces the BatchNorm-backward sums, the second (nf_tc_aux_dgrad_dy, after the sums have been finished) forms da again and
// writes dy = BatchNorm-backward(da) directly, so da is never stored and the separate apply pass (read y and da, write dy)
// disappears: 1.75 activation-sized tensors less memory traffic per layer step for one more read of the narrow dh.
bool nf_tc_dgrad_two_pass(const nf_layer* L) {
  return L->fam[3] && !wide_aux(L) && !L->o.maxpool && fold_ok(L->Ha, L->Wa, L->F, L->Cout, 2, 1, 3) &&
         (size_t)(sm_count() / (L->Cout / 64)) * 8 * 2 * L->Cout <= L->red_floats;
}

int nf_tc_aux_dgrad_dy(nf_layer* L, double M) {
  if (!nf_tc_dgrad_two_pass(L) || L->skip || L->skip_grad) return NF_EUNSUPPORTED;
  int nb = 0;
  BnBwdIn bn{L->y, L->scale, L->shift, L->mu, L->invstd};
  bn.sdz = L->sdz; bn.sdzx = L->sdzx; bn.inv_m = (float)(1.0 / M);
  return run_fwd(L->o.N, L->Ha, L->Wa, L->F, L->Cout, L->dh, L->shadow + L->off[NF_P_WA], L->dy, 4, nullptr, 0, L->status, &nb, 2,
                 nullptr, 1, &bn);
}

int nf_tc_aux_dgrad(nf_layer* L, int* bn_nb) {
  int nb = 0;
  *bn_nb = 0;
  if (nf_tc_dgrad_two_pass(L) && !L->skip && !L->skip_grad) {  // first pass: sums only, nothing stored
    const BnBwdIn bn{L->y, L->scale, L->shift, L->mu, L->invstd};
    return run_fwd(L->o.N, L->Ha, L->Wa, L->F, L->Cout, L->dh, L->shadow + L->off[NF_P_WA], L->da, 3, L->red, L->red_floats, L->status,
                   bn_nb, 2, nullptr, 1, &bn);
  }
  const bool wide = wide_aux(L);
  const void* w = L->shadow + L->off[NF_P_WA];
  if (wide) {
    const int rc = nf_k_flip_weights(L->shadow + L->off[NF_P_WA], L->F, L->Cout, L->wa_t);
    if (rc != NF_OK) return rc;
    w = L->wa_t;
  }
  const int epi = wide ? 0 : 2;
  // Without a pool (and without a shortcut) da has the shape of y, and the kernel that produces it also reduces
  // (dz, dz*xhat) per channel while it holds the tile: the BatchNorm backward then needs no reduction pass.
  if (!L->o.maxpool && !L->skip) {
    const BnBwdIn bn{L->y, L->scale, L->shift, L->mu, L->invstd};
    bool fits;
    if (fold_ok(L->Ha, L->Wa, L->F, L->Cout, epi, 1, 2)) {
      fits = (size_t)(sm_count() / (L->Cout / 64)) * 8 * 2 * L->Cout <= L->red_floats;
    } else {
      const TcPlan pl = plan_fwd(L->Ha, L->Wa, L->F, L->Cout, L->o.N, epi, 1, 1);
      fits = pl.ok && (size_t)pl.grid * pl.parts * 2 * L->Cout <= L->red_floats;
    }
    if (fits)
      return run_fwd(L->o.N, L->Ha, L->Wa, L->F, L->Cout, L->dh, w, L->da, 2, L->red, L->red_floats, L->status, bn_nb, epi, nullptr,
                     1, &bn);
  }
  return run_fwd(L->o.N, L->Ha, L->Wa, L->F, L->Cout, L->dh, w, L->da, 0, nullptr, 0, L->status, &nb, epi);
}

int nf_tc_aux_wgrad(nf_layer* L, const void* a) {
  return run_wgrad(L->o.N, L->Ha, L->Wa, L->Cout, L->F, a, L->dh, L->wpart, L->wpart_floats, L->grad + L->off[NF_P_WA],
                   L->status, wide_aux(L) ? 0 : 1);
}

size_t nf_tc_conv3x3_wgrad_scratch_floats(int N, int H, int W, int Cin, int Cout, int stride) {
  const WgPlan pl = plan_wgrad((H - 1) / stride + 1, (W - 1) / stride + 1, Cin, Cout, N, 0, stride);
  return pl.ok ? pl.part_floats : 0;
}

static __device__ int32_t g_op_status;  // status word of the stand-alone operations (one per device that loads the library)

int nf_tc_op_status_ptr(int32_t** out) {
  static int32_t* st_dev[kMaxDevices];
  int32_t*& st = st_dev[current_device()];
  if (!st) NF_CUDA(cudaGetSymbolAddress((void**)&st, g_op_status));
  *out = st;
  return NF_OK;
}

int nf_tc_conv3x3_forward(const void* x, const void* w, int N, int H, int W, int Cin, int Cout, int stride, void* y) {
  int32_t* st = nullptr;
  if (nf_tc_op_status_ptr(&st) != NF_OK) return NF_ECUDA;
  int nb = 0;
  return run_fwd(N, H, W, Cin, Cout, x, w, y, 0, nullptr, 0, st, &nb, 0, nullptr, stride);
}

int nf_tc_conv3x3_wgrad(const void* x, const void* g, int N, int H, int W, int Cin, int Cout, int stride, float* part,
                        size_t part_floats, float* dw) {
  int32_t* st = nullptr;
  if (nf_tc_op_status_ptr(&st) != NF_OK) return NF_ECUDA;
  return run_wgrad(N, H, W, Cin, Cout, x, g, part, part_floats, dw, st, 0, stride);
}

// One CTA of one warp waits, with the bounded wait every tensor-core kernel uses, on a barrier that nobody ever
// arrives at, and then leaves the way those kernels do: abort flag set by the waiter, NF_ETIMEOUT raised in the status
// word, waited time reported.  No TMA, no tensor memory, nothing else in flight.
__global__ void bounded_wait_probe_kernel(unsigned long long limit_ns, int32_t* status, unsigned long long* waited_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();
  const unsigned long long t0 = ptx::globaltimer();
  const bool done = __all_sync(0xffffffffu, ptx::mbar_wait(&bar, 0, &abort_flag, limit_ns));
  const unsigned long long t1 = ptx::globaltimer();
  __syncthreads();
  if (threadIdx.x == 0) {
    if (!done && abort_flag) atomicOr(status, NF_ETIMEOUT);
    *waited_ns = t1 - t0;
  }
}

int nf_tc_bounded_wait_probe(unsigned long long limit_ns, unsigned long long* waited_ns_dev) {
  int32_t* st = nullptr;
  if (nf_tc_op_status_ptr(&st) != NF_OK) return NF_ECUDA;
  bounded_wait_probe_kernel<<<1, 32, 0, g_nf_stream>>>(limit_ns, st, waited_ns_dev);
  NF_LAUNCHED();
  return NF_OK;
}

int nf_tc_op_status(int32_t* out) {
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  NF_CUDA(cudaMemcpyFromSymbol(out, g_op_status, sizeof(int32_t)));
  const int32_t zero = 0;
  NF_CUDA(cudaMemcpyToSymbol(g_op_status, &zero, sizeof(int32_t)));
  return NF_OK;
}
