// Allocation-free weight gradient: the split partial sums live in a fixed device array that is
// part of the library image, for callers that cannot provide (or allocate) scratch memory.
#include "nf_internal.h"
#include "nf_tc.h"

// 16 MiB on every GPU that loads the library, until the process exits.
static __device__ __align__(256) float g_static_scratch[NF_STATIC_SCRATCH_BYTES / sizeof(float)];

namespace {
constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices];  // device address of g_static_scratch, per device; looked up on first use

// In host code the name g_static_scratch is only a handle for the symbol, not a device address, so
// the address a kernel may use has to be asked for, once per device and with that device current.
int static_scratch(float** out) {
  int dev = 0;
  NF_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return NF_EUNSUPPORTED;
  if (!g_scratch_ptr[dev]) {
    float* p = nullptr;
    NF_CUDA(cudaGetSymbolAddress((void**)&p, g_static_scratch));
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return NF_OK;
}
}  // namespace

extern "C" int nf_conv3x3_wgrad_static(int dtype, const void* x, const void* g, int N, int H, int W, int Cin,
                                       int Cout, int stride, float* dw) {
  if (!x || !g || !dw || (dtype != NF_F32 && dtype != NF_BF16) || N < 1 || H < 1 || W < 1 || Cin < 1 || Cout < 1 ||
      (stride != 1 && stride != 2))
    return NF_EINVAL;
  if (((uintptr_t)x | (uintptr_t)g | (uintptr_t)dw) & 15) return NF_EALIGN;
  const size_t need = nf_conv3x3_wgrad_scratch_bytes(N, H, W, Cin, Cout, stride);
  if (need == 0 || need > NF_STATIC_SCRATCH_BYTES) return NF_ENOWS;  // larger than the built-in array: refused
  float* scratch = nullptr;
  const int rc = static_scratch(&scratch);
  if (rc != NF_OK) return rc;
  // Same dispatch as nf_conv3x3_wgrad: the tcgen05 kernels where they cover the shape, else the CUDA-core kernel.
  // Both write every partial they later read, so stale contents of the shared array are harmless.
  const size_t floats = NF_STATIC_SCRATCH_BYTES / sizeof(float);
  if (dtype == NF_BF16) {
    const int tc = nf_tc_conv3x3_wgrad(x, g, N, H, W, Cin, Cout, stride, scratch, floats, dw);
    if (tc != NF_EUNSUPPORTED) return tc;
  }
  return nf_k_wgrad(dtype, x, N, H, W, Cin, g, Cout, stride, scratch, floats, dw);
}
