// Tensor-core convolution kernels (placeholder selection: everything on the CUDA-core family).
#include "nf_tc.h"

void nf_tc_select(nf_layer* L) { L->fam[0] = L->fam[1] = L->fam[2] = L->fam[3] = 0; }
size_t nf_tc_scratch_floats(const nf_layer*) { return 0; }
int nf_tc_prepare(nf_layer*) { return NF_OK; }
int nf_tc_conv_fwd(nf_layer*, const void*, int&) { return NF_EUNSUPPORTED; }
int nf_tc_conv_fwd_eval(nf_layer*, const void*, int) { return NF_EUNSUPPORTED; }
int nf_tc_wgrad(nf_layer*, const void*) { return NF_EUNSUPPORTED; }
