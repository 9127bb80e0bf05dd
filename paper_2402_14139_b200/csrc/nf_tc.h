// Tensor-core (tcgen05 / TMEM / TMA) convolution kernels: interface used by the step sequencer.
#pragma once
#include "nf_internal.h"

// Chooses, per operation, whether the configured shape runs on the tcgen05 kernels (L->fam[]).
void nf_tc_select(nf_layer* L);
// Floats of split-K scratch the tensor-core weight gradient needs (0 if unused).
size_t nf_tc_scratch_floats(const nf_layer* L);
// y = conv(x) in bf16 plus per-CTA channel partials (sum, sum of squares) in L->red; nb = partial count.
int nf_tc_conv_fwd(nf_layer* L, const void* x, int& nb);
// Same convolution for `count` samples without statistics (cache-filling forward).
int nf_tc_conv_fwd_eval(nf_layer* L, const void* x, int count);
// grad(W) = wgrad(x, L->dy) into the gradient arena.
int nf_tc_wgrad(nf_layer* L, const void* x);
// Floats of channel-partial scratch (L->red) the tensor-core forward needs.
size_t nf_tc_red_floats(const nf_layer* L);
// Stand-alone forward on the tensor-core path (NF_EUNSUPPORTED if the shape is not covered) and the
// status word (nf_device_flag bits) of the stand-alone operations.
int nf_tc_conv3x3_forward(const void* x, const void* w, int N, int H, int W, int Cin, int Cout, int stride, void* y);
int nf_tc_op_status(int32_t* out);
// Device address of that status word on the current device (looked up once per device).
int nf_tc_op_status_ptr(int32_t** out);
// Stand-alone weight gradient on the tensor-core path and the split-K scratch (floats) it needs (0: shape not covered).
size_t nf_tc_conv3x3_wgrad_scratch_floats(int N, int H, int W, int Cin, int Cout, int stride);
int nf_tc_conv3x3_wgrad(const void* x, const void* g, int N, int H, int W, int Cin, int Cout, int stride, float* part,
                        size_t part_floats, float* dw);
// Aux conv forward on tensor cores for `count` samples: L->h = ReLU(conv(a, Wa) + ba) in bf16.
int nf_tc_aux_fwd(nf_layer* L, const void* a, int count);
// BatchNorm + ReLU and the aux conv forward in one kernel: act_out = ReLU(L->y * scale + shift) and
// L->h = ReLU(conv(act_out, Wa) + ba), both in bf16.  NF_EUNSUPPORTED (nothing launched) when the layer's shape is not
// covered or it has a shortcut; nf_tc_bn_aux_fused tells whether the shape is covered.
bool nf_tc_bn_aux_fused(const nf_layer* L);
// Whether that kernel also replaces h by pooling partials (L->wpart: [tile][4][F], tiles of 14 x 8 pixels in row-major order
// per image) and a sign mask (in L->h: one bit per element, [N][Ha][Wa][F/8] bytes); nf_tc_pool_part_floats is the size of
// the partials (the workspace plan reserves it in the split-K scratch).
bool nf_tc_aux_pool_fused(const nf_layer* L);
size_t nf_tc_pool_part_floats(const nf_layer* L);
int nf_tc_bn_aux_fwd(nf_layer* L, void* act_out);
// Aux conv weight gradient on tensor cores: grad(Wa) = wgrad(a, L->dh).
int nf_tc_aux_wgrad(nf_layer* L, const void* a);
// Aux conv input gradient on tensor cores: L->da = dgrad(L->dh, Wa) in bf16.  Where the kernel can also reduce
// the BatchNorm-backward sums (no pool, folded-tap shape) it leaves *bn_nb > 0 partial blocks in L->red
// ([block][2][Cout]: sum dz, sum dz*xhat); otherwise *bn_nb = 0.
int nf_tc_aux_dgrad(nf_layer* L, int* bn_nb);
// Self-check of the bounded wait: one small CTA waits limit_ns on a barrier nobody arrives at; *waited_ns_dev (device)
// receives the time it waited and NF_ETIMEOUT is raised in the stand-alone status word.
int nf_tc_bounded_wait_probe(unsigned long long limit_ns, unsigned long long* waited_ns_dev);
// Two-pass input gradient: when nf_tc_dgrad_two_pass(L) holds (and the layer has no shortcut), nf_tc_aux_dgrad only reduces
// the BatchNorm-backward sums (L->da stays unwritten) and, once L->sdz / L->sdzx hold the finished sums, nf_tc_aux_dgrad_dy
// writes L->dy = BatchNorm-backward(da) with da formed again inside the kernel; M = elements per channel of the whole batch.
bool nf_tc_dgrad_two_pass(const nf_layer* L);
int nf_tc_aux_dgrad_dy(nf_layer* L, double M);
