// C ABI of libnf: handles, workspace planning, parameter exchange and the launch sequence of
// one local-layer step (Algorithm 2 body) and of the cache-filling forward pass.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <vector>

#include "nf_internal.h"
#include "nf_tc.h"

cudaStream_t g_nf_stream = 0;
long long g_nf_launches = 0;
static char g_nf_err[256] = "";

int nf_cuda_check(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return NF_OK;
  snprintf(g_nf_err, sizeof g_nf_err, "%s: %s", what, cudaGetErrorString(e));
  return NF_ECUDA;
}

namespace {

// ---- per-operation event timing
struct TraceRec { cudaEvent_t a, b; int op, slot; };
std::vector<TraceRec> g_recs;
size_t g_rec_used = 0;
bool g_trace_on = false;
double g_trace_ms[NF_TRACE_OPS][NF_TRACE_SLOTS];
long long g_trace_cnt[NF_TRACE_OPS][NF_TRACE_SLOTS];
int g_trace_slot = 0;
bool g_defer_update = false;  // nf_block_step: the layers' updates are launched together after the last layer

void trace_begin(int op) {
  if (!g_trace_on) return;
  if (g_rec_used == g_recs.size()) {
    if (g_recs.size() >= 65536) return;
    TraceRec r;
    if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) return;
    g_recs.push_back(r);
  }
  g_recs[g_rec_used].op = op;
  g_recs[g_rec_used].slot = g_trace_slot;
  cudaEventRecord(g_recs[g_rec_used].a, g_nf_stream);
}
void trace_end() {
  if (!g_trace_on || g_rec_used >= g_recs.size()) return;
  cudaEventRecord(g_recs[g_rec_used].b, g_nf_stream);
  ++g_rec_used;
}
int trace_flush() {
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  for (size_t i = 0; i < g_rec_used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, g_recs[i].a, g_recs[i].b) == cudaSuccess) {
      g_trace_ms[g_recs[i].op][g_recs[i].slot] += ms;
      g_trace_cnt[g_recs[i].op][g_recs[i].slot] += 1;
    }
  }
  g_rec_used = 0;
  return NF_OK;
}

// Carves the workspace; with base == nullptr only sizes it.
struct Carver {
  char* base;
  size_t off;
  void* take(size_t bytes) {
    off = nf_align_up(off, 256);
    void* p = base ? base + off : nullptr;
    off += bytes;
    return p;
  }
};

size_t plan(nf_layer* L, char* base, bool assign) {
  nf_layer tmp;
  nf_layer* D = assign ? L : &tmp;
  if (!assign) tmp = *L;
  Carver c{base, 0};
  const size_t es = nf_esize(L->o.dtype);
  const size_t N = L->o.N, Co = L->Cout, F = L->F, K = L->classes;
  const size_t ny = N * L->Ho * L->Wo * Co, na = N * L->Ha * L->Wa * Co, nh = N * L->Ha * L->Wa * F;
  D->status = (int32_t*)c.take(256);
  D->val = (float*)c.take(L->arena * 4);
  D->mom = (float*)c.take(L->arena * 4);
  D->grad = (float*)c.take(L->arena * 4);
  D->shadow = (bf16*)c.take(L->arena * 2);
  D->wa_t = (bf16*)c.take(F > 64 ? (size_t)9 * Co * F * 2 : 0);
  D->wpad = (bf16*)c.take(L->cin_pad ? (size_t)9 * Co * L->cin_pad * 2 : 0);
  D->gwpad = (float*)c.take(L->cin_pad ? (size_t)9 * Co * L->cin_pad * 4 : 0);
  D->rmean = (float*)c.take(Co * 4);
  D->rvar = (float*)c.take(Co * 4);
  D->scale = (float*)c.take(Co * 4);
  D->shift = (float*)c.take(Co * 4);
  D->mu = (float*)c.take(Co * 4);
  D->invstd = (float*)c.take(Co * 4);
  D->sdz = (float*)c.take(Co * 4);
  D->sdzx = (float*)c.take(Co * 4);
  const size_t state_end = c.off;
  D->y = c.take(ny * es);
  D->dy = c.take(ny * es);
  D->h = c.take(nh * es);
  D->dh = c.take(nh * es);
  D->da = c.take(na * es);
  D->act = c.take(na * es);
  D->xpad = c.take(L->cin_pad ? N * L->H * L->W * L->cin_pad * es : 0);
  D->p = (float*)c.take(N * 4 * F * 4);
  D->dp = (float*)c.take(N * 4 * F * 4);
  D->parg = (int32_t*)c.take(N * 4 * F * 4);
  D->dptot = (double*)c.take(4 * Co * 8);
  D->logits = (float*)c.take(N * K * 4);
  D->dlogits = (float*)c.take(N * K * 4);
  D->lossn = (float*)c.take(N * 4);
  size_t r1 = (size_t)nf_k_channel_blocks(N * L->Ho * L->Wo, (int)Co) * 2 * Co;
  size_t r2 = (size_t)nf_k_channel_blocks(N * L->Ha * L->Wa, (int)F) * 2 * F;
  D->red_floats = r1 > r2 ? r1 : r2;
  const size_t r3 = nf_tc_red_floats(L);
  if (r3 > D->red_floats) D->red_floats = r3;
  D->red = (float*)c.take(D->red_floats * 4);
  size_t w1 = (size_t)nf_k_wgrad_splits((int)N, L->Ho, L->Cin, (int)Co) * 9 * Co * L->Cin;
  size_t w2 = (size_t)nf_k_wgrad_splits((int)N, L->Ha, (int)Co, (int)F) * 9 * F * Co;
  D->wpart_floats = w1 > w2 ? w1 : w2;
  const size_t tc = nf_tc_scratch_floats(L);
  if (tc > D->wpart_floats) D->wpart_floats = tc;
  if (nf_tc_aux_pool_fused(L) && nf_tc_pool_part_floats(L) > D->wpart_floats) D->wpart_floats = nf_tc_pool_part_floats(L);
  if (nf_head_is_large((int)N, (int)(4 * F), (int)K)) {  // tiled head: logits before the bias, up to 16 batch ranges of gWf
    size_t hs = nf_head_scratch_floats((int)N, (int)(4 * F), (int)K);
    if (hs < (size_t)16 * K * 4 * F) hs = (size_t)16 * K * 4 * F;
    if (hs > D->wpart_floats) D->wpart_floats = hs;
  } else {
    const size_t hs = nf_head_small_scratch_floats((int)N, (int)(4 * F), (int)K);  // class-sliced head: shares of the softmax and of dp
    if (hs > D->wpart_floats) D->wpart_floats = hs;
  }
  D->wpart = (float*)c.take(D->wpart_floats * 4);
  if (L->o.host_io) {
    D->stage_x = c.take(N * L->H * L->W * L->Cin * es);
    D->stage_labels = (int32_t*)c.take(N * 4);
    D->stage_act = c.take(na * es);
    D->stage_loss = (float*)c.take(256);
    D->stage_xb[0] = D->stage_x;
    D->stage_lb[0] = D->stage_labels;
    D->stage_xb[1] = L->o.host_io == 2 ? c.take(N * L->H * L->W * L->Cin * es) : nullptr;
    D->stage_lb[1] = L->o.host_io == 2 ? (int32_t*)c.take(N * 4) : nullptr;
    D->stage_cur = 0;
    D->pre_x = nullptr;
    D->pre_l = nullptr;
  } else {
    D->stage_x = D->stage_act = nullptr;
    D->stage_labels = nullptr;
    D->stage_loss = nullptr;
  }
  if (assign) L->ws_bytes = state_end;  // bytes cleared at bind time
  return nf_align_up(c.off, 256);
}

void derive(nf_layer* L) {
  const int s = L->o.stride;
  L->Ho = (L->H - 1) / s + 1;
  L->Wo = (L->W - 1) / s + 1;
  L->Ha = L->o.maxpool ? L->Ho / 2 : L->Ho;
  L->Wa = L->o.maxpool ? L->Wo / 2 : L->Wo;
  const size_t cnt[NF_NPARAM] = {(size_t)9 * L->Cout * L->Cin, (size_t)L->Cout, (size_t)L->Cout,
                                 (size_t)9 * L->F * L->Cout,   (size_t)L->F,    (size_t)L->classes * 4 * L->F,
                                 (size_t)L->classes};
  size_t o = 0;
  for (int i = 0; i < NF_NPARAM; ++i) {
    L->off[i] = o;
    L->cnt[i] = cnt[i];
    o = nf_align_up(o + cnt[i], 64);
  }
  L->arena = o;
  nf_tc_select(L);
}

bool misaligned(const void* p) { return ((uintptr_t)p & 15) != 0; }

// logical [A][B][3][3]  <->  kernel [tap][Ap][B] (rows A..Ap-1 are padding, kept zero)
void to_kernel_layout(const float* src, float* dst, size_t A, size_t Ap, size_t B) {
  for (size_t a = 0; a < A; ++a)
    for (size_t b = 0; b < B; ++b)
      for (int t = 0; t < 9; ++t) dst[(t * Ap + a) * B + b] = src[(a * B + b) * 9 + t];
}
void from_kernel_layout(const float* src, float* dst, size_t A, size_t Ap, size_t B) {
  for (size_t a = 0; a < A; ++a)
    for (size_t b = 0; b < B; ++b)
      for (int t = 0; t < 9; ++t) dst[(a * B + b) * 9 + t] = src[(t * Ap + a) * B + b];
}

// Converts one parameter tensor between the caller's logical form (n_log floats) and the padded kernel
// form (cnt floats, zero in the padding).  dir 0: logical -> kernel, 1: kernel -> logical.
void convert_param(const nf_layer* L, int id, const float* src, float* dst, int dir) {
  const size_t F = L->Flog, Fp = L->F, Co = L->Cout, K = L->classes;
  switch (id) {
    case NF_P_W:
      if (dir == 0) to_kernel_layout(src, dst, Co, Co, L->Cin); else from_kernel_layout(src, dst, Co, Co, L->Cin);
      break;
    case NF_P_WA:
      if (dir == 0) to_kernel_layout(src, dst, F, Fp, Co); else from_kernel_layout(src, dst, F, Fp, Co);
      break;
    case NF_P_BA:
      memcpy(dst, src, F * sizeof(float));
      break;
    case NF_P_WF:
      for (size_t k = 0; k < K; ++k)
        if (dir == 0) memcpy(dst + k * 4 * Fp, src + k * 4 * F, 4 * F * sizeof(float));
        else memcpy(dst + k * 4 * F, src + k * 4 * Fp, 4 * F * sizeof(float));
      break;
    default: {
      const size_t n = id == NF_P_BF ? K : Co;
      memcpy(dst, src, n * sizeof(float));
    }
  }
}

size_t logical_count(const nf_layer* L, int id) {
  switch (id) {
    case NF_P_W: return (size_t)9 * L->Cout * L->Cin;
    case NF_P_WA: return (size_t)9 * L->Flog * L->Cout;
    case NF_P_BA: return L->Flog;
    case NF_P_WF: return (size_t)L->classes * 4 * L->Flog;
    case NF_P_BF: return L->classes;
    default: return L->Cout;
  }
}

}  // namespace

extern "C" {

nf_layer* nf_layer_create(int Cin, int Cout, int H, int W, int F, int classes) {
  if (Cin < 1 || Cout < 1 || H < 1 || W < 1 || F < 1 || classes < 1) return nullptr;
  nf_layer* L = (nf_layer*)calloc(1, sizeof(nf_layer));
  if (!L) return nullptr;
  L->Cin = Cin; L->Cout = Cout; L->H = H; L->W = W; L->Flog = F; L->F = (F + 7) / 8 * 8; L->classes = classes;
  L->o.N = 1; L->o.stride = 1; L->o.maxpool = 0; L->o.dtype = NF_BF16;
  L->o.momentum = 0.9f; L->o.bn_eps = 1e-5f; L->o.bn_momentum = 0.1f; L->o.host_io = 0;
  derive(L);
  return L;
}

void nf_layer_destroy(nf_layer* L) { free(L); }

int nf_layer_configure(nf_layer* L, const nf_layer_opts* o) {
  if (!L || !o) return NF_EINVAL;
  if (o->N < 1 || (o->stride != 1 && o->stride != 2) || (o->dtype != NF_F32 && o->dtype != NF_BF16)) return NF_EINVAL;
  if (!(o->momentum >= 0.f && o->momentum < 1.f) || !(o->bn_eps > 0.f) || !(o->bn_momentum >= 0.f && o->bn_momentum <= 1.f))
    return NF_EINVAL;
  const int Ho = (L->H - 1) / o->stride + 1, Wo = (L->W - 1) / o->stride + 1;
  if (o->maxpool && ((Ho & 1) || (Wo & 1))) return NF_EINVAL;
  if ((o->loss != NF_LOSS_CE && o->loss != NF_LOSS_MSE) || (o->aux_pool != NF_POOL_AVG && o->aux_pool != NF_POOL_MAX)) return NF_EINVAL;
  L->o = *o;
  L->o.maxpool = o->maxpool ? 1 : 0;
  L->o.host_io = o->host_io == 2 ? 2 : o->host_io ? 1 : 0;
  L->ws = nullptr;
  derive(L);
  return NF_OK;
}

size_t nf_layer_workspace_bytes(const nf_layer* L) {
  if (!L) return 0;
  return plan(const_cast<nf_layer*>(L), nullptr, false);
}

int nf_layer_bind_workspace(nf_layer* L, void* dev, size_t bytes) {
  if (!L || !dev) return NF_EINVAL;
  if ((uintptr_t)dev & 255) return NF_EALIGN;
  if (bytes < nf_layer_workspace_bytes(L)) return NF_ENOWS;
  plan(L, (char*)dev, true);
  L->ws = (char*)dev;
  NF_CUDA(cudaMemsetAsync(dev, 0, L->ws_bytes, g_nf_stream));
  std::vector<float> ones(L->Cout, 1.0f);
  NF_CUDA(cudaMemcpyAsync(L->val + L->off[NF_P_GAMMA], ones.data(), L->Cout * 4, cudaMemcpyHostToDevice, g_nf_stream));
  NF_CUDA(cudaMemcpyAsync(L->rvar, ones.data(), L->Cout * 4, cudaMemcpyHostToDevice, g_nf_stream));
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  return nf_k_shadow(L->val, L->shadow, L->arena);
}

static int param_ptr(nf_layer* L, int which, float** dev, size_t* n, int* conv_a, int* conv_b) {
  const int id = which & 0xff, kind = which & 0xf00;
  *conv_a = *conv_b = 0;
  if (id == NF_P_RMEAN || id == NF_P_RVAR) {
    if (kind != NF_K_VALUE) return NF_EINVAL;
    *dev = id == NF_P_RMEAN ? L->rmean : L->rvar;
    *n = L->Cout;
    return NF_OK;
  }
  if (id < 0 || id >= NF_NPARAM) return NF_EINVAL;
  float* base = kind == NF_K_VALUE ? L->val : kind == NF_K_MOMENTUM ? L->mom : kind == NF_K_GRAD ? L->grad : nullptr;
  if (!base) return NF_EINVAL;
  *dev = base + L->off[id];
  *n = L->cnt[id];
  if (id == NF_P_W) { *conv_a = L->Cout; *conv_b = L->Cin; }
  if (id == NF_P_WA) { *conv_a = L->F; *conv_b = L->Cout; }
  return NF_OK;
}

int nf_layer_set_param(nf_layer* L, int which, const float* host, size_t n) {
  if (!L || !host) return NF_EINVAL;
  if (!L->ws) return NF_ENOWS;
  if ((which & 0xf00) == NF_K_GRAD) return NF_EINVAL;
  float* dev; size_t cnt; int A, B;
  int rc = param_ptr(L, which, &dev, &cnt, &A, &B);
  if (rc != NF_OK) return rc;
  const int id = which & 0xff;
  if (n != logical_count(L, id)) return NF_EINVAL;
  std::vector<float> tmp(cnt, 0.f);
  convert_param(L, id, host, tmp.data(), 0);
  NF_CUDA(cudaMemcpyAsync(dev, tmp.data(), cnt * 4, cudaMemcpyHostToDevice, g_nf_stream));
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  if ((which & 0xf00) == NF_K_VALUE && id < NF_NPARAM) {
    rc = nf_k_shadow(L->val, L->shadow, L->arena);
    if (rc != NF_OK) return rc;
    NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  }
  return NF_OK;
}

int nf_layer_get_param(nf_layer* L, int which, float* host, size_t n) {
  if (!L || !host) return NF_EINVAL;
  if (!L->ws) return NF_ENOWS;
  float* dev; size_t cnt; int A, B;
  int rc = param_ptr(L, which, &dev, &cnt, &A, &B);
  if (rc != NF_OK) return rc;
  const int id = which & 0xff;
  if (n != logical_count(L, id)) return NF_EINVAL;
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  std::vector<float> tmp(cnt);
  NF_CUDA(cudaMemcpy(tmp.data(), dev, cnt * 4, cudaMemcpyDeviceToHost));
  convert_param(L, id, tmp.data(), host, 1);
  return NF_OK;
}

#define NF_TRY(x)                 \
  do {                            \
    int rc_ = (x);                \
    if (rc_ != NF_OK) return rc_; \
  } while (0)

// The whole step (phase < 0, world = 1), or one of the four phases of the data-parallel step: 0 = conv forward and
// the rank's per-channel sums; 1 = normalise with the statistics of the whole batch ... aux input gradient and the
// rank's BatchNorm-backward sums; 2 = BatchNorm backward with the sums of the whole batch, weight gradient; 3 = update.
static int step_phases(nf_layer* L, const void* x, const int32_t* labels, float lr, float* loss_out, void* act_out, int phase,
                       int world) {
  if (!L || !x || !labels || !loss_out || !act_out) return NF_EINVAL;
  if (!L->ws) return NF_ENOWS;
  if (misaligned(x) || misaligned(act_out) || ((uintptr_t)labels & 3) || ((uintptr_t)loss_out & 3)) return NF_EALIGN;
  const int dt = L->o.dtype, N = L->o.N, Ci = L->Cin, Co = L->Cout, F = L->F, K = L->classes, s = L->o.stride;
  const int pool = L->o.maxpool, Ho = L->Ho, Wo = L->Wo, Ha = L->Ha, Wa = L->Wa, D = 4 * F;
  const double M = (double)N * Ho * Wo * world;   // BatchNorm sample count of the whole batch
  const int n_scale = N * world;                  // batch size in the loss mean
  const bool all = phase < 0;
  const void* Wm = dt == NF_F32 ? (const void*)(L->val + L->off[NF_P_W]) : (const void*)(L->shadow + L->off[NF_P_W]);
  const void* Wx = dt == NF_F32 ? (const void*)(L->val + L->off[NF_P_WA]) : (const void*)(L->shadow + L->off[NF_P_WA]);
  float* g = L->grad;
  int nb = 0;

  // Eq. 1: conv, BatchNorm (batch statistics), ReLU, optional max-pool -> act_out
  if (all || phase == 0) {
  trace_begin(0);
  if (L->fam[0]) {
    NF_TRY(nf_tc_conv_fwd(L, x, nb));
  } else {
    NF_TRY(nf_k_conv(dt, x, N, L->H, L->W, Ci, Wm, (long)Co * Ci, Ci, 1, 0, nullptr, 0, s, Co, L->y));
    NF_TRY(nf_k_channel_sums(dt, L->y, (size_t)N * Ho * Wo, Co, L->red, L->red_floats, &nb));
  }
  trace_end();
  if (!all) return nf_k_partial_totals(L->red, nb, Co, L->dptot);
  }
  if (all || phase == 1) {
  trace_begin(1);
  if (all) {
    NF_TRY(nf_k_bn_finalize(L->red, nb, Co, M, L->val + L->off[NF_P_GAMMA], L->val + L->off[NF_P_BETA], L->o.bn_eps,
                              L->o.bn_momentum, L->scale, L->shift, L->mu, L->invstd, L->rmean, L->rvar));
  } else {
    NF_TRY(nf_k_bn_finalize_tot(L->dptot, Co, M, L->val + L->off[NF_P_GAMMA], L->val + L->off[NF_P_BETA], L->o.bn_eps,
                                  L->o.bn_momentum, L->scale, L->shift, L->mu, L->invstd, L->rmean, L->rvar));
  }
  // where the shape allows, the aux forward kernel normalises y on the way in and writes act_out itself
  const bool fused_bn_aux = nf_tc_bn_aux_fused(L) && !L->skip;
  if (!fused_bn_aux) NF_TRY(nf_k_bn_apply(dt, L->y, N, Ho, Wo, Co, pool, L->scale, L->shift, act_out, L->skip));
  trace_end();
  // Eq. 2: aux conv + ReLU, average pool to 2x2, linear; Eq. 3: softmax cross-entropy
  trace_begin(2);
  if (fused_bn_aux) {
    NF_TRY(nf_tc_bn_aux_fwd(L, act_out));
  } else if (L->fam[2]) {
    NF_TRY(nf_tc_aux_fwd(L, act_out, N));
  } else {
    NF_TRY(nf_k_conv(dt, act_out, N, Ha, Wa, Co, Wx, (long)F * Co, Co, 1, 0, L->val + L->off[NF_P_BA], 1, 1, F, L->h));
  }
  trace_end();
  trace_begin(3);
  // h_masked: the aux forward left pooling partials (L->wpart) and a sign mask (in L->h) instead of h
  const bool h_masked = fused_bn_aux && nf_tc_aux_pool_fused(L);
  if (h_masked) {
    NF_TRY(nf_k_pool_finish(L->wpart, N, Ha / 8, Wa / 14, F, 1.f / (float)((Ha / 2) * (Wa / 2)), L->p));
  } else if (L->o.aux_pool == NF_POOL_MAX) {
    NF_TRY(nf_k_auxmax(dt, L->h, N, Ha, Wa, F, L->p, L->parg));
  } else {
    int rc = dt == NF_BF16 ? nf_k_avgpool_fast(L->h, N, Ha, Wa, F, L->wpart, L->wpart_floats, L->p) : NF_EUNSUPPORTED;
    if (rc == NF_EUNSUPPORTED) rc = nf_k_avgpool(dt, L->h, N, Ha, Wa, F, L->p);
    if (rc != NF_OK) return rc;
  }
  if (nf_head_is_large(N, D, K)) {  // late blocks: tens of thousands of samples, up to 1024 head inputs
    NF_TRY(nf_head_step(L->p, labels, N, D, K, L->val + L->off[NF_P_WF], L->val + L->off[NF_P_BF], L->logits, L->dlogits, L->dp,
                        L->lossn, L->status, L->o.loss, g + L->off[NF_P_WF], g + L->off[NF_P_BF], loss_out, L->wpart,
                        L->wpart_floats, n_scale));
  } else {
    // forward, loss and the gradients of gamma_n cut by class slices; heads wider than that covers: one block per sample
    int rc = nf_head_small_step(L->p, labels, N, D, K, L->val + L->off[NF_P_WF], L->val + L->off[NF_P_BF], L->logits, L->dp, L->lossn,
                                L->status, L->o.loss, g + L->off[NF_P_WF], g + L->off[NF_P_BF], loss_out, L->wpart, L->wpart_floats,
                                n_scale);
    if (rc == NF_EUNSUPPORTED) {
      NF_TRY(nf_k_fc_ce(L->p, labels, N, D, K, L->val + L->off[NF_P_WF], L->val + L->off[NF_P_BF], L->logits, L->dlogits,
                        L->dp, L->lossn, L->status, L->o.loss, n_scale));
      rc = nf_k_fc_wgrad(L->p, L->dlogits, L->lossn, N, D, K, g + L->off[NF_P_WF], g + L->off[NF_P_BF], loss_out, L->status, n_scale);
    }
    if (rc != NF_OK) return rc;
  }
  trace_end();
  trace_begin(4);
  int dh_nb = 0;
  if (h_masked) {
    NF_TRY(nf_k_dh_mask((const uint8_t*)L->h, L->dp, N, Ha, Wa, F, L->dh, L->red, L->red_floats, &dh_nb));
  } else if (L->o.aux_pool == NF_POOL_MAX) {
    NF_TRY(nf_k_dh_max(dt, L->h, L->dp, L->parg, N, Ha, Wa, F, L->dh));
  } else {
    int rc = dt == NF_BF16 ? nf_k_dh_fast(L->h, L->dp, N, Ha, Wa, F, L->dh, L->red, L->red_floats, &dh_nb) : NF_EUNSUPPORTED;
    if (rc == NF_EUNSUPPORTED) {
      dh_nb = 0;
      rc = nf_k_dh(dt, L->h, L->dp, N, Ha, Wa, F, L->dh);
    }
    if (rc != NF_OK) return rc;
  }
  if (dh_nb) NF_TRY(nf_k_sum_partials(L->red, dh_nb, F, 0, g + L->off[NF_P_BA]));
  if (L->fam[3]) {
    NF_TRY(nf_tc_aux_wgrad(L, act_out));
  } else {
    NF_TRY(nf_k_wgrad(dt, act_out, N, Ha, Wa, Co, L->dh, F, 1, L->wpart, L->wpart_floats, g + L->off[NF_P_WA]));
  }
  if (!dh_nb) {
    NF_TRY(nf_k_channel_sums(dt, L->dh, (size_t)N * Ha * Wa, F, L->red, L->red_floats, &nb));
    NF_TRY(nf_k_sum_partials(L->red, nb, F, 0, g + L->off[NF_P_BA]));
  }
  trace_end();
  // gradient at the aux input
  trace_begin(8);
  int bn_nb = 0;  // > 0: the input-gradient kernel has already left the BatchNorm-backward partial sums in L->red
  if (L->fam[3]) {
    NF_TRY(nf_tc_aux_dgrad(L, &bn_nb));
  } else {
    NF_TRY(nf_k_conv(dt, L->dh, N, Ha, Wa, F, Wx, (long)F * Co, 1, Co, 1, nullptr, 0, 1, Co, L->da));
  }
  // a trainable shortcut joined at the BatchNorm output gets the gradient at that sum
  if (L->skip_grad) NF_TRY(nf_k_write_dz(dt, L->y, L->da, N, Ho, Wo, Co, pool, L->scale, L->shift, L->skip, L->skip_grad));
  trace_end();
  // back through pool / ReLU / BatchNorm
  trace_begin(5);
  if (bn_nb) {
    nb = bn_nb;
  } else {
    NF_TRY(nf_k_bn_bwd_reduce(dt, L->y, L->da, N, Ho, Wo, Co, pool, L->scale, L->shift, L->mu, L->invstd, L->red,
                                L->red_floats, &nb, L->skip));
  }
  if (!all) return nf_k_partial_totals(L->red, nb, Co, L->dptot + 2 * Co);
  }
  if (all || phase == 2) {
  if (all) {
    NF_TRY(nf_k_bn_bwd_finalize(L->red, nb, Co, L->sdz, L->sdzx, g + L->off[NF_P_GAMMA], g + L->off[NF_P_BETA]));
  } else {
    NF_TRY(nf_k_bn_bwd_finalize_tot(L->dptot + 2 * Co, Co, world, L->sdz, L->sdzx, g + L->off[NF_P_GAMMA], g + L->off[NF_P_BETA]));
  }
  if (nf_tc_dgrad_two_pass(L) && !L->skip && !L->skip_grad) {  // second pass of the input gradient writes dy itself; da was never stored
    NF_TRY(nf_tc_aux_dgrad_dy(L, M));
  } else {
    NF_TRY(nf_k_bn_bwd_apply(dt, L->y, L->da, N, Ho, Wo, Co, pool, L->scale, L->shift, L->mu, L->invstd, L->sdz, L->sdzx,
                             M, L->dy, L->skip));
  }
  trace_end();
  // gradient of theta_n (the layer input receives none), then the update
  trace_begin(6);
  if (L->fam[1]) {
    NF_TRY(nf_tc_wgrad(L, x));
  } else {
    NF_TRY(nf_k_wgrad(dt, x, N, L->H, L->W, Ci, L->dy, Co, s, L->wpart, L->wpart_floats, g + L->off[NF_P_W]));
  }
  trace_end();
  if (!all) return NF_OK;
  }
  if (g_defer_update) return NF_OK;
  trace_begin(7);
  NF_TRY(nf_k_sgd(L->val, L->mom, L->grad, L->shadow, L->arena, lr, L->o.momentum));
  trace_end();
  return NF_OK;
}

int nf_layer_step(nf_layer* L, const void* x, const int32_t* labels, float lr, float* loss_out, void* act_out) {
  return step_phases(L, x, labels, lr, loss_out, act_out, -1, 1);
}

int nf_layer_set_skip(nf_layer* L, const void* skip) {
  if (!L) return NF_EINVAL;
  if (skip && misaligned(skip)) return NF_EALIGN;
  L->skip = skip;
  return NF_OK;
}

int nf_layer_set_skip_grad(nf_layer* L, void* dz_out) {
  if (!L) return NF_EINVAL;
  if (dz_out && misaligned(dz_out)) return NF_EALIGN;
  L->skip_grad = dz_out;
  return NF_OK;
}

int nf_layer_step_dp(nf_layer* L, int phase, const void* x, const int32_t* labels, float lr, float* loss_out, void* act_out,
                     int world) {
  if (phase < 0 || phase > 3 || world < 1) return NF_EINVAL;
  return step_phases(L, x, labels, lr, loss_out, act_out, phase, world);
}

int nf_layer_dp_buffer(nf_layer* L, int which, void** dev_ptr, size_t* bytes) {
  if (!L || !dev_ptr || !bytes || which < 0 || which > 2) return NF_EINVAL;
  if (!L->ws) return NF_ENOWS;
  if (which == 2) {
    *dev_ptr = L->grad;
    *bytes = L->arena * sizeof(float);
  } else {
    *dev_ptr = L->dptot + (size_t)which * 2 * L->Cout;
    *bytes = (size_t)2 * L->Cout * sizeof(double);
  }
  return NF_OK;
}

int nf_layer_stored_tensor(nf_layer* L, int which, void** dev_ptr, size_t* bytes) {
  if (!L || !dev_ptr || !bytes) return NF_EINVAL;
  if (!L->ws) return NF_ENOWS;
  const size_t es = nf_esize(L->o.dtype), N = L->o.N;
  const size_t ny = N * L->Ho * L->Wo * L->Cout, na = N * L->Ha * L->Wa * L->Cout, nh = N * L->Ha * L->Wa * L->F;
  switch (which) {
    case NF_T_Y: *dev_ptr = L->y; *bytes = ny * es; break;
    case NF_T_DY: *dev_ptr = L->dy; *bytes = ny * es; break;
    case NF_T_H: *dev_ptr = L->h; *bytes = nh * es; break;
    case NF_T_DH: *dev_ptr = L->dh; *bytes = nh * es; break;
    case NF_T_DA: *dev_ptr = L->da; *bytes = na * es; break;
    case NF_T_P: *dev_ptr = L->p; *bytes = N * 4 * L->F * sizeof(float); break;
    case NF_T_DP: *dev_ptr = L->dp; *bytes = N * 4 * L->F * sizeof(float); break;
    case NF_T_LOGITS: *dev_ptr = L->logits; *bytes = N * L->classes * sizeof(float); break;
    case NF_T_HMASK: *dev_ptr = L->h; *bytes = nh / 8; break;
    default: return NF_EINVAL;
  }
  return NF_OK;
}

int nf_layer_step_host(nf_layer* L, const void* xh, const int32_t* lh, float lr, float* loss_h, void* act_h) {
  if (!L || !xh || !lh || !loss_h) return NF_EINVAL;
  if (!L->ws) return NF_ENOWS;
  if (!L->o.host_io) return NF_EINVAL;
  const size_t es = nf_esize(L->o.dtype), N = L->o.N;
  const size_t xb = N * L->H * L->W * L->Cin * es, ab = N * L->Ha * L->Wa * L->Cout * es;
  NF_CUDA(cudaMemcpyAsync(L->stage_x, xh, xb, cudaMemcpyHostToDevice, g_nf_stream));
  NF_CUDA(cudaMemcpyAsync(L->stage_labels, lh, N * 4, cudaMemcpyHostToDevice, g_nf_stream));
  NF_TRY(nf_layer_step(L, L->stage_x, L->stage_labels, lr, L->stage_loss, L->stage_act));
  NF_CUDA(cudaMemcpyAsync(loss_h, L->stage_loss, 4, cudaMemcpyDeviceToHost, g_nf_stream));
  if (act_h) NF_CUDA(cudaMemcpyAsync(act_h, L->stage_act, ab, cudaMemcpyDeviceToHost, g_nf_stream));
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  return NF_OK;
}

int nf_layer_status(nf_layer* L) {
  if (!L) return NF_EINVAL;
  if (!L->ws) return NF_ENOWS;
  int32_t v = 0;
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  NF_CUDA(cudaMemcpy(&v, L->status, 4, cudaMemcpyDeviceToHost));
  NF_CUDA(cudaMemset(L->status, 0, 4));
  return v;
}

nf_block* nf_block_create(nf_layer* const* layers, int n) {
  if (!layers || n < 1) return nullptr;
  for (int i = 0; i < n; ++i) {
    if (!layers[i] || !layers[i]->ws) return nullptr;
    if (i > 0) {
      const nf_layer *a = layers[i - 1], *b = layers[i];
      if (a->Cout != b->Cin || a->Ha != b->H || a->Wa != b->W || a->o.dtype != b->o.dtype || a->o.N != b->o.N) return nullptr;
    }
  }
  nf_block* B = (nf_block*)calloc(1, sizeof(nf_block));
  if (!B) return nullptr;
  B->layers = (nf_layer**)calloc(n, sizeof(nf_layer*));
  if (!B->layers) { free(B); return nullptr; }
  B->n = n;
  memcpy(B->layers, layers, n * sizeof(nf_layer*));
  return B;
}

void nf_block_destroy(nf_block* B) {
  if (!B) return;
  free(B->layers);
  free(B);
}

static int layer_eval_forward(nf_layer* L, const void* in, int count, void* dst);

int nf_block_cache_n(nf_block* B, const void* x, void* out, int count) {
  if (!B || !x || !out) return NF_EINVAL;
  if (count < 1 || count > B->layers[0]->o.N) return NF_EINVAL;
  if (misaligned(x) || misaligned(out)) return NF_EALIGN;
  const void* in = x;
  for (int l = 0; l < B->n; ++l) {
    nf_layer* L = B->layers[l];
    void* dst = l == B->n - 1 ? out : L->dy;
    NF_TRY(layer_eval_forward(L, in, count, dst));
    in = dst;
  }
  return NF_OK;
}

// eval-mode forward of one layer for `count` samples into dst (conv, running-statistics BatchNorm, ReLU, pool)
static int layer_eval_forward(nf_layer* L, const void* in, int count, void* dst) {
  const int dt = L->o.dtype;
  const void* Wm = dt == NF_F32 ? (const void*)(L->val + L->off[NF_P_W]) : (const void*)(L->shadow + L->off[NF_P_W]);
  if (L->fam[0]) {
    NF_TRY(nf_tc_conv_fwd_eval(L, in, count));
  } else {
    NF_TRY(nf_k_conv(dt, in, count, L->H, L->W, L->Cin, Wm, (long)L->Cout * L->Cin, L->Cin, 1, 0, nullptr, 0, L->o.stride,
                       L->Cout, L->y));
  }
  NF_TRY(nf_k_bn_eval_coeffs(L->Cout, L->val + L->off[NF_P_GAMMA], L->val + L->off[NF_P_BETA], L->o.bn_eps, L->rmean, L->rvar,
                               L->scale, L->shift));
  return nf_k_bn_apply(dt, L->y, count, L->Ho, L->Wo, L->Cout, L->o.maxpool, L->scale, L->shift, dst, L->skip);
}

int nf_layer_predict(nf_layer* L, const void* x, int count, void* act_out, float* logits_out, int32_t* pred_out) {
  if (!L || !x || !pred_out) return NF_EINVAL;
  if (!L->ws) return NF_ENOWS;
  if (count < 1 || count > L->o.N) return NF_EINVAL;
  if (misaligned(x) || (act_out && misaligned(act_out))) return NF_EALIGN;
  const int dt = L->o.dtype, Co = L->Cout, F = L->F, Ha = L->Ha, Wa = L->Wa;
  void* a = act_out ? act_out : L->act;
  NF_TRY(layer_eval_forward(L, x, count, a));
  const void* Wx = dt == NF_F32 ? (const void*)(L->val + L->off[NF_P_WA]) : (const void*)(L->shadow + L->off[NF_P_WA]);
  if (L->fam[2]) {
    NF_TRY(nf_tc_aux_fwd(L, a, count));
  } else {
    NF_TRY(nf_k_conv(dt, a, count, Ha, Wa, Co, Wx, (long)F * Co, Co, 1, 0, L->val + L->off[NF_P_BA], 1, 1, F, L->h));
  }
  if (L->o.aux_pool == NF_POOL_MAX) {
    NF_TRY(nf_k_auxmax(dt, L->h, count, Ha, Wa, F, L->p, L->parg));
  } else {
    int rc = dt == NF_BF16 ? nf_k_avgpool_fast(L->h, count, Ha, Wa, F, L->wpart, L->wpart_floats, L->p) : NF_EUNSUPPORTED;
    if (rc == NF_EUNSUPPORTED) rc = nf_k_avgpool(dt, L->h, count, Ha, Wa, F, L->p);
    if (rc != NF_OK) return rc;
  }
  // the caller's logits have `classes` columns over the logical 4*Flog inputs; the padded inputs are zero
  if (nf_head_is_large(count, 4 * F, L->classes)) {
    float* lg = logits_out ? logits_out : L->logits;
    NF_TRY(nf_head_logits(L->p, count, 4 * F, L->classes, L->val + L->off[NF_P_WF], L->val + L->off[NF_P_BF], lg, L->wpart));
    return nf_head_predict(lg, count, L->classes, pred_out);
  }
  return nf_k_fc_predict(L->p, count, 4 * F, L->classes, L->val + L->off[NF_P_WF], L->val + L->off[NF_P_BF], logits_out, pred_out);
}

int nf_count_equal(const int32_t* a, const int32_t* b, long long n, unsigned long long* count) {
  if (!a || !b || !count || n < 1) return NF_EINVAL;
  return nf_k_count_equal(a, b, n, count);
}

long long nf_layer_param_count(const nf_layer* L, int part) {
  if (!L) return NF_EINVAL;
  const long long main = 9LL * L->Cout * L->Cin + 2LL * L->Cout;
  const long long aux = 9LL * L->Flog * L->Cout + L->Flog + (long long)L->classes * (4 * L->Flog + 1);
  return part == 0 ? main : part == 1 ? aux : main + aux;
}

int nf_select_exit(const double* val_accuracy, const long long* params, int n_layers) {
  if (!val_accuracy || !params || n_layers < 1) return NF_EINVAL;
  int best = 0;
  for (int i = 1; i < n_layers; ++i)
    if (val_accuracy[i] > val_accuracy[best] || (val_accuracy[i] == val_accuracy[best] && params[i] < params[best])) best = i;
  return best;
}

int nf_block_cache(nf_block* B, const void* x, void* out) {
  if (!B) return NF_EINVAL;
  return nf_block_cache_n(B, x, out, B->layers[0]->o.N);
}

int nf_block_step(nf_block* B, const void* x, const int32_t* labels, float lr, float* loss_out, void* act_out) {
  if (!B || !x || !labels || !loss_out) return NF_EINVAL;
  const void* in = x;
  for (int l = 0; l < B->n; ++l) {
    nf_layer* L = B->layers[l];
    void* dst = (l == B->n - 1 && act_out) ? act_out : L->act;
    g_trace_slot = l < NF_TRACE_SLOTS ? l : NF_TRACE_SLOTS - 1;
    g_defer_update = true;  // no layer reads another layer's parameters, so the updates can wait for the end of the pass
    const int rc = nf_layer_step(L, in, labels, lr, loss_out + l, dst);
    g_defer_update = false;
    g_trace_slot = 0;
    if (rc != NF_OK) return rc;
    in = dst;
  }
  // Algorithm 2's update of every layer of the block, one launch per group of layers with equal momentum
  trace_begin(7);
  for (int l0 = 0; l0 < B->n;) {
    SgdTable tb{};
    const float mu = B->layers[l0]->o.momentum;
    int l = l0;
    for (; l < B->n && tb.count < kSgdMaxArenas && B->layers[l]->o.momentum == mu; ++l) {
      nf_layer* L = B->layers[l];
      tb.val[tb.count] = L->val; tb.mom[tb.count] = L->mom; tb.grad[tb.count] = L->grad; tb.shadow[tb.count] = L->shadow;
      tb.n[tb.count++] = L->arena;
    }
    NF_TRY(nf_k_sgd_multi(tb, lr, mu));
    l0 = l;
  }
  trace_end();
  return NF_OK;
}

int nf_block_step_host(nf_block* B, const void* xh, const int32_t* lh, float lr, float* loss_h, void* act_h) {
  if (!B || !xh || !lh || !loss_h) return NF_EINVAL;
  nf_layer* L0 = B->layers[0];
  nf_layer* Ll = B->layers[B->n - 1];
  if (!L0->o.host_io || B->n > 64) return NF_EINVAL;
  const size_t es = nf_esize(L0->o.dtype), N = L0->o.N;
  NF_CUDA(cudaMemcpyAsync(L0->stage_x, xh, N * L0->H * L0->W * L0->Cin * es, cudaMemcpyHostToDevice, g_nf_stream));
  NF_CUDA(cudaMemcpyAsync(L0->stage_labels, lh, N * 4, cudaMemcpyHostToDevice, g_nf_stream));
  NF_TRY(nf_block_step(B, L0->stage_x, L0->stage_labels, lr, L0->stage_loss, nullptr));
  NF_CUDA(cudaMemcpyAsync(loss_h, L0->stage_loss, 4 * (size_t)B->n, cudaMemcpyDeviceToHost, g_nf_stream));
  if (act_h)
    NF_CUDA(cudaMemcpyAsync(act_h, Ll->act, N * Ll->Ha * Ll->Wa * Ll->Cout * es, cudaMemcpyDeviceToHost, g_nf_stream));
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  return NF_OK;
}

int nf_trace_enable(int on) {
  if (trace_flush() != NF_OK) return NF_ECUDA;
  g_trace_on = on != 0;
  memset(g_trace_ms, 0, sizeof g_trace_ms);
  memset(g_trace_cnt, 0, sizeof g_trace_cnt);
  return NF_OK;
}

int nf_trace_read(int op, int slot, double* ms_total, long long* groups) {
  if (op < 0 || op >= NF_TRACE_OPS || slot < 0 || slot >= NF_TRACE_SLOTS || !ms_total || !groups) return NF_EINVAL;
  if (trace_flush() != NF_OK) return NF_ECUDA;
  *ms_total = g_trace_ms[op][slot];
  *groups = g_trace_cnt[op][slot];
  return NF_OK;
}

// copy stream and event of the input prefetch (created on first use; they hold no device memory)
static cudaStream_t g_copy_stream = nullptr;
static cudaEvent_t g_copy_done = nullptr;

int nf_block_step_host_next(nf_block* B, const void* xh, const int32_t* lh, float lr, float* loss_h, void* act_h,
                            const void* next_xh, const int32_t* next_lh) {
  if (!B || !xh || !lh || !loss_h) return NF_EINVAL;
  nf_layer* L0 = B->layers[0];
  nf_layer* Ll = B->layers[B->n - 1];
  if (L0->o.host_io != 2 || B->n > 64 || ((next_xh == nullptr) != (next_lh == nullptr))) return NF_EINVAL;
  if (!g_copy_stream) {
    NF_CUDA(cudaStreamCreateWithFlags(&g_copy_stream, cudaStreamNonBlocking));
    NF_CUDA(cudaEventCreateWithFlags(&g_copy_done, cudaEventDisableTiming));
  }
  const size_t es = nf_esize(L0->o.dtype), N = L0->o.N, xbytes = N * L0->H * L0->W * L0->Cin * es;
  if (L0->pre_x == xh && L0->pre_l == lh) {  // this batch was started on its way during the previous call
    L0->stage_cur ^= 1;
    NF_CUDA(cudaStreamWaitEvent(g_nf_stream, g_copy_done, 0));
  } else {
    NF_CUDA(cudaMemcpyAsync(L0->stage_xb[L0->stage_cur], xh, xbytes, cudaMemcpyHostToDevice, g_nf_stream));
    NF_CUDA(cudaMemcpyAsync(L0->stage_lb[L0->stage_cur], lh, N * 4, cudaMemcpyHostToDevice, g_nf_stream));
  }
  L0->pre_x = nullptr;
  L0->pre_l = nullptr;
  if (next_xh) {  // the other buffer is free: the step that read it has been waited for before its call returned
    const int nb = L0->stage_cur ^ 1;
    NF_CUDA(cudaMemcpyAsync(L0->stage_xb[nb], next_xh, xbytes, cudaMemcpyHostToDevice, g_copy_stream));
    NF_CUDA(cudaMemcpyAsync(L0->stage_lb[nb], next_lh, N * 4, cudaMemcpyHostToDevice, g_copy_stream));
    NF_CUDA(cudaEventRecord(g_copy_done, g_copy_stream));
    L0->pre_x = next_xh;
    L0->pre_l = next_lh;
  }
  NF_TRY(nf_block_step(B, L0->stage_xb[L0->stage_cur], L0->stage_lb[L0->stage_cur], lr, L0->stage_loss, nullptr));
  NF_CUDA(cudaMemcpyAsync(loss_h, L0->stage_loss, 4 * (size_t)B->n, cudaMemcpyDeviceToHost, g_nf_stream));
  if (act_h)
    NF_CUDA(cudaMemcpyAsync(act_h, Ll->act, N * Ll->Ha * Ll->Wa * Ll->Cout * es, cudaMemcpyDeviceToHost, g_nf_stream));
  NF_CUDA(cudaStreamSynchronize(g_nf_stream));
  return NF_OK;
}

int nf_cache_gather(const void* cache, const int32_t* cache_labels, int cache_rows, const int32_t* idx, int count,
                    size_t row_bytes, void* out, int32_t* out_labels) {
  if (!cache || !idx || !out || cache_rows < 1 || count < 1 || row_bytes == 0 || (row_bytes & 15)) return NF_EINVAL;
  if ((cache_labels == nullptr) != (out_labels == nullptr)) return NF_EINVAL;
  if (misaligned(cache) || misaligned(out)) return NF_EALIGN;
  int32_t* st = nullptr;
  NF_TRY(nf_tc_op_status_ptr(&st));
  return nf_k_gather(cache, cache_labels, cache_rows, idx, count, row_bytes, out, out_labels, st);
}

static bool conv_args_ok(int dtype, int N, int H, int W, int Cin, int Cout, int stride) {
  return (dtype == NF_F32 || dtype == NF_BF16) && N >= 1 && H >= 1 && W >= 1 && Cin >= 1 && Cout >= 1 &&
         (stride == 1 || stride == 2);
}

int nf_conv3x3_forward(int dtype, const void* x, const void* w, int N, int H, int W, int Cin, int Cout, int stride,
                       void* y) {
  if (!x || !w || !y || !conv_args_ok(dtype, N, H, W, Cin, Cout, stride)) return NF_EINVAL;
  if (misaligned(x) || misaligned(w) || misaligned(y)) return NF_EALIGN;
  if (dtype == NF_BF16) {
    const int rc = nf_tc_conv3x3_forward(x, w, N, H, W, Cin, Cout, stride, y);
    if (rc != NF_EUNSUPPORTED) return rc;
  }
  return nf_k_conv(dtype, x, N, H, W, Cin, w, (long)Cout * Cin, Cin, 1, 0, nullptr, 0, stride, Cout, y);
}

size_t nf_conv3x3_wgrad_scratch_bytes(int N, int H, int W, int Cin, int Cout, int stride) {
  if (!conv_args_ok(NF_F32, N, H, W, Cin, Cout, stride)) return 0;
  const int Ho = (H - 1) / stride + 1;
  size_t fl = (size_t)nf_k_wgrad_splits(N, Ho, Cin, Cout) * 9 * Cout * Cin;
  const size_t tc = nf_tc_conv3x3_wgrad_scratch_floats(N, H, W, Cin, Cout, stride);
  if (tc > fl) fl = tc;
  return fl * sizeof(float);
}

int nf_conv3x3_wgrad(int dtype, const void* x, const void* g, int N, int H, int W, int Cin, int Cout, int stride,
                     void* scratch, size_t scratch_bytes, float* dw) {
  if (!x || !g || !scratch || !dw || !conv_args_ok(dtype, N, H, W, Cin, Cout, stride)) return NF_EINVAL;
  if (misaligned(x) || misaligned(g) || misaligned(scratch) || misaligned(dw)) return NF_EALIGN;
  if (dtype == NF_BF16) {
    const int rc = nf_tc_conv3x3_wgrad(x, g, N, H, W, Cin, Cout, stride, (float*)scratch, scratch_bytes / sizeof(float), dw);
    if (rc != NF_EUNSUPPORTED) return rc;
  }
  return nf_k_wgrad(dtype, x, N, H, W, Cin, g, Cout, stride, (float*)scratch, scratch_bytes / sizeof(float), dw);
}

int nf_op_status(void) {
  int32_t v = 0;
  const int rc = nf_tc_op_status(&v);
  return rc == NF_OK ? (int)v : rc;
}

int nf_selftest_bounded_wait(unsigned long long limit_ns, unsigned long long* waited_ns_dev) {
  if (!waited_ns_dev || limit_ns == 0 || limit_ns > 1000000000ull) return NF_EINVAL;  // at most one second
  if ((uintptr_t)waited_ns_dev & 7) return NF_EALIGN;
  return nf_tc_bounded_wait_probe(limit_ns, waited_ns_dev);
}

// Algorithm 1, second part.  One pass over the layers: a block stays open while the capped batch size of the next layer
// is within rho (relative to the current layer's) of the current one; the block's batch size is the running minimum of
// its members.
int nf_partition(const int* max_batch, int n_layers, int Bcap, double rho, int* block_first, int* block_batch) {
  if (!max_batch || !block_first || !block_batch || n_layers < 1 || Bcap < 1 || !(rho >= 0.0)) return NF_EINVAL;
  for (int i = 0; i < n_layers; ++i)
    if (max_batch[i] < 1) return NF_EINVAL;
  auto capped = [&](int i) { return std::min(max_batch[i], Bcap); };
  int nblocks = 0;
  for (int i = 0; i < n_layers; ++i) {
    const int b = capped(i);
    const bool joins = i > 0 && fabs((double)b - (double)capped(i - 1)) <= rho * (double)capped(i - 1);
    if (joins) {
      block_batch[nblocks - 1] = std::min(block_batch[nblocks - 1], b);
    } else {
      block_first[nblocks] = i;
      block_batch[nblocks++] = b;
    }
  }
  return nblocks;
}

int nf_aan_filters(const int* channels, int n_layers, int first_downsample, int* filters_out) {
  if (!channels || !filters_out || n_layers < 1 || first_downsample < 0) return NF_EINVAL;
  int lo = channels[0], hi = channels[0];
  for (int i = 0; i < n_layers; ++i) {
    if (channels[i] < 1) return NF_EINVAL;
    if (channels[i] < lo) lo = channels[i];
    if (channels[i] > hi) hi = channels[i];
  }
  for (int i = 0; i < n_layers; ++i) {
    const int f = (i < first_downsample ? lo : hi) / 2;
    filters_out[i] = f < 1 ? 1 : f;
  }
  return NF_OK;
}

int nf_fit_line(const double* batches, const double* bytes, int k, double* slope, double* intercept) {
  if (!batches || !bytes || !slope || !intercept || k < 2) return NF_EINVAL;
  double sx = 0, sy = 0, sxx = 0, sxy = 0;
  for (int i = 0; i < k; ++i) {
    sx += batches[i]; sy += bytes[i]; sxx += batches[i] * batches[i]; sxy += batches[i] * bytes[i];
  }
  const double den = k * sxx - sx * sx;
  if (!(den > 0.0)) return NF_EINVAL;  // all batch sizes equal
  *slope = (k * sxy - sx * sy) / den;
  *intercept = (sy - *slope * sx) / k;
  return NF_OK;
}

int nf_profile_layer(int Cin, int Cout, int H, int W, int F, int classes, const nf_layer_opts* opts, const int* batches, int k,
                     double* bytes_out, double* slope, double* intercept) {
  if (!opts || !batches || !slope || !intercept || k < 2) return NF_EINVAL;
  nf_layer* L = nf_layer_create(Cin, Cout, H, W, F, classes);
  if (!L) return NF_EINVAL;
  std::vector<double> xs(k), ys(k);
  for (int i = 0; i < k; ++i) {
    nf_layer_opts o = *opts;
    o.N = batches[i];
    const int rc = nf_layer_configure(L, &o);
    if (rc != NF_OK) {
      nf_layer_destroy(L);
      return rc;
    }
    xs[i] = (double)o.N;
    ys[i] = (double)nf_layer_workspace_bytes(L) + (double)o.N * H * W * Cin * (double)nf_esize(o.dtype);
    if (bytes_out) bytes_out[i] = ys[i];
  }
  nf_layer_destroy(L);
  return nf_fit_line(xs.data(), ys.data(), k, slope, intercept);
}

long long nf_max_batch(double slope, double intercept, double budget_bytes) {
  if (!(slope > 0.0)) return NF_EINVAL;
  const double t = floor((budget_bytes - intercept) / slope + 1e-12);
  return t < 0.0 ? 0 : (long long)t;
}

int nf_set_stream(void* s) {
  g_nf_stream = (cudaStream_t)s;
  return NF_OK;
}

long long nf_launch_count(void) { return g_nf_launches; }

const char* nf_layer_kernel_family(const nf_layer* L, int op) {
  if (!L || op < 0 || op > 6) return "";
  if (op == 4) return nf_tc_bn_aux_fused(L) && !L->skip ? "fused" : "separate";
  if (op == 5) return nf_tc_bn_aux_fused(L) && !L->skip && nf_tc_aux_pool_fused(L) ? "mask" : "stored";
  if (op == 6) return nf_tc_dgrad_two_pass(L) && !L->skip && !L->skip_grad ? "two-pass" : "stored";
  return L->fam[op] ? "tcgen05" : "cuda-core";
}

const char* nf_strerror(int st) {
  switch (st) {
    case NF_OK: return "ok";
    case NF_EINVAL: return "invalid argument";
    case NF_EALIGN: return "misaligned device pointer";
    case NF_ENOWS: return "workspace missing or too small";
    case NF_EUNSUPPORTED: return "unsupported shape";
    case NF_ECUDA: return "CUDA runtime error";
    default: return "unknown status";
  }
}

const char* nf_last_cuda_error(void) { return g_nf_err; }

}  // extern "C"
