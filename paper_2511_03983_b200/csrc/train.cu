// twist_subnet_ffn_fwd/bwd and twist_subnet_attn_proj_fwd/bwd: the local training step of the
// S subnets on their dense slices (FFN of App. A: y = C act(W x); projections of the multi-head
// attention definition).  bf16: grouped tcgen05 GEMMs with fused epilogues.  fp32: plain SIMT
// kernels (tiny correctness workload only).
#include <math.h>

#include <initializer_list>

#include "gemm_sm100.cuh"
#include "glue.cuh"
#include "plan.cuh"

namespace twist {
namespace {

#define TWIST_TRY(expr)               \
  do {                                \
    int rc__ = (expr);                \
    if (rc__ != TWIST_OK) return rc__;\
  } while (0)

// The kernels touch these arrays with 16-byte (the byte mask: 8-byte) vector accesses; a pointer that breaks the
// rule is refused here instead of faulting on the device.  NULL passes (absence is checked where it matters).
bool all_aligned16(std::initializer_list<const void*> ptrs) {
  for (const void* p : ptrs)
    if (!aligned16(p)) return false;
  return true;
}
bool aligned8(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 7u) == 0; }

int check_ffn(const twist_ffn_args* a) {
  if (!a) return TWIST_ERR_NULL;
  if (a->n_subnets <= 0 || a->tokens <= 0 || a->d_model <= 0 || a->f_sub <= 0) return TWIST_ERR_SHAPE;
  if (a->ffn_kind < TWIST_FFN_RELU || a->ffn_kind > TWIST_FFN_SWIGLU) return TWIST_ERR_SHAPE;
  if (a->dtype != TWIST_FP32 && a->dtype != TWIST_BF16) return TWIST_ERR_SHAPE;
  if (a->dtype == TWIST_BF16 && (a->d_model % 8 || a->f_sub % 8)) return TWIST_ERR_SHAPE;
  if (!all_aligned16({a->x, a->w_gu, a->w_down, a->w_gu_master, a->w_down_master, a->pre, a->hh, a->y, a->dy, a->dpre,
                      a->dx, a->dw_gu, a->dw_down, a->tgt, a->loss_ws, a->y_residual, a->dx_residual, a->m_gu, a->v_gu,
                      a->m_down, a->v_down}) || !aligned8(a->hidden_mask))
    return TWIST_ERR_SHAPE;
  return TWIST_OK;
}

// Checks the fused-loss arguments of a forward call; *fused tells whether the loss is requested.
int check_fused(const void* tgt, float* loss, const void* dgrad, void* ws, size_t ws_bytes, int S, int T, int width,
                const int32_t* valid_cols, int seg_begin, int seg_width, bool* fused) {
  *fused = tgt != nullptr;
  if (!*fused) return TWIST_OK;
  if (!loss || !dgrad) return TWIST_ERR_NULL;
  if (!ws || ws_bytes < twist_fused_loss_workspace_bytes(S, T, width)) return TWIST_ERR_WORKSPACE;
  if (valid_cols && (seg_begin < 0 || seg_begin >= width || seg_width <= 0 || (width - seg_begin) % seg_width != 0 ||
                     seg_begin % 8 != 0 || seg_width % 8 != 0))
    return TWIST_ERR_SHAPE;
  return TWIST_OK;
}

// Output GEMM of a forward call with the loss fused into its epilogue (bf16).
int launch_fused_loss(int layout, const GemmOperand& A, const GemmOperand& B, GemmParams p, void* out, const void* tgt,
                      void* dgrad, float* loss, void* ws, const int32_t* valid_cols, int seg_begin, int seg_width,
                      cudaStream_t st, const uint8_t* col_mask = nullptr) {
  p.col_mask = col_mask;
  p.out0 = static_cast<__nv_bfloat16*>(out);
  p.out1 = static_cast<__nv_bfloat16*>(dgrad);
  p.in0 = static_cast<const __nv_bfloat16*>(tgt);
  p.dw = static_cast<float*>(ws);
  p.valid_cols = valid_cols;
  p.seg_begin = valid_cols ? seg_begin : 0;
  p.seg_width = valid_cols ? seg_width : p.N;
  // the last CTA of the launch reduces the partial sums itself; a separate (tiny) launch does it where no per-stream
  // counter is to be had
  p.loss_out = loss;
  p.done_ctr = fused_loss_counter(st);
  TWIST_TRY(launch_gemm_bf16(layout, out ? EPI_MSE : EPI_MSE_NOY, A, B, p, st));
  if (p.done_ctr) return TWIST_OK;
  return finish_fused_loss(p.dw, p.groups, p.M, p.N, valid_cols, p.seg_begin, p.seg_width, loss, st);
}

// Fills the optimiser part of a weight-gradient launch; returns the epilogue to use or a negative status.
int optimizer_epilogue(const twist_optimizer& o, float lr, float* m, float* v, GemmParams* p) {
  if (o.kind == TWIST_OPT_SGD) return EPI_SGD;
  if (o.kind != TWIST_OPT_ADAM) return TWIST_ERR_SHAPE;
  if (lr == 0.f) return EPI_SGD;                                   // nothing to update: plain gradient launch
  if (!m || !v) return TWIST_ERR_NULL;
  if (o.step < 1 || !(o.beta1 >= 0.f && o.beta1 < 1.f) || !(o.beta2 >= 0.f && o.beta2 < 1.f) || !(o.eps >= 0.f))
    return TWIST_ERR_SHAPE;
  p->adam_m = m; p->adam_v = v;
  p->beta1 = o.beta1; p->beta2 = o.beta2; p->adam_eps = o.eps;
  p->bias1 = (float)(1.0 / (1.0 - pow((double)o.beta1, (double)o.step)));
  p->bias2 = (float)(1.0 / (1.0 - pow((double)o.beta2, (double)o.step)));
  return EPI_ADAM;
}

GemmParams base_params(int M, int N, int K, int groups, float scale) {
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.M = M; p.N = N; p.K = K; p.groups = groups; p.scale = scale;
  return p;
}

}  // namespace
}  // namespace twist

using namespace twist;

extern "C" size_t twist_fused_loss_workspace_bytes(int32_t n_subnets, int32_t tokens, int32_t width) {
  if (n_subnets <= 0 || tokens <= 0 || width <= 0) return 0;
  const size_t a = fused_loss_partials(n_subnets, tokens, width) * sizeof(float);
  const size_t b = twist_mse_workspace_bytes(n_subnets);      // the fp32 dtype runs the stand-alone loss kernels
  return a > b ? a : b;
}

extern "C" int32_t twist_subnet_ffn_fwd(const twist_ffn_args* a, void* stream) {
  TWIST_TRY(check_ffn(a));
  PlanScope scope(a->plan);
  bool fused = false;
  TWIST_TRY(check_fused(a->tgt, a->loss, a->dy, a->loss_ws, a->loss_ws_bytes, a->n_subnets, a->tokens, a->d_model,
                        nullptr, 0, 0, &fused));
  if (!a->x || !a->w_gu || !a->w_down || !a->pre || !a->hh || (!a->y && !fused)) return TWIST_ERR_NULL;
  if (a->dtype == TWIST_FP32 && !a->y) return TWIST_ERR_NULL;
  if (a->y_residual && (fused || a->dtype == TWIST_FP32)) return TWIST_ERR_UNSUPPORTED;
  if (a->hidden_mask && a->dtype == TWIST_FP32) return TWIST_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int S = a->n_subnets, T = a->tokens, d = a->d_model, f = a->f_sub;
  const bool swiglu = a->ffn_kind == TWIST_FFN_SWIGLU;
  const int gf = swiglu ? 2 * f : f;
  if (a->dtype == TWIST_FP32) {
    const float* x = static_cast<const float*>(a->x);
    float* pre = static_cast<float*>(a->pre);
    float* hh = static_cast<float*>(a->hh);
    TWIST_TRY(sgemm_f32(false, true, x, static_cast<const float*>(a->w_gu), pre, T, gf, d, d, d, gf, (long long)T * d,
                        (long long)gf * d, (long long)T * gf, S, 1.f, st));
    TWIST_TRY(act_fwd_f32(pre, hh, (long long)S * T, f, a->ffn_kind, st));
    TWIST_TRY(sgemm_f32(false, false, hh, static_cast<const float*>(a->w_down), static_cast<float*>(a->y), T, d, f, f, d,
                        d, (long long)T * f, (long long)f * d, (long long)T * d, S, a->out_scale, st));
    if (!fused) return TWIST_OK;
    return twist_mse_fwd_bwd(a->y, a->tgt, const_cast<void*>(a->dy), a->loss, S, T, d, nullptr, 0, 0, TWIST_FP32,
                             a->loss_ws, a->loss_ws_bytes, stream);
  }
  // pre (and hh) = epilogue(X W_gu^T)
  GemmParams p = base_params(T, f, d, S, 1.f);
  p.out0 = static_cast<__nv_bfloat16*>(a->pre);
  p.out1 = static_cast<__nv_bfloat16*>(a->hh);
  p.b_split = f;
  p.act_kind = a->ffn_kind;
  p.hmask = a->hidden_mask;
  TWIST_TRY(launch_gemm_bf16(0, swiglu ? EPI_SWIGLU_FWD : EPI_ACT_FWD, GemmOperand{a->x, T, d},
                             GemmOperand{a->w_gu, gf, d}, p, st));
  // Y = out_scale * hh W_down  (+ loss and dY in the same epilogue when requested)
  GemmParams q = base_params(T, d, f, S, a->out_scale);
  if (fused)
    return launch_fused_loss(1, GemmOperand{a->hh, T, f}, GemmOperand{a->w_down, f, d}, q, a->y, a->tgt,
                             const_cast<void*>(a->dy), a->loss, a->loss_ws, nullptr, 0, 0, st);
  q.out0 = static_cast<__nv_bfloat16*>(a->y);
  q.in0 = static_cast<const __nv_bfloat16*>(a->y_residual);
  return launch_gemm_bf16(1, a->y_residual ? EPI_RESID : EPI_STORE, GemmOperand{a->hh, T, f}, GemmOperand{a->w_down, f, d},
                          q, st);
}

extern "C" int32_t twist_subnet_ffn_bwd(const twist_ffn_args* a, void* stream) {
  TWIST_TRY(check_ffn(a));
  PlanScope scope(a->plan);
  if (!a->x || !a->w_gu || !a->w_down || !a->pre || !a->hh || !a->dy || !a->dpre) return TWIST_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int S = a->n_subnets, T = a->tokens, d = a->d_model, f = a->f_sub;
  const bool swiglu = a->ffn_kind == TWIST_FFN_SWIGLU;
  const int gf = swiglu ? 2 * f : f;
  if (a->dtype == TWIST_FP32) {
    if (!a->dw_gu || !a->dw_down) return TWIST_ERR_NULL;
    if (a->dx_residual || a->opt.kind != TWIST_OPT_SGD || a->hidden_mask) return TWIST_ERR_UNSUPPORTED;
    const float* x = static_cast<const float*>(a->x);
    const float* dy = static_cast<const float*>(a->dy);
    const float* pre = static_cast<const float*>(a->pre);
    const float* hh = static_cast<const float*>(a->hh);
    float* dpre = static_cast<float*>(a->dpre);
    float* wgu = static_cast<float*>(a->w_gu);
    float* wd = static_cast<float*>(a->w_down);
    // dHh = out_scale * dY W_down^T, parked in dpre (SwiGLU: in the "up" half), then through the activation in place
    TWIST_TRY(sgemm_f32(false, true, dy, wd, dpre + (swiglu ? f : 0), T, f, d, d, d, gf, (long long)T * d,
                        (long long)f * d, (long long)T * gf, S, a->out_scale, st));
    TWIST_TRY(act_bwd_f32(pre, dpre, (long long)S * T, f, a->ffn_kind, st));
    if (a->dx)
      TWIST_TRY(sgemm_f32(false, false, dpre, wgu, static_cast<float*>(a->dx), T, d, gf, gf, d, d, (long long)T * gf,
                          (long long)gf * d, (long long)T * d, S, 1.f, st));
    TWIST_TRY(sgemm_f32(true, false, dpre, x, a->dw_gu, gf, d, T, gf, d, d, (long long)T * gf, (long long)T * d,
                        (long long)gf * d, S, 1.f, st));
    TWIST_TRY(sgemm_f32(true, false, hh, dy, a->dw_down, f, d, T, f, d, d, (long long)T * f, (long long)T * d,
                        (long long)f * d, S, a->out_scale, st));
    if (a->lr != 0.f) {
      TWIST_TRY(sgd_f32(wgu, a->dw_gu, a->lr, (long long)S * gf * d, st));
      TWIST_TRY(sgd_f32(wd, a->dw_down, a->lr, (long long)S * f * d, st));
    }
    return TWIST_OK;
  }
  if ((a->lr != 0.f || a->master_from_slice) && (!a->w_gu_master || !a->w_down_master)) return TWIST_ERR_NULL;
  if (a->dx_residual && !a->dx) return TWIST_ERR_NULL;
  // dpre = act'(pre) * (out_scale * dY W_down^T)
  GemmParams p = base_params(T, f, d, S, a->out_scale);
  p.out0 = static_cast<__nv_bfloat16*>(a->dpre);
  p.in0 = static_cast<const __nv_bfloat16*>(a->pre);
  p.act_kind = a->ffn_kind;
  p.hmask = a->hidden_mask;
  TWIST_TRY(launch_gemm_bf16(0, swiglu ? EPI_DSWIGLU : EPI_DACT, GemmOperand{a->dy, T, d}, GemmOperand{a->w_down, f, d},
                             p, st));
  // dX = dpre W_gu   (before the weights are updated)
  if (a->dx) {
    GemmParams q = base_params(T, d, gf, S, 1.f);
    q.out0 = static_cast<__nv_bfloat16*>(a->dx);
    q.in0 = static_cast<const __nv_bfloat16*>(a->dx_residual);
    TWIST_TRY(launch_gemm_bf16(1, a->dx_residual ? EPI_RESID : EPI_STORE, GemmOperand{a->dpre, T, gf},
                               GemmOperand{a->w_gu, gf, d}, q, st));
  }
  // dW_down = out_scale * hh^T dY, fused SGD
  GemmParams r = base_params(f, d, T, S, a->out_scale);
  r.out0 = static_cast<__nv_bfloat16*>(a->w_down);
  r.master = a->w_down_master;
  r.dw = a->dw_down;
  r.lr = a->lr;
  r.master_init = a->master_from_slice;
  int epi = optimizer_epilogue(a->opt, a->lr, a->m_down, a->v_down, &r);
  if (epi < 0) return epi;
  TWIST_TRY(launch_gemm_bf16(2, epi, GemmOperand{a->hh, T, f}, GemmOperand{a->dy, T, d}, r, st));
  // dW_gu = dpre^T X, fused SGD
  GemmParams u = base_params(gf, d, T, S, 1.f);
  u.out0 = static_cast<__nv_bfloat16*>(a->w_gu);
  u.master = a->w_gu_master;
  u.dw = a->dw_gu;
  u.lr = a->lr;
  u.master_init = a->master_from_slice;
  epi = optimizer_epilogue(a->opt, a->lr, a->m_gu, a->v_gu, &u);
  if (epi < 0) return epi;
  return launch_gemm_bf16(2, epi, GemmOperand{a->dpre, T, gf}, GemmOperand{a->x, T, d}, u, st);
}

static int check_proj(const twist_proj_args* a) {
  if (!a) return TWIST_ERR_NULL;
  if (a->n_subnets <= 0 || a->tokens <= 0 || a->d_model <= 0 || a->n <= 0) return TWIST_ERR_SHAPE;
  if (a->which != TWIST_PROJ_QKV && a->which != TWIST_PROJ_O) return TWIST_ERR_SHAPE;
  if (a->dtype != TWIST_FP32 && a->dtype != TWIST_BF16) return TWIST_ERR_SHAPE;
  if (a->dtype == TWIST_BF16 && (a->d_model % 8 || a->n % 8)) return TWIST_ERR_SHAPE;
  if (!all_aligned16({a->in, a->w, a->w_master, a->out, a->d_out, a->d_in, a->dw, a->tgt, a->loss_ws, a->out_residual,
                      a->d_in_residual, a->m, a->v}) || !aligned8(a->col_mask))
    return TWIST_ERR_SHAPE;
  if (a->col_mask && a->dtype != TWIST_BF16) return TWIST_ERR_UNSUPPORTED;
  return TWIST_OK;
}

extern "C" int32_t twist_subnet_attn_proj_fwd(const twist_proj_args* a, void* stream) {
  TWIST_TRY(check_proj(a));
  PlanScope scope(a->plan);
  const int S = a->n_subnets, T = a->tokens, d = a->d_model, n = a->n;
  const bool qkv = a->which == TWIST_PROJ_QKV;
  const int w_out = qkv ? n : d;      // width of the output
  bool fused = false;
  // An arbitrary column set for the loss (col_mask, with valid_cols[s] = its size) is a one-group prefix rule
  // as far as the normaliser goes.
  const bool by_mask = qkv && a->col_mask != nullptr && a->tgt != nullptr;      // (TWIST_PROJ_O: the mask acts in bwd)
  const int seg_begin = by_mask ? 0 : a->seg_begin, seg_width = by_mask ? w_out : a->seg_width;
  if (by_mask && (!a->valid_cols || a->dtype != TWIST_BF16)) return a->valid_cols ? TWIST_ERR_UNSUPPORTED : TWIST_ERR_NULL;
  TWIST_TRY(check_fused(a->tgt, a->loss, a->d_out, a->loss_ws, a->loss_ws_bytes, S, T, w_out, a->valid_cols,
                        seg_begin, seg_width, &fused));
  if (!a->in || !a->w || (!a->out && !fused)) return TWIST_ERR_NULL;
  if (a->out_residual && (fused || qkv || a->dtype == TWIST_FP32)) return TWIST_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (a->dtype == TWIST_FP32) {
    if (!a->out) return TWIST_ERR_NULL;
    const float* in = static_cast<const float*>(a->in);
    const float* w = static_cast<const float*>(a->w);
    float* out = static_cast<float*>(a->out);
    if (qkv)
      TWIST_TRY(sgemm_f32(false, true, in, w, out, T, n, d, d, d, n, (long long)T * d, (long long)n * d,
                          (long long)T * n, S, a->out_scale, st));
    else
      TWIST_TRY(sgemm_f32(false, false, in, w, out, T, d, n, n, d, d, (long long)T * n, (long long)n * d,
                          (long long)T * d, S, a->out_scale, st));
    if (!fused) return TWIST_OK;
    return twist_mse_fwd_bwd(out, a->tgt, const_cast<void*>(a->d_out), a->loss, S, T, w_out, a->valid_cols,
                             a->seg_begin, a->seg_width, TWIST_FP32, a->loss_ws, a->loss_ws_bytes, stream);
  }
  const GemmOperand A{a->in, T, qkv ? d : n}, W{a->w, n, d};
  GemmParams p = qkv ? base_params(T, n, d, S, a->out_scale) : base_params(T, d, n, S, a->out_scale);
  const int layout = qkv ? 0 : 1;
  if (fused)
    return launch_fused_loss(layout, A, W, p, a->out, a->tgt, const_cast<void*>(a->d_out), a->loss, a->loss_ws,
                             a->valid_cols, seg_begin, seg_width, st, by_mask ? a->col_mask : nullptr);
  p.out0 = static_cast<__nv_bfloat16*>(a->out);
  p.in0 = static_cast<const __nv_bfloat16*>(a->out_residual);
  return launch_gemm_bf16(layout, a->out_residual ? EPI_RESID : EPI_STORE, A, W, p, st);
}

extern "C" int32_t twist_subnet_attn_proj_bwd(const twist_proj_args* a, void* stream) {
  TWIST_TRY(check_proj(a));
  PlanScope scope(a->plan);
  if (!a->in || !a->w || !a->d_out) return TWIST_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int S = a->n_subnets, T = a->tokens, d = a->d_model, n = a->n;
  const bool qkv = a->which == TWIST_PROJ_QKV;
  const int w_in = qkv ? d : n;       // width of `in`
  const int w_out = qkv ? n : d;      // width of `d_out`
  if (a->dtype == TWIST_FP32) {
    if (!a->dw) return TWIST_ERR_NULL;
    if (a->d_in_residual || a->opt.kind != TWIST_OPT_SGD) return TWIST_ERR_UNSUPPORTED;
    const float* in = static_cast<const float*>(a->in);
    const float* dout = static_cast<const float*>(a->d_out);
    float* w = static_cast<float*>(a->w);
    if (a->d_in) {
      if (qkv)   // dX = dQKV W
        TWIST_TRY(sgemm_f32(false, false, dout, w, static_cast<float*>(a->d_in), T, d, n, n, d, d, (long long)T * n,
                            (long long)n * d, (long long)T * d, S, a->out_scale, st));
      else       // dA = out_scale * dY W^T
        TWIST_TRY(sgemm_f32(false, true, dout, w, static_cast<float*>(a->d_in), T, n, d, d, d, n, (long long)T * d,
                            (long long)n * d, (long long)T * n, S, a->out_scale, st));
    }
    if (qkv)     // dW [n][d] = dQKV^T X
      TWIST_TRY(sgemm_f32(true, false, dout, in, a->dw, n, d, T, n, d, d, (long long)T * n, (long long)T * d,
                          (long long)n * d, S, a->out_scale, st));
    else         // dW [n][d] = out_scale * A^T dY
      TWIST_TRY(sgemm_f32(true, false, in, dout, a->dw, n, d, T, n, d, d, (long long)T * n, (long long)T * d,
                          (long long)n * d, S, a->out_scale, st));
    if (a->lr != 0.f) TWIST_TRY(sgd_f32(w, a->dw, a->lr, (long long)S * n * d, st));
    return TWIST_OK;
  }
  if ((a->lr != 0.f || a->master_from_slice) && !a->w_master) return TWIST_ERR_NULL;
  if (a->d_in_residual && (!qkv || !a->d_in)) return TWIST_ERR_UNSUPPORTED;
  if (a->d_in) {
    if (qkv) {
      GemmParams p = base_params(T, d, n, S, a->out_scale);
      p.out0 = static_cast<__nv_bfloat16*>(a->d_in);
      p.in0 = static_cast<const __nv_bfloat16*>(a->d_in_residual);
      TWIST_TRY(launch_gemm_bf16(1, a->d_in_residual ? EPI_RESID : EPI_STORE, GemmOperand{a->d_out, T, n},
                                 GemmOperand{a->w, n, d}, p, st));
    } else {
      GemmParams p = base_params(T, n, d, S, a->out_scale);
      p.out0 = static_cast<__nv_bfloat16*>(a->d_in);
      p.hmask = a->col_mask;             // a masked worker: no gradient flows into the heads it does not hold
      TWIST_TRY(launch_gemm_bf16(0, EPI_STORE, GemmOperand{a->d_out, T, d}, GemmOperand{a->w, n, d}, p, st));
    }
  }
  GemmParams r = base_params(n, d, T, S, a->out_scale);
  r.out0 = static_cast<__nv_bfloat16*>(a->w);
  r.master = a->w_master;
  r.dw = a->dw;
  r.lr = a->lr;
  r.master_init = a->master_from_slice;
  const int epi = optimizer_epilogue(a->opt, a->lr, a->m, a->v, &r);
  if (epi < 0) return epi;
  if (qkv) return launch_gemm_bf16(2, epi, GemmOperand{a->d_out, T, w_out}, GemmOperand{a->in, T, w_in}, r, st);
  return launch_gemm_bf16(2, epi, GemmOperand{a->in, T, w_in}, GemmOperand{a->d_out, T, w_out}, r, st);
}
