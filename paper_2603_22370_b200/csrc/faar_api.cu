// extern "C" entry points of libfaar.so: argument validation, workspace carving,
// kernel sequencing.  No device memory is allocated here.
#include <math.h>
#include <initializer_list>
#include <new>

#include "faar_internal.cuh"

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int cuda_fail(faar_ctx* ctx, int e) {
  if (e == 0) return FAAR_OK;
  ctx->last_cuda_error = e;
  return FAAR_ERR_CUDA;
}

// Largest temperature the GEMM calls take: the BF16 operand's FP32 evaluation has a relative error of about
// 6e-7 + 7.5e-8 beta, which at 1024 is still 25 times below the BF16 spacing.
constexpr float FAAR_BETA_MAX = 1024.0f;

int check_shape(const faar_shape* s) {
  if (!s) return FAAR_ERR_INVALID_ARG;
  if (s->O <= 0 || s->K <= 0 || s->T <= 0) return FAAR_ERR_SHAPE;
  if (s->K % 16 != 0) return FAAR_ERR_SHAPE;
  return FAAR_OK;
}

// The backward epilogue forms offsets of up to 7 rows of V in 32-bit element counts.
int check_bwd_k(const faar_shape* s) { return (long long)s->K * 8 > 0x7FFFFFFFll ? FAAR_ERR_SHAPE : FAAR_OK; }

// Chained steps: wsoft_ready is only honoured if the last backward call on this context wrote, into this
// very workspace, the operand for this step's beta.
int check_chain(const faar_ctx* ctx, const faar_hparams* hp, const void* ws) {
  if (!hp->wsoft_ready) return FAAR_OK;
  return (ctx->wsoft_ws == ws && ctx->wsoft_beta == hp->beta) ? FAAR_OK : FAAR_ERR_INVALID_ARG;
}

// Leading dimension of Y_ref / Y_q for the layout the shape declares.
int check_ldy(const faar_shape* s) {
  if (s->yref_transposed) {
    if (s->ldy < ((int64_t)s->T + 15) / 16 * 16) return FAAR_ERR_SHAPE;
    if (s->ldy % 8) return FAAR_ERR_ALIGN;
    return FAAR_OK;
  }
  return s->ldy < s->O ? FAAR_ERR_SHAPE : FAAR_OK;
}

int check_ws(const faar_shape* s, const void* ws, size_t ws_bytes) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return FAAR_ERR_WORKSPACE;
  if (ws_bytes < faar_ws_plan(s).total) return FAAR_ERR_WORKSPACE;
  return FAAR_OK;
}

int check_hp(const faar_hparams* hp, bool need_opt) {
  if (!hp) return FAAR_ERR_INVALID_ARG;
  if (!(hp->beta > 0.f) || !(hp->beta <= FAAR_BETA_MAX) || !isfinite(hp->mse_scale) || !isfinite(hp->lambda_round))
    return FAAR_ERR_INVALID_ARG;
  if (!(hp->act_scale >= 0.f) || !isfinite(hp->act_scale)) return FAAR_ERR_INVALID_ARG;
  if (!(hp->beta_next >= 0.f) || !(hp->beta_next <= FAAR_BETA_MAX)) return FAAR_ERR_INVALID_ARG;
  if (need_opt) {
    if (hp->opt != 0 && hp->opt != 1) return FAAR_ERR_INVALID_ARG;
    if (!isfinite(hp->lr)) return FAAR_ERR_INVALID_ARG;
    if (hp->opt == 1 && (hp->step < 1 || !(hp->beta1 >= 0.f && hp->beta1 < 1.f) ||
                         !(hp->beta2 >= 0.f && hp->beta2 < 1.f) || !(hp->eps >= 0.f)))
      return FAAR_ERR_INVALID_ARG;
  }
  return FAAR_OK;
}

// Makes the context's device current for the duration of a call.  err != 0: the switch failed and
// nothing may be launched.
struct DeviceGuard {
  int prev = -1;
  int err = 0;
  explicit DeviceGuard(int dev) {
    cudaError_t e = cudaGetDevice(&prev);
    if (e == cudaSuccess && prev != dev) e = cudaSetDevice(dev); else if (e == cudaSuccess) prev = -1;
    if (e != cudaSuccess) { err = (int)e; prev = -1; }
  }
  ~DeviceGuard() { if (prev >= 0) (void)cudaSetDevice(prev); }
};
#define FAAR_DEVICE_GUARD(ctx)                  \
  DeviceGuard device_guard_((ctx)->device);     \
  if (device_guard_.err) return cuda_fail((ctx), device_guard_.err)

int fwd_impl(faar_ctx* ctx, const faar_shape* s, const faar_hparams* hp, const void* X, const void* Y_ref,
             const float* V, const uint8_t* code, const uint8_t* scales, const float* s_global, void* dYt,
             void* Y_q, uint8_t* ws, const faar_ws_layout& l, int* n_partials) {
  __nv_bfloat16* wsoft = reinterpret_cast<__nv_bfloat16*>(ws + l.off_wsoft);
  int e = 0;
  if (!hp->wsoft_ready) {   // else: the previous backward pass left this step's operand in the workspace
    e = faar_launch_softquant_eval(ctx, s, V, code, scales, s_global, hp->beta, nullptr, nullptr, wsoft);
    if (e) return e;
  }
  faar_gemm_args a = {};
  a.mode = FAAR_GEMM_FWD;
  a.M = s->O; a.N = s->T; a.Kc = s->K;
  a.A = wsoft; a.lda = s->K;
  a.B = X; a.ldb = s->ldx;
  a.status = reinterpret_cast<uint32_t*>(ws);
  a.Yout = Y_q; a.yout_dtype = FAAR_BF16; a.ldy = s->ldy;
  a.Yref = Y_ref; a.yref_dtype = s->yref_dtype; a.yref_t = s->yref_transposed;
  a.dYt = reinterpret_cast<__nv_bfloat16*>(dYt); a.ld_dyt = l.ld_dyt;
  a.mse2c = 2.0f * hp->mse_scale;
  a.act_scale = hp->act_scale > 0.f ? hp->act_scale : 1.0f;
  a.partials = reinterpret_cast<float*>(ws + l.off_mse_partials);
  return faar_launch_gemm(ctx, &a, n_partials);
}

int bwd_impl(faar_ctx* ctx, const faar_shape* s, const faar_hparams* hp, const void* dYt, const void* Xt,
             float* V, const uint8_t* code, const uint8_t* scales, const float* s_global, float* adam_m,
             float* adam_u, float* dV, uint8_t* ws, const faar_ws_layout& l, int* n_partials,
             float* loss_out2 = nullptr, int n_mse_partials = 0, int row_major = 0) {
  faar_gemm_args a = {};
  if (loss_out2) {
    // the kernel's last CTA sums the forward's MSE partials and its own Round Loss partials
    a.fin_counter = reinterpret_cast<uint32_t*>(ws) + 2;
    a.fin_mse_partials = reinterpret_cast<const float*>(ws + l.off_mse_partials);
    a.fin_n_mse = n_mse_partials;
    a.fin_scale_mse = hp->mse_scale;
    a.fin_scale_round = (float)(1.0 / ((double)s->O * (double)s->K));
    a.fin_out2 = loss_out2;
  }
  a.mode = FAAR_GEMM_BWD;
  a.M = s->O; a.N = s->K; a.Kc = s->T;
  if (row_major == 1) {                    // dY [T, ldy] and X [T, ldx] as they are: token index = contraction row
    a.A = dYt; a.lda = s->ldy; a.a_mn = 1;
    a.B = Xt; a.ldb = s->ldx; a.b_mn = 1;
  } else if (row_major == 2) {             // dY^T from the forward kernel, X [T, ldx] as it is
    a.A = dYt; a.lda = l.ld_dyt;
    a.B = Xt; a.ldb = s->ldx; a.b_mn = 1;
  } else {
    a.A = dYt; a.lda = l.ld_dyt;
    a.B = Xt; a.ldb = s->ldxt;
  }
  a.status = reinterpret_cast<uint32_t*>(ws);
  a.partials = reinterpret_cast<float*>(ws + l.off_round_partials);
  a.V = V; a.code = code; a.scales = scales; a.s_global = s_global;
  a.adam_m = adam_m; a.adam_u = adam_u; a.dV = dV;
  a.beta = hp->beta;
  if (hp->beta_next > 0.f) {
    a.wsoft_next = reinterpret_cast<__nv_bfloat16*>(ws + l.off_wsoft);
    a.beta_next = hp->beta_next;
    ctx->wsoft_ws = ws;
    ctx->wsoft_beta = hp->beta_next;
  } else if (ctx->wsoft_ws == ws) {
    ctx->wsoft_ws = nullptr;               // V moves on without a matching operand
  }
  a.act_scale = hp->act_scale > 0.f ? hp->act_scale : 1.0f;
  a.lam_over_n = (float)((double)hp->lambda_round / ((double)s->O * (double)s->K));
  a.lr = hp->lr; a.b1 = hp->beta1; a.b2 = hp->beta2; a.eps = hp->eps; a.opt = hp->opt;
  if (hp->opt == 1) {
    a.inv_bc1 = (float)(1.0 / (1.0 - pow((double)hp->beta1, (double)hp->step)));
    a.inv_bc2 = (float)(1.0 / (1.0 - pow((double)hp->beta2, (double)hp->step)));
  }
  return faar_launch_gemm(ctx, &a, n_partials);
}

int check_gemm_operands(const faar_shape* s, bool need_x, bool need_xt) {
  if (need_x && (s->ldx < s->K || s->ldx % 8)) return s->ldx < s->K ? FAAR_ERR_SHAPE : FAAR_ERR_ALIGN;
  if (need_xt && (s->ldxt < s->T || s->ldxt % 8)) return s->ldxt < s->T ? FAAR_ERR_SHAPE : FAAR_ERR_ALIGN;
  return FAAR_OK;
}

// Everything faar_layer_step checks before it enqueues anything (also run by faar_layer_step_host before its
// first copy, so that a refused call leaves the staging buffers and the copy stream untouched).
int validate_step(const faar_ctx* ctx, const faar_shape* s, const faar_hparams* hp, const void* X, const void* Xt,
                  const void* Y_ref, const float* V, const uint8_t* code, const uint8_t* scales, const float* s_global,
                  const float* adam_m, const float* adam_u, const float* loss_out2, const void* workspace,
                  size_t workspace_bytes) {
  if (!ctx || !X || !Xt || !Y_ref || !V || !code || !scales || !s_global || !loss_out2) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(s);
  if (st) return st;
  if ((st = check_hp(hp, true))) return st;
  if (hp->opt == 1 && (!adam_m || !adam_u)) return FAAR_ERR_INVALID_ARG;
  if (s->yref_dtype != FAAR_BF16 && s->yref_dtype != FAAR_F32) return FAAR_ERR_DTYPE;
  if ((st = check_bwd_k(s))) return st;
  if ((st = check_ldy(s))) return st;
  if ((st = check_gemm_operands(s, true, true))) return st;
  if (!aligned16(X) || !aligned16(Xt) || !aligned16(V) || !aligned16(code) || (adam_m && !aligned16(adam_m)) ||
      (adam_u && !aligned16(adam_u)))
    return FAAR_ERR_ALIGN;
  if ((st = check_ws(s, workspace, workspace_bytes))) return st;
  return check_chain(ctx, hp, workspace);
}

}  // namespace

faar_prof_scope::faar_prof_scope(faar_ctx* ctx, int kernel_id) : c(ctx), pair(-1) {
  if (!c->prof_on) return;
  const int i = c->prof_used;
  while ((int)c->prof_events.size() < 2 * (i + 1)) {
    cudaEvent_t ev;
    if (cudaEventCreate(&ev) != cudaSuccess) return;
    c->prof_events.push_back(ev);
  }
  if (cudaEventRecord(c->prof_events[2 * i], c->stream) != cudaSuccess) return;
  c->prof_kernel.push_back(kernel_id);
  c->prof_used = i + 1;
  pair = i;
}

faar_prof_scope::~faar_prof_scope() {
  if (pair >= 0) cudaEventRecord(c->prof_events[2 * pair + 1], c->stream);
}

namespace {
int check_rows_cols(int rows, int cols, std::initializer_list<int64_t> lds, std::initializer_list<const void*> ptrs) {
  if (rows <= 0 || cols <= 0 || cols % 8) return FAAR_ERR_SHAPE;
  for (int64_t ld : lds) {
    if (ld < cols) return FAAR_ERR_SHAPE;
    if (ld % 8) return FAAR_ERR_ALIGN;
  }
  for (const void* q : ptrs)
    if (q && !aligned16(q)) return FAAR_ERR_ALIGN;
  return FAAR_OK;
}
int check_attention(int batch, int seq, int n_heads, int n_kv_heads, int head_dim, int64_t ldq, int64_t ldkv, int64_t ldo) {
  if (batch <= 0 || seq <= 0 || n_heads <= 0 || n_kv_heads <= 0 || n_heads % n_kv_heads) return FAAR_ERR_SHAPE;
  if (head_dim != 64 && head_dim != 128) return FAAR_ERR_SHAPE;
  if ((long long)batch * seq > 0x7FFFFFFFll) return FAAR_ERR_SHAPE;
  if (ldq < (int64_t)n_heads * head_dim || ldo < (int64_t)n_heads * head_dim || ldkv < (int64_t)n_kv_heads * head_dim)
    return FAAR_ERR_SHAPE;
  if (ldq % 8 || ldkv % 8 || ldo % 8) return FAAR_ERR_ALIGN;
  return FAAR_OK;
}
}  // namespace

extern "C" {

const char* faar_status_string(int status) {
  switch (status) {
    case FAAR_OK: return "ok";
    case FAAR_ERR_INVALID_ARG: return "invalid argument";
    case FAAR_ERR_SHAPE: return "unsupported shape";
    case FAAR_ERR_ALIGN: return "misaligned pointer or leading dimension";
    case FAAR_ERR_DTYPE: return "unsupported dtype";
    case FAAR_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case FAAR_ERR_ARCH: return "device is not sm_100";
    case FAAR_ERR_CUDA: return "CUDA error";
    case FAAR_ERR_TIMEOUT: return "device-side wait gave up";
  }
  return "unknown status";
}

int faar_create(faar_ctx** out, int device, void* stream) {
  if (!out) return FAAR_ERR_INVALID_ARG;
  *out = nullptr;
  cudaDeviceProp prop;
  cudaError_t e = cudaGetDeviceProperties(&prop, device);
  if (e != cudaSuccess) return FAAR_ERR_CUDA;
  if (prop.major != 10) return FAAR_ERR_ARCH;
  faar_ctx* c = new (std::nothrow) faar_ctx();
  if (!c) return FAAR_ERR_INVALID_ARG;
  c->device = device;
  c->num_sms = prop.multiProcessorCount;
  c->stream = reinterpret_cast<cudaStream_t>(stream);
  c->last_cuda_error = 0;
  c->encode_tiled = nullptr;
  c->tune_bn = 0;
  c->tune_tail = -1;
  c->tune_attention_fragments = 0;
  c->tune_wide = -1;
  c->last_gemm_split = 0;
  for (int i = 0; i < FAAR_GEMM_VARIANTS; ++i) c->gemm_max_pairs[i] = 0;
  c->wsoft_ws = nullptr;
  c->wsoft_beta = 0.f;
  c->copy_stream = nullptr;
  c->ev_copied = nullptr;
  c->ev_done[0] = c->ev_done[1] = nullptr;
  c->host_calls = 0;
  c->last_staging = nullptr;
  c->last_gemm_bn = 0;
  c->last_gemm_pairs = 0;
  c->prof_on = false;
  c->prof_used = 0;
  cudaDriverEntryPointQueryResult q;
  e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &c->encode_tiled, cudaEnableDefault, &q);
  if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !c->encode_tiled) {
    delete c;
    return FAAR_ERR_CUDA;
  }
  *out = c;
  return FAAR_OK;
}

int faar_destroy(faar_ctx* ctx) {
  if (ctx) {
    for (cudaEvent_t ev : ctx->prof_events) cudaEventDestroy(ev);
    if (ctx->ev_copied) cudaEventDestroy(ctx->ev_copied);
    for (int i = 0; i < 2; ++i)
      if (ctx->ev_done[i]) cudaEventDestroy(ctx->ev_done[i]);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  }
  delete ctx;
  return FAAR_OK;
}

const char* faar_kernel_name(int kernel) {
  switch (kernel) {
    case FAAR_K_AMAX: return "amax";
    case FAAR_K_SOFTQUANT_INIT: return "softquant_init";
    case FAAR_K_SOFT_WEIGHTS: return "soft_weights";
    case FAAR_K_GEMM_REF: return "gemm_ref";
    case FAAR_K_GEMM_FWD: return "gemm_fwd";
    case FAAR_K_GEMM_BWD: return "gemm_bwd";
    case FAAR_K_ROUND_LOSS: return "round_loss";
    case FAAR_K_FINALIZE: return "finalize";
    case FAAR_K_HARDEN_PACK: return "harden_pack";
    case FAAR_K_TRANSPOSE: return "transpose";
    case FAAR_K_ACT_FAKEQUANT: return "act_fakequant";
    case FAAR_K_ALIGN_LOSS: return "align_loss";
    case FAAR_K_GLUE: return "glue";
    case FAAR_K_NVFP4_GEMM: return "nvfp4_gemm";
    case FAAR_K_ATTENTION: return "attention";
  }
  return "unknown";
}

int faar_profile_begin(faar_ctx* ctx) {
  if (!ctx) return FAAR_ERR_INVALID_ARG;
  ctx->prof_on = true;
  ctx->prof_used = 0;
  ctx->prof_kernel.clear();
  return FAAR_OK;
}

int faar_profile_end(faar_ctx* ctx, faar_kernel_time* out, int capacity, int* count) {
  if (!ctx || !out || !count || capacity < 0) return FAAR_ERR_INVALID_ARG;
  FAAR_DEVICE_GUARD(ctx);
  ctx->prof_on = false;
  *count = 0;
  cudaError_t e = cudaStreamSynchronize(ctx->stream);
  if (e != cudaSuccess) return cuda_fail(ctx, (int)e);
  int launches[FAAR_K_COUNT] = {0};
  double total[FAAR_K_COUNT] = {0.0};
  for (int i = 0; i < ctx->prof_used; ++i) {
    float ms = 0.f;
    e = cudaEventElapsedTime(&ms, ctx->prof_events[2 * i], ctx->prof_events[2 * i + 1]);
    if (e != cudaSuccess) return cuda_fail(ctx, (int)e);
    const int k = ctx->prof_kernel[i];
    launches[k] += 1;
    total[k] += ms;
  }
  for (int k = 0; k < FAAR_K_COUNT && *count < capacity; ++k) {
    if (!launches[k]) continue;
    out[*count].kernel = k;
    out[*count].launches = launches[k];
    out[*count].total_ms = (float)total[k];
    *count += 1;
  }
  ctx->prof_used = 0;
  return FAAR_OK;
}

int faar_set_stream(faar_ctx* ctx, void* stream) {
  if (!ctx) return FAAR_ERR_INVALID_ARG;
  ctx->stream = reinterpret_cast<cudaStream_t>(stream);
  return FAAR_OK;
}

int faar_last_cuda_error(const faar_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

int faar_tune_tile_n(faar_ctx* ctx, int bn) {
  if (!ctx) return FAAR_ERR_INVALID_ARG;
  if (bn != 0 && (bn < 128 || bn > 256 || bn % 16 != 0)) return FAAR_ERR_INVALID_ARG;
  ctx->tune_bn = bn;
  return FAAR_OK;
}

int faar_tune_tail_split(faar_ctx* ctx, int columns) {
  if (!ctx || columns < -1) return FAAR_ERR_INVALID_ARG;
  ctx->tune_tail = columns;
  return FAAR_OK;
}

int faar_last_tail_split(const faar_ctx* ctx, int* columns) {
  if (!ctx || !columns) return FAAR_ERR_INVALID_ARG;
  *columns = ctx->last_gemm_split;
  return FAAR_OK;
}

int faar_tune_wide_tiles(faar_ctx* ctx, int mode) {
  if (!ctx || mode < -1 || mode > 1) return FAAR_ERR_INVALID_ARG;
  ctx->tune_wide = mode;
  return FAAR_OK;
}

int faar_attention_status(faar_ctx* ctx, uint32_t* detail_out) {
  if (!ctx) return FAAR_ERR_INVALID_ARG;
  FAAR_DEVICE_GUARD(ctx);
  uint32_t code = 0;
  int e = faar_attention_tc_status(&code);
  if (detail_out) *detail_out = code;
  if (e) return cuda_fail(ctx, e);
  return code ? FAAR_ERR_TIMEOUT : FAAR_OK;
}

int faar_tune_attention(faar_ctx* ctx, int mode) {
  if (!ctx || mode < 0 || mode > 2) return FAAR_ERR_INVALID_ARG;
  ctx->tune_attention_fragments = mode;
  return FAAR_OK;
}

int faar_last_gemm_config(const faar_ctx* ctx, int* bn, int* cta_pairs) {
  if (!ctx || !bn || !cta_pairs) return FAAR_ERR_INVALID_ARG;
  *bn = ctx->last_gemm_bn;
  *cta_pairs = ctx->last_gemm_pairs;
  return FAAR_OK;
}

int faar_workspace_size(const faar_shape* shape, size_t* bytes) {
  if (!bytes) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(shape);
  if (st) return st;
  *bytes = faar_ws_plan(shape).total;
  return FAAR_OK;
}

int faar_workspace_init(faar_ctx* ctx, void* workspace, size_t workspace_bytes) {
  if (!ctx) return FAAR_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < FAAR_WS_HEADER)
    return FAAR_ERR_WORKSPACE;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, (int)cudaMemsetAsync(workspace, 0, FAAR_WS_HEADER, ctx->stream));
}

int faar_check_status(faar_ctx* ctx, const void* workspace, uint32_t* detail_out) {
  if (!ctx || !workspace) return FAAR_ERR_INVALID_ARG;
  FAAR_DEVICE_GUARD(ctx);
  uint32_t word = 0;
  cudaError_t e = cudaStreamSynchronize(ctx->stream);
  if (e == cudaSuccess) e = cudaMemcpy(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(ctx, (int)e);
  if (detail_out) *detail_out = word;
  return word ? FAAR_ERR_TIMEOUT : FAAR_OK;
}

int faar_selftest_wait_timeout(faar_ctx* ctx, void* workspace, size_t workspace_bytes, unsigned int limit_us) {
  if (!ctx) return FAAR_ERR_INVALID_ARG;
  if (limit_us == 0 || limit_us > 1000000u) return FAAR_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < FAAR_WS_HEADER)
    return FAAR_ERR_WORKSPACE;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_wait_selftest(ctx, reinterpret_cast<uint32_t*>(workspace), 1000ull * limit_us));
}

int faar_softquant_init(faar_ctx* ctx, const faar_shape* s, const void* W, float s_global_in, uint8_t* scales,
                        float* s_global_out, uint8_t* code, float* V_init, void* workspace,
                        size_t workspace_bytes) {
  if (!ctx || !W || !scales || !s_global_out || !code || !V_init) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(s);
  if (st) return st;
  if (s->w_dtype != FAAR_BF16 && s->w_dtype != FAAR_F32) return FAAR_ERR_DTYPE;
  if (s->ldw < s->K) return FAAR_ERR_SHAPE;
  if ((int64_t)s->O * (s->K / 8) > 0xFFFFFFFFll) return FAAR_ERR_SHAPE;   // 8-element groups are counted in 32 bits
  if (s->ldw % 8 || !aligned16(W) || !aligned16(V_init) || !aligned16(code)) return FAAR_ERR_ALIGN;
  if (!isfinite(s_global_in) || s_global_in < 0.f) return FAAR_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < FAAR_WS_HEADER)
    return FAAR_ERR_WORKSPACE;
  FAAR_DEVICE_GUARD(ctx);
  unsigned long long* amax_word = reinterpret_cast<unsigned long long*>(workspace) + 2;
  return cuda_fail(ctx, faar_launch_softquant_init(ctx, s, W, s_global_in, scales, s_global_out, code, V_init,
                                                   amax_word));
}

int faar_softquant_eval(faar_ctx* ctx, const faar_shape* s, const float* V, const uint8_t* code,
                        const uint8_t* scales, const float* s_global, float beta, float* W_soft, float* h,
                        void* W_soft_bf16) {
  if (!ctx || !V || !code || !scales || !s_global) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(s);
  if (st) return st;
  if (!(beta > 0.f) || !isfinite(beta)) return FAAR_ERR_INVALID_ARG;
  if (!aligned16(V) || !aligned16(code) || (W_soft && !aligned16(W_soft)) || (h && !aligned16(h)) ||
      (W_soft_bf16 && !aligned16(W_soft_bf16)))
    return FAAR_ERR_ALIGN;
  if (!W_soft && !h && !W_soft_bf16) return FAAR_OK;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_softquant_eval(ctx, s, V, code, scales, s_global, beta, W_soft, h,
                                                   reinterpret_cast<__nv_bfloat16*>(W_soft_bf16)));
}

int faar_softquant_operand_f32(faar_ctx* ctx, const faar_shape* s, const float* V, const uint8_t* code,
                               const uint8_t* scales, const float* s_global, float beta, float* W_operand) {
  if (!ctx || !V || !code || !scales || !s_global || !W_operand) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(s);
  if (st) return st;
  if (!(beta > 0.f) || !(beta <= FAAR_BETA_MAX)) return FAAR_ERR_INVALID_ARG;
  if (!aligned16(V) || !aligned16(code) || !aligned16(W_operand)) return FAAR_ERR_ALIGN;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_softquant_eval(ctx, s, V, code, scales, s_global, beta, nullptr, nullptr, nullptr,
                                                   W_operand));
}

int faar_transpose_bf16(faar_ctx* ctx, int rows, int cols, const void* in, int64_t ld_in, void* out,
                        int64_t ld_out) {
  if (!ctx || !in || !out) return FAAR_ERR_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || ld_in < cols || ld_out < rows) return FAAR_ERR_SHAPE;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_transpose_bf16(ctx, rows, cols, in, ld_in, out, ld_out));
}

int faar_act_fakequant(faar_ctx* ctx, int T, int K, const void* X, int64_t ldx, float s_global_in, void* Xq_units,
                       int64_t ldq, float* s_global_out, uint8_t* packed, uint8_t* scales, void* workspace,
                       size_t workspace_bytes) {
  if (!ctx || !X || !Xq_units || !s_global_out) return FAAR_ERR_INVALID_ARG;
  if (T <= 0 || K <= 0 || K % 16 != 0 || ldx < K || ldq < K) return FAAR_ERR_SHAPE;
  if ((int64_t)T * (K / 8) > 0xFFFFFFFFll) return FAAR_ERR_SHAPE;
  if (ldx % 8 || ldq % 8 || !aligned16(X) || !aligned16(Xq_units) || (packed && !aligned16(packed))) return FAAR_ERR_ALIGN;
  if (!isfinite(s_global_in) || s_global_in < 0.f) return FAAR_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < FAAR_WS_HEADER)
    return FAAR_ERR_WORKSPACE;
  FAAR_DEVICE_GUARD(ctx);
  unsigned long long* amax_word = reinterpret_cast<unsigned long long*>(workspace) + 2;
  return cuda_fail(ctx, faar_launch_act_fakequant(ctx, T, K, X, ldx, s_global_in, Xq_units, ldq, s_global_out, packed,
                                                  scales, amax_word));
}

int faar_layer_ref(faar_ctx* ctx, const faar_shape* s, const void* X, const void* W, void* Y_ref,
                   void* workspace, size_t workspace_bytes) {
  if (!ctx || !X || !W || !Y_ref) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(s);
  if (st) return st;
  if (s->w_dtype != FAAR_BF16) return FAAR_ERR_DTYPE;
  if (s->yref_dtype != FAAR_BF16 && s->yref_dtype != FAAR_F32) return FAAR_ERR_DTYPE;
  if (s->ldw < s->K) return FAAR_ERR_SHAPE;
  if ((st = check_ldy(s))) return st;
  if ((st = check_gemm_operands(s, true, false))) return st;
  if (s->ldw % 8 || !aligned16(X) || !aligned16(W)) return FAAR_ERR_ALIGN;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < FAAR_WS_HEADER)
    return FAAR_ERR_WORKSPACE;
  FAAR_DEVICE_GUARD(ctx);
  faar_gemm_args a = {};
  a.mode = FAAR_GEMM_REF;
  a.M = s->O; a.N = s->T; a.Kc = s->K;
  a.A = W; a.lda = s->ldw;
  a.B = X; a.ldb = s->ldx;
  a.status = reinterpret_cast<uint32_t*>(workspace);
  a.Yout = Y_ref; a.yout_dtype = s->yref_dtype; a.ldy = s->ldy; a.yref_t = s->yref_transposed;
  return cuda_fail(ctx, faar_launch_gemm(ctx, &a, nullptr));
}

int faar_layer_dx(faar_ctx* ctx, const faar_shape* s, float beta, const void* dY, const float* V, const uint8_t* code,
                  const uint8_t* scales, const float* s_global, void* WsoftT, void* dX, void* workspace,
                  size_t workspace_bytes) {
  (void)WsoftT;                                  // kept in the signature; the operand is read untransposed now
  if (!ctx || !dY || !V || !code || !scales || !s_global || !dX) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(s);
  if (st) return st;
  if (!(beta > 0.f) || !isfinite(beta)) return FAAR_ERR_INVALID_ARG;
  if (s->ldy < s->O || s->ldx < s->K) return FAAR_ERR_SHAPE;
  if (s->ldy % 8 || s->ldx % 8 || !aligned16(dY) || !aligned16(V) || !aligned16(code) || !aligned16(dX))
    return FAAR_ERR_ALIGN;
  if ((st = check_ws(s, workspace, workspace_bytes))) return st;
  FAAR_DEVICE_GUARD(ctx);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const faar_ws_layout l = faar_ws_plan(s);
  __nv_bfloat16* wsoft = reinterpret_cast<__nv_bfloat16*>(ws + l.off_wsoft);
  if (ctx->wsoft_ws == workspace) ctx->wsoft_ws = nullptr;     // the operand slot is overwritten below
  int e = faar_launch_softquant_eval(ctx, s, V, code, scales, s_global, beta, nullptr, nullptr, wsoft);
  if (e) return cuda_fail(ctx, e);
  // dX^T[K,T] = W_soft^T[K,O] * dY[T,O]^T, written transposed as dX[T,K].  W_soft [O,K] is that A operand with
  // its M index (k) contiguous and the contraction index (o) as the row: read as it is.
  faar_gemm_args a = {};
  a.mode = FAAR_GEMM_REF;
  a.M = s->K; a.N = s->T; a.Kc = s->O;
  a.A = wsoft; a.lda = s->K; a.a_mn = 1;
  a.B = dY; a.ldb = s->ldy;
  a.status = reinterpret_cast<uint32_t*>(ws);
  a.Yout = dX; a.yout_dtype = FAAR_BF16; a.ldy = s->ldx;
  return cuda_fail(ctx, faar_launch_gemm(ctx, &a, nullptr));
}

int faar_layer_dx_operand(faar_ctx* ctx, const faar_shape* s, const void* dY, const void* Wsoft, void* dX,
                          void* workspace, size_t workspace_bytes) {
  if (!ctx || !dY || !Wsoft || !dX) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(s);
  if (st) return st;
  if (s->ldy < s->O || s->ldx < s->K || s->ldw < s->K) return FAAR_ERR_SHAPE;
  if (s->ldy % 8 || s->ldx % 8 || s->ldw % 8 || !aligned16(dY) || !aligned16(Wsoft) || !aligned16(dX)) return FAAR_ERR_ALIGN;
  if ((st = check_ws(s, workspace, workspace_bytes))) return st;
  FAAR_DEVICE_GUARD(ctx);
  // dX^T[K,T] = W_soft^T[K,O] * dY[T,O]^T written transposed as dX[T,K], as in faar_layer_dx
  faar_gemm_args a = {};
  a.mode = FAAR_GEMM_REF;
  a.M = s->K; a.N = s->T; a.Kc = s->O;
  a.A = Wsoft; a.lda = s->ldw; a.a_mn = 1;
  a.B = dY; a.ldb = s->ldy;
  a.status = reinterpret_cast<uint32_t*>(workspace);
  a.Yout = dX; a.yout_dtype = FAAR_BF16; a.ldy = s->ldx;
  return cuda_fail(ctx, faar_launch_gemm(ctx, &a, nullptr));
}

int faar_layer_fwd(faar_ctx* ctx, const faar_shape* s, const faar_hparams* hp, const void* X, const void* Y_ref,
                   const float* V, const uint8_t* code, const uint8_t* scales, const float* s_global, void* dYt,
                   float* loss_mse, void* Y_q, void* workspace, size_t workspace_bytes) {
  if (!ctx || !X || !Y_ref || !V || !code || !scales || !s_global || !dYt || !loss_mse) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(s);
  if (st) return st;
  if ((st = check_hp(hp, false))) return st;
  if (s->yref_dtype != FAAR_BF16 && s->yref_dtype != FAAR_F32) return FAAR_ERR_DTYPE;
  if ((st = check_ldy(s))) return st;
  if ((st = check_gemm_operands(s, true, false))) return st;
  if (!aligned16(X) || !aligned16(V) || !aligned16(code) || !aligned16(dYt)) return FAAR_ERR_ALIGN;
  if ((st = check_ws(s, workspace, workspace_bytes))) return st;
  if ((st = check_chain(ctx, hp, workspace))) return st;
  FAAR_DEVICE_GUARD(ctx);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const faar_ws_layout l = faar_ws_plan(s);
  int np = 0;
  int e = fwd_impl(ctx, s, hp, X, Y_ref, V, code, scales, s_global, dYt, Y_q, ws, l, &np);
  if (e) return cuda_fail(ctx, e);
  e = faar_launch_finalize(ctx, reinterpret_cast<float*>(ws + l.off_mse_partials), np, hp->mse_scale, loss_mse,
                           nullptr, 0, 0.f, nullptr);
  return cuda_fail(ctx, e);
}

int faar_round_loss(faar_ctx* ctx, const float* V, int64_t N, float* loss_round, void* workspace,
                    size_t workspace_bytes) {
  if (!ctx || !V || !loss_round) return FAAR_ERR_INVALID_ARG;
  if (N <= 0) return FAAR_ERR_SHAPE;
  if (!aligned16(V)) return FAAR_ERR_ALIGN;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
      workspace_bytes < FAAR_WS_HEADER + 2 * sizeof(float) * FAAR_MAX_PARTIALS)
    return FAAR_ERR_WORKSPACE;
  FAAR_DEVICE_GUARD(ctx);
  float* partials = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace) + FAAR_WS_HEADER +
                                             sizeof(float) * FAAR_MAX_PARTIALS);
  int np = 0;
  int e = faar_launch_round_partials(ctx, V, N, partials, &np);
  if (e) return cuda_fail(ctx, e);
  e = faar_launch_finalize(ctx, partials, np, (float)(1.0 / (double)N), loss_round, nullptr, 0, 0.f, nullptr);
  return cuda_fail(ctx, e);
}

int faar_layer_bwd(faar_ctx* ctx, const faar_shape* s, const faar_hparams* hp, const void* dYt, const void* Xt,
                   float* V, const uint8_t* code, const uint8_t* scales, const float* s_global, float* adam_m,
                   float* adam_u, float* dV, void* workspace, size_t workspace_bytes) {
  if (!ctx || !dYt || !Xt || !V || !code || !scales || !s_global) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(s);
  if (st) return st;
  if ((st = check_hp(hp, true))) return st;
  if (hp->opt == 1 && (!adam_m || !adam_u)) return FAAR_ERR_INVALID_ARG;
  if ((st = check_bwd_k(s))) return st;
  if ((st = check_gemm_operands(s, false, true))) return st;
  if (!aligned16(dYt) || !aligned16(Xt) || !aligned16(V) || !aligned16(code) || (adam_m && !aligned16(adam_m)) ||
      (adam_u && !aligned16(adam_u)) || (dV && !aligned16(dV)))
    return FAAR_ERR_ALIGN;
  if ((st = check_ws(s, workspace, workspace_bytes))) return st;
  FAAR_DEVICE_GUARD(ctx);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const faar_ws_layout l = faar_ws_plan(s);
  return cuda_fail(ctx, bwd_impl(ctx, s, hp, dYt, Xt, V, code, scales, s_global, adam_m, adam_u, dV, ws, l, nullptr));
}

int faar_layer_bwd_rowmajor(faar_ctx* ctx, const faar_shape* s, const faar_hparams* hp, const void* dY, const void* X,
                            float* V, const uint8_t* code, const uint8_t* scales, const float* s_global, float* adam_m,
                            float* adam_u, float* dV, void* workspace, size_t workspace_bytes) {
  if (!ctx || !dY || !X || !V || !code || !scales || !s_global) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(s);
  if (st) return st;
  if ((st = check_hp(hp, true))) return st;
  if (hp->opt == 1 && (!adam_m || !adam_u)) return FAAR_ERR_INVALID_ARG;
  if ((st = check_bwd_k(s))) return st;
  if (s->ldy < s->O || s->ldx < s->K) return FAAR_ERR_SHAPE;
  if (s->ldy % 8 || s->ldx % 8 || !aligned16(dY) || !aligned16(X) || !aligned16(V) || !aligned16(code) ||
      (adam_m && !aligned16(adam_m)) || (adam_u && !aligned16(adam_u)) || (dV && !aligned16(dV)))
    return FAAR_ERR_ALIGN;
  if ((st = check_ws(s, workspace, workspace_bytes))) return st;
  FAAR_DEVICE_GUARD(ctx);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const faar_ws_layout l = faar_ws_plan(s);
  return cuda_fail(ctx, bwd_impl(ctx, s, hp, dY, X, V, code, scales, s_global, adam_m, adam_u, dV, ws, l, nullptr, nullptr, 0,
                                 1));
}

int faar_layer_step(faar_ctx* ctx, const faar_shape* s, const faar_hparams* hp, const void* X, const void* Xt,
                    const void* Y_ref, float* V, const uint8_t* code, const uint8_t* scales, const float* s_global,
                    float* adam_m, float* adam_u, float* loss_out2, void* workspace, size_t workspace_bytes) {
  int st = validate_step(ctx, s, hp, X, Xt, Y_ref, V, code, scales, s_global, adam_m, adam_u, loss_out2, workspace,
                         workspace_bytes);
  if (st) return st;
  FAAR_DEVICE_GUARD(ctx);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const faar_ws_layout l = faar_ws_plan(s);
  void* dYt = ws + l.off_dyt;
  int np_mse = 0, np_round = 0;
  int e = fwd_impl(ctx, s, hp, X, Y_ref, V, code, scales, s_global, dYt, nullptr, ws, l, &np_mse);
  if (e) return cuda_fail(ctx, e);
  e = bwd_impl(ctx, s, hp, dYt, Xt, V, code, scales, s_global, adam_m, adam_u, nullptr, ws, l, &np_round, loss_out2,
               np_mse);
  return cuda_fail(ctx, e);
}

int faar_nvfp4_expand(faar_ctx* ctx, int rows, int K, const void* packed, const void* scales, void* out, int64_t ld) {
  if (!ctx || !packed || !scales || !out) return FAAR_ERR_INVALID_ARG;
  if (rows <= 0 || K <= 0 || K % 16 || ld < K) return FAAR_ERR_SHAPE;
  if (ld % 8 || !aligned16(out) || (reinterpret_cast<uintptr_t>(packed) & 7u)) return FAAR_ERR_ALIGN;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_nvfp4_expand(ctx, rows, K, reinterpret_cast<const uint8_t*>(packed),
                                                 reinterpret_cast<const uint8_t*>(scales), out, ld));
}

// Copy-stream bookkeeping shared by the host-batch entry points: creates the stream and events on first use and
// makes the copy stream wait until the staging set `key` is free again.  Returns the event slot of this call.
static cudaError_t begin_host_copy(faar_ctx* ctx, const void* key, int* slot_out) {
  cudaError_t e = cudaSuccess;
  if (!ctx->copy_stream) {                       // host resources of this path, created on first use
    e = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_copied, cudaEventDisableTiming);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming);
    if (e != cudaSuccess) return e;
  }
  // The staging buffers of this call were last read by the step of two calls ago when the caller
  // alternates between two sets (then this copy overlaps the previous step), by the previous step
  // when it reuses one set (then the copy waits for it).
  const unsigned long long n = ctx->host_calls++;
  const int slot = (int)(n & 1);
  if (n >= 2) e = cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_done[slot], 0);
  if (e == cudaSuccess && n >= 1 && ctx->last_staging == key)
    e = cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_done[slot ^ 1], 0);
  if (e == cudaSuccess && n == 0) {              // order after whatever the caller enqueued before (set-up)
    e = cudaEventRecord(ctx->ev_done[slot], ctx->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_done[slot], 0);
  }
  ctx->last_staging = key;
  *slot_out = slot;
  return e;
}

int faar_layer_step_host_nvfp4(faar_ctx* ctx, const faar_shape* s, const faar_hparams* hp, const void* Xpacked_host,
                               const void* Xscales_host, const void* Y_ref_host, void* Xpacked_dev, void* Xscales_dev,
                               void* Xq_dev, void* Yref_dev, float* V, const uint8_t* code, const uint8_t* scales,
                               const float* s_global, float* adam_m, float* adam_u, float* loss_dev2,
                               float* loss_host2, void* workspace, size_t workspace_bytes) {
  if (!ctx || !Xpacked_host || !Xscales_host || !Y_ref_host || !Xpacked_dev || !Xscales_dev || !Xq_dev || !Yref_dev ||
      !loss_dev2 || !loss_host2)
    return FAAR_ERR_INVALID_ARG;
  // every check of the step itself, before the first copy is enqueued (X^T is not needed: the dW GEMM reads
  // the expanded batch with the token index as its contraction row)
  int st = validate_step(ctx, s, hp, Xq_dev, Xq_dev, Yref_dev, V, code, scales, s_global, adam_m, adam_u, loss_dev2,
                         workspace, workspace_bytes);
  if (st) return st;
  if (!(hp->act_scale > 0.f)) return FAAR_ERR_INVALID_ARG;      // the tensor scale of the quantised batch
  if ((reinterpret_cast<uintptr_t>(Xpacked_dev) & 15u) || (reinterpret_cast<uintptr_t>(Xscales_dev) & 15u)) return FAAR_ERR_ALIGN;
  FAAR_DEVICE_GUARD(ctx);
  int slot = 0;
  cudaError_t e = begin_host_copy(ctx, Xq_dev, &slot);
  const size_t ybytes = s->yref_dtype == FAAR_BF16 ? 2 : 4;
  const size_t n_val = (size_t)s->T * (size_t)s->K;
  if (e == cudaSuccess) e = cudaMemcpyAsync(Xpacked_dev, Xpacked_host, n_val / 2, cudaMemcpyHostToDevice, ctx->copy_stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(Xscales_dev, Xscales_host, n_val / 16, cudaMemcpyHostToDevice, ctx->copy_stream);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(Yref_dev, Y_ref_host, (size_t)(s->yref_transposed ? s->O : s->T) * (size_t)s->ldy * ybytes,
                        cudaMemcpyHostToDevice, ctx->copy_stream);
  if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_copied, ctx->copy_stream);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->stream, ctx->ev_copied, 0);
  if (e != cudaSuccess) return cuda_fail(ctx, (int)e);
  int le = faar_launch_nvfp4_expand(ctx, s->T, s->K, reinterpret_cast<const uint8_t*>(Xpacked_dev),
                                    reinterpret_cast<const uint8_t*>(Xscales_dev), Xq_dev, s->ldx);
  if (le) return cuda_fail(ctx, le);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const faar_ws_layout l = faar_ws_plan(s);
  void* dYt = ws + l.off_dyt;
  int np_mse = 0, np_round = 0;
  le = fwd_impl(ctx, s, hp, Xq_dev, Yref_dev, V, code, scales, s_global, dYt, nullptr, ws, l, &np_mse);
  if (le) return cuda_fail(ctx, le);
  le = bwd_impl(ctx, s, hp, dYt, Xq_dev, V, code, scales, s_global, adam_m, adam_u, nullptr, ws, l, &np_round, loss_dev2,
                np_mse, 2);
  if (le) return cuda_fail(ctx, le);
  e = cudaMemcpyAsync(loss_host2, loss_dev2, 2 * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream);
  if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_done[slot], ctx->stream);
  return cuda_fail(ctx, (int)e);
}

int faar_layer_step_host(faar_ctx* ctx, const faar_shape* s, const faar_hparams* hp, const void* X_host,
                         const void* Y_ref_host, const void* W, void* X_dev, void* Xt_dev, void* Yref_dev, float* V,
                         const uint8_t* code, const uint8_t* scales, const float* s_global, float* adam_m,
                         float* adam_u, float* loss_dev2, float* loss_host2, void* workspace,
                         size_t workspace_bytes) {
  if (!ctx || !X_host || (!Y_ref_host && !W) || !X_dev || !Xt_dev || !Yref_dev || !loss_dev2 || !loss_host2)
    return FAAR_ERR_INVALID_ARG;
  // every check of the step itself, before the first copy is enqueued
  int st = validate_step(ctx, s, hp, X_dev, Xt_dev, Yref_dev, V, code, scales, s_global, adam_m, adam_u, loss_dev2,
                         workspace, workspace_bytes);
  if (st) return st;
  if (!Y_ref_host) {                             // what faar_layer_ref will ask of W
    if (s->w_dtype != FAAR_BF16) return FAAR_ERR_DTYPE;
    if (s->ldw < s->K) return FAAR_ERR_SHAPE;
    if (s->ldw % 8 || !aligned16(W)) return FAAR_ERR_ALIGN;
  }
  FAAR_DEVICE_GUARD(ctx);
  int slot = 0;
  cudaError_t e = begin_host_copy(ctx, X_dev, &slot);
  const size_t ybytes = s->yref_dtype == FAAR_BF16 ? 2 : 4;
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(X_dev, X_host, (size_t)s->T * (size_t)s->ldx * 2, cudaMemcpyHostToDevice, ctx->copy_stream);
  if (e == cudaSuccess && Y_ref_host)
    e = cudaMemcpyAsync(Yref_dev, Y_ref_host, (size_t)(s->yref_transposed ? s->O : s->T) * (size_t)s->ldy * ybytes,
                        cudaMemcpyHostToDevice,
                        ctx->copy_stream);
  if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_copied, ctx->copy_stream);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->stream, ctx->ev_copied, 0);
  if (e != cudaSuccess) return cuda_fail(ctx, (int)e);
  st = faar_transpose_bf16(ctx, s->T, s->K, X_dev, s->ldx, Xt_dev, s->ldxt);
  if (st) return st;
  if (!Y_ref_host) {                             // the batch's frozen target from the X that has just arrived
    st = faar_layer_ref(ctx, s, X_dev, W, Yref_dev, workspace, workspace_bytes);
    if (st) return st;
  }
  st = faar_layer_step(ctx, s, hp, X_dev, Xt_dev, Yref_dev, V, code, scales, s_global, adam_m, adam_u, loss_dev2,
                       workspace, workspace_bytes);
  if (st) return st;
  e = cudaMemcpyAsync(loss_host2, loss_dev2, 2 * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream);
  if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_done[slot], ctx->stream);
  return cuda_fail(ctx, (int)e);
}

int faar_silu_mul(faar_ctx* ctx, int rows, int cols, const void* gate, int64_t ldg, const void* up, int64_t ldu,
                  void* out, int64_t ldo) {
  if (!ctx || !gate || !up || !out) return FAAR_ERR_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || cols % 8 || ldg < cols || ldu < cols || ldo < cols) return FAAR_ERR_SHAPE;
  if (ldg % 8 || ldu % 8 || ldo % 8 || !aligned16(gate) || !aligned16(up) || !aligned16(out)) return FAAR_ERR_ALIGN;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_silu_mul(ctx, rows, cols, gate, ldg, up, ldu, out, ldo));
}

int faar_nvfp4_gemm(faar_ctx* ctx, int M, int N, int K, const uint8_t* A_packed, const uint8_t* A_scales_tiled,
                    const float* A_s_global, const uint8_t* B_packed, const uint8_t* B_scales_tiled, const float* B_s_global,
                    void* C, int64_t ldc, void* workspace, size_t workspace_bytes) {
  if (!ctx || !A_packed || !A_scales_tiled || !A_s_global || !B_packed || !B_scales_tiled || !B_s_global || !C)
    return FAAR_ERR_INVALID_ARG;
  if (M <= 0 || N <= 0 || K <= 0 || K % 32 != 0 || ldc < N) return FAAR_ERR_SHAPE;
  if (!aligned16(A_packed) || !aligned16(B_packed) || !aligned16(A_scales_tiled) || !aligned16(B_scales_tiled) ||
      (reinterpret_cast<uintptr_t>(C) & 1u))
    return FAAR_ERR_ALIGN;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < FAAR_WS_HEADER)
    return FAAR_ERR_WORKSPACE;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_nvfp4_gemm(ctx, M, N, K, A_packed, A_scales_tiled, A_s_global, B_packed, B_scales_tiled,
                                               B_s_global, C, ldc, reinterpret_cast<uint32_t*>(workspace)));
}

// ---- element-wise pieces of a decoder block (full-model alignment) -----------------------------------
int faar_rmsnorm(faar_ctx* ctx, int rows, int cols, const void* x, int64_t ldx, const float* g, float eps, void* y,
                 int64_t ldy, float* rstd) {
  if (!ctx || !x || !g || !y) return FAAR_ERR_INVALID_ARG;
  if (!(eps >= 0.f) || !isfinite(eps)) return FAAR_ERR_INVALID_ARG;
  int st = check_rows_cols(rows, cols, {ldx, ldy}, {x, g, y});
  if (st) return st;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_rmsnorm(ctx, rows, cols, x, ldx, nullptr, 0, nullptr, 0, g, eps, y, ldy, rstd));
}

int faar_add_rmsnorm(faar_ctx* ctx, int rows, int cols, const void* a, int64_t lda, const void* b, int64_t ldb, void* sum,
                     int64_t lds, const float* g, float eps, void* y, int64_t ldy, float* rstd) {
  if (!ctx || !a || !b || !sum || !g || !y) return FAAR_ERR_INVALID_ARG;
  if (!(eps >= 0.f) || !isfinite(eps)) return FAAR_ERR_INVALID_ARG;
  int st = check_rows_cols(rows, cols, {lda, ldb, lds, ldy}, {a, b, sum, g, y});
  if (st) return st;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_rmsnorm(ctx, rows, cols, a, lda, b, ldb, sum, lds, g, eps, y, ldy, rstd));
}

int faar_rmsnorm_bwd(faar_ctx* ctx, int rows, int cols, const void* dy, int64_t lddy, const void* x, int64_t ldx,
                     const float* g, const float* rstd, const void* add, int64_t ldadd, void* dx, int64_t lddx) {
  if (!ctx || !dy || !x || !g || !rstd || !dx) return FAAR_ERR_INVALID_ARG;
  int st = check_rows_cols(rows, cols, {lddy, ldx, lddx}, {dy, x, g, dx, add});
  if (st) return st;
  if (add && (ldadd < cols || ldadd % 8)) return ldadd < cols ? FAAR_ERR_SHAPE : FAAR_ERR_ALIGN;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_rmsnorm_bwd(ctx, rows, cols, dy, nullptr, nullptr, lddy, x, ldx, g, rstd, add, ldadd, dx, lddx));
}

int faar_rmsnorm_bwd_sum(faar_ctx* ctx, int rows, int cols, const void* dy, const void* dy2, const void* dy3, int64_t lddy,
                         const void* x, int64_t ldx, const float* g, const float* rstd, const void* add, int64_t ldadd,
                         void* dx, int64_t lddx) {
  if (!ctx || !dy || !x || !g || !rstd || !dx) return FAAR_ERR_INVALID_ARG;
  if (dy3 && !dy2) return FAAR_ERR_INVALID_ARG;
  int st = check_rows_cols(rows, cols, {lddy, ldx, lddx}, {dy, dy2, dy3, x, g, dx, add});
  if (st) return st;
  if (add && (ldadd < cols || ldadd % 8)) return ldadd < cols ? FAAR_ERR_SHAPE : FAAR_ERR_ALIGN;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_rmsnorm_bwd(ctx, rows, cols, dy, dy2, dy3, lddy, x, ldx, g, rstd, add, ldadd, dx, lddx));
}

int faar_rope(faar_ctx* ctx, int rows, int n_heads, int head_dim, const void* x, int64_t ldx, const int* positions,
              float theta, int inverse, void* y, int64_t ldy) {
  if (!ctx || !x || !positions || !y) return FAAR_ERR_INVALID_ARG;
  if (n_heads <= 0 || head_dim <= 0 || head_dim % 16) return FAAR_ERR_SHAPE;
  if (!(theta > 1.f) || !isfinite(theta)) return FAAR_ERR_INVALID_ARG;
  int st = check_rows_cols(rows, n_heads * head_dim, {ldx, ldy}, {x, y});
  if (st) return st;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_rope(ctx, rows, n_heads, head_dim, x, ldx, positions, theta, inverse, y, ldy));
}

int faar_silu_mul_bwd(faar_ctx* ctx, int rows, int cols, const void* dout, int64_t ldd, const void* gate, int64_t ldg,
                      const void* up, int64_t ldu, void* dgate, int64_t lddg, void* dup, int64_t lddu) {
  if (!ctx || !dout || !gate || !up || !dgate || !dup) return FAAR_ERR_INVALID_ARG;
  int st = check_rows_cols(rows, cols, {ldd, ldg, ldu, lddg, lddu}, {dout, gate, up, dgate, dup});
  if (st) return st;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_silu_mul_bwd(ctx, rows, cols, dout, ldd, gate, ldg, up, ldu, dgate, lddg, dup, lddu));
}

int faar_add(faar_ctx* ctx, int rows, int cols, const void* a, int64_t lda, const void* b, int64_t ldb, void* out,
             int64_t ldo) {
  if (!ctx || !a || !b || !out) return FAAR_ERR_INVALID_ARG;
  int st = check_rows_cols(rows, cols, {lda, ldb, ldo}, {a, b, out});
  if (st) return st;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_add(ctx, rows, cols, a, lda, b, ldb, out, ldo));
}

int faar_attention_fwd(faar_ctx* ctx, int batch, int seq, int n_heads, int n_kv_heads, int head_dim, const void* q,
                       int64_t ldq, const void* k, const void* v, int64_t ldkv, void* out, int64_t ldo, float* lse) {
  if (!ctx || !q || !k || !v || !out || !lse) return FAAR_ERR_INVALID_ARG;
  int st = check_attention(batch, seq, n_heads, n_kv_heads, head_dim, ldq, ldkv, ldo);
  if (st) return st;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return FAAR_ERR_ALIGN;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_attention_fwd(ctx, batch, seq, n_heads, n_kv_heads, head_dim, q, ldq, k, v, ldkv, out, ldo, lse));
}

int faar_attention_bwd(faar_ctx* ctx, int batch, int seq, int n_heads, int n_kv_heads, int head_dim, const void* q,
                       int64_t ldq, const void* k, const void* v, int64_t ldkv, const void* out, const void* dout,
                       int64_t ldo, const float* lse, float* dsum, void* dq, void* dk, void* dv) {
  if (!ctx || !q || !k || !v || !out || !dout || !lse || !dsum || !dq || !dk || !dv) return FAAR_ERR_INVALID_ARG;
  int st = check_attention(batch, seq, n_heads, n_kv_heads, head_dim, ldq, ldkv, ldo);
  if (st) return st;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(dout) || !aligned16(dq) ||
      !aligned16(dk) || !aligned16(dv))
    return FAAR_ERR_ALIGN;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_attention_bwd(ctx, batch, seq, n_heads, n_kv_heads, head_dim, q, ldq, k, v, ldkv, out,
                                                  dout, ldo, lse, dsum, dq, dk, dv));
}

int faar_embedding(faar_ctx* ctx, int rows, int cols, int vocab, const void* table, int64_t ldt, const int* tokens,
                   void* out, int64_t ldo) {
  if (!ctx || !table || !tokens || !out) return FAAR_ERR_INVALID_ARG;
  if (vocab <= 0) return FAAR_ERR_SHAPE;
  int st = check_rows_cols(rows, cols, {ldt, ldo}, {table, out});
  if (st) return st;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_embedding(ctx, rows, cols, vocab, table, ldt, tokens, out, ldo));
}

int faar_swizzle_scales(faar_ctx* ctx, int rows, int cols, const uint8_t* scales, uint8_t* scales_tiled,
                        size_t tiled_bytes) {
  if (!ctx || !scales || !scales_tiled) return FAAR_ERR_INVALID_ARG;
  if (rows <= 0 || cols <= 0) return FAAR_ERR_SHAPE;
  if (tiled_bytes < (size_t)((rows + 127) / 128) * (size_t)((cols + 3) / 4) * 512) return FAAR_ERR_SHAPE;
  if (reinterpret_cast<uintptr_t>(scales_tiled) & 3u) return FAAR_ERR_ALIGN;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_swizzle_scales(ctx, rows, cols, scales, scales_tiled));
}

int faar_align_loss_workspace_size(int T, int vocab, size_t* bytes) {
  if (!bytes) return FAAR_ERR_INVALID_ARG;
  if (T <= 0 || vocab <= 0) return FAAR_ERR_SHAPE;
  *bytes = faar_align_up(FAAR_WS_HEADER + 2 * sizeof(float) * (size_t)T, 1024);      // two partial sums per CTA
  return FAAR_OK;
}

int faar_align_loss(faar_ctx* ctx, int T, int vocab, int hidden, const void* Z_fp, const void* Z_q, int64_t ldz,
                    const void* H_fp, const void* H_q, int64_t ldh, float tau, float lambda_kl, void* dZ_q, void* dH_q,
                    float* loss_out2, void* workspace, size_t workspace_bytes) {
  if (!ctx || !Z_fp || !Z_q || !H_fp || !H_q || !loss_out2) return FAAR_ERR_INVALID_ARG;
  if (!(tau > 0.f) || !isfinite(tau) || !isfinite(lambda_kl)) return FAAR_ERR_INVALID_ARG;
  if (T <= 0 || vocab <= 0 || hidden <= 0) return FAAR_ERR_SHAPE;
  if (ldz < ((int64_t)vocab + 7) / 8 * 8 || ldh < ((int64_t)hidden + 7) / 8 * 8) return FAAR_ERR_SHAPE;
  if (ldz % 8 || ldh % 8) return FAAR_ERR_ALIGN;
  if (!aligned16(Z_fp) || !aligned16(Z_q) || !aligned16(H_fp) || !aligned16(H_q) || (dZ_q && !aligned16(dZ_q)) ||
      (dH_q && !aligned16(dH_q)))
    return FAAR_ERR_ALIGN;
  size_t need = 0;
  int st = faar_align_loss_workspace_size(T, vocab, &need);
  if (st) return st;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need) return FAAR_ERR_WORKSPACE;
  FAAR_DEVICE_GUARD(ctx);
  float* kl_p = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace) + FAAR_WS_HEADER);
  float* mse_p = kl_p + (size_t)T;
  int np = 0;
  int e = faar_launch_align_loss(ctx, T, vocab, hidden, Z_fp, Z_q, ldz, H_fp, H_q, ldh, tau, lambda_kl, dZ_q, dH_q, kl_p,
                                 mse_p, &np);
  if (e) return cuda_fail(ctx, e);
  e = faar_launch_finalize(ctx, kl_p, np, (float)(1.0 / (double)T), loss_out2, mse_p, np, 1.0f, loss_out2 + 1);
  return cuda_fail(ctx, e);
}

int faar_harden_pack(faar_ctx* ctx, const faar_shape* s, const float* V, const uint8_t* code, const uint8_t* scales,
                     const float* s_global, uint8_t* packed, uint8_t* scales_out, uint8_t* decisions, void* W_final,
                     int wfinal_dtype) {
  if (!ctx || !V || !code || !scales || !packed) return FAAR_ERR_INVALID_ARG;
  int st = check_shape(s);
  if (st) return st;
  if (W_final && !s_global) return FAAR_ERR_INVALID_ARG;
  if (W_final && wfinal_dtype != FAAR_BF16 && wfinal_dtype != FAAR_F32) return FAAR_ERR_DTYPE;
  if (!aligned16(V) || !aligned16(code) || !aligned16(packed) || (W_final && !aligned16(W_final)))
    return FAAR_ERR_ALIGN;
  FAAR_DEVICE_GUARD(ctx);
  return cuda_fail(ctx, faar_launch_harden_pack(ctx, s, V, code, scales, s_global, packed, scales_out, decisions,
                                                W_final, wfinal_dtype));
}

}  // extern "C"
