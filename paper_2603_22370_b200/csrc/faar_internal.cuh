// Internal declarations shared by the translation units of libfaar.so.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "faar.h"

#include <vector>

constexpr int FAAR_GEMM_VARIANTS = 8;     // REF, FWD, BWD x 4 optimiser / chaining variants

struct faar_ctx {
  int device;
  int num_sms;
  cudaStream_t stream;
  int last_cuda_error;
  void* encode_tiled;  // cuTensorMapEncodeTiled, resolved through the runtime
  int tune_bn;                            // 0 = choose the GEMM tile width automatically
  int tune_tail;                          // -1 = choose the tail split automatically, else columns to split
  int tune_wide;                          // 1 = 256 x 512 GEMM tiles wherever the shape allows; -1 (default), 0 = never
  int tune_attention_fragments;           // head_dim 64 attention: 0 = tcgen05 kernels, 2 = mma.sync kernels, 1 = the shared-memory fragment kernels
  int last_gemm_bn, last_gemm_pairs, last_gemm_split;   // what the last GEMM launch used
  // CTA pairs this context's device can hold at once, per GEMM kernel instantiation (0 = not asked yet)
  int gemm_max_pairs[FAAR_GEMM_VARIANTS];
  // chained steps: the workspace and the beta of the forward operand that the last backward call wrote
  const void* wsoft_ws;
  float wsoft_beta;
  // host-batch path (faar_layer_step_host): copies run on their own stream, ordered by events
  cudaStream_t copy_stream;
  cudaEvent_t ev_copied, ev_done[2];
  unsigned long long host_calls;
  const void* last_staging;
  // per-kernel timing (faar_profile_begin / faar_profile_end)
  bool prof_on;
  int prof_used;                          // event pairs used since faar_profile_begin
  std::vector<cudaEvent_t> prof_events;   // 2 per launch: start, stop
  std::vector<int> prof_kernel;           // kernel id per pair
};

// Brackets one kernel launch with a pair of CUDA events when profiling is on.
struct faar_prof_scope {
  faar_ctx* c;
  int pair;
  faar_prof_scope(faar_ctx* ctx, int kernel_id);
  ~faar_prof_scope();
};

// ---- workspace layout -------------------------------------------------------
// [0, 256)            header: word 0 = status (0 = ok), word 2 = count of dW-GEMM
//                     CTAs that have finished (zero between launches), bytes 16..23 = tensor maximum of
//                     the last set-up pass (high word: the pass's serial number, low word: max |W| bits)
// [256, 256+P)        loss partials (float): MSE region then Round region
// [..]                W_soft bf16 [O,K]
// [..]                dYt bf16 [O, ceil8(T)]
constexpr size_t FAAR_WS_HEADER = 256;
constexpr int FAAR_MAX_PARTIALS = 16384;  // per loss term

struct faar_ws_layout {
  size_t off_mse_partials, off_round_partials, off_wsoft, off_dyt, total;
  int64_t ld_dyt;
};

static inline size_t faar_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static inline faar_ws_layout faar_ws_plan(const faar_shape* s) {
  faar_ws_layout l;
  l.ld_dyt = ((int64_t)s->T + 7) / 8 * 8;
  size_t off = FAAR_WS_HEADER;
  l.off_mse_partials = off;
  off += sizeof(float) * FAAR_MAX_PARTIALS;
  l.off_round_partials = off;
  off += sizeof(float) * FAAR_MAX_PARTIALS;
  off = faar_align_up(off, 1024);
  l.off_wsoft = off;
  off += (size_t)s->O * (size_t)s->K * 2;
  off = faar_align_up(off, 1024);
  l.off_dyt = off;
  off += (size_t)s->O * (size_t)l.ld_dyt * 2;
  l.total = faar_align_up(off, 1024);
  return l;
}

// ---- launchers (each returns a cudaError_t as int) ---------------------------
int faar_launch_softquant_init(faar_ctx*, const faar_shape*, const void* W, float s_global_in,
                               uint8_t* scales, float* s_global_out, uint8_t* code, float* V,
                               unsigned long long* amax_word);
int faar_launch_nvfp4_expand(faar_ctx*, int rows, int K, const uint8_t* packed, const uint8_t* scales, void* out, int64_t ld);
int faar_launch_attention_fwd64_tc(faar_ctx*, int B, int S, int H, int Hkv, const void* q, int64_t ldq, const void* k,
                                   const void* v, int64_t ldk, void* out, int64_t ldo, float* lse, float scale_log2);
int faar_launch_attention_dq64_tc(faar_ctx*, int B, int S, int H, int Hkv, const void* q, int64_t ldq, const void* k,
                                  const void* v, int64_t ldk, const void* dout, int64_t ldo, const float* lse,
                                  const float* dsum, void* dq, float scale_log2);
int faar_launch_attention_dkv64_tc(faar_ctx*, int B, int S, int H, int Hkv, const void* q, int64_t ldq, const void* k,
                                   const void* v, int64_t ldk, const void* dout, int64_t ldo, const float* lse,
                                   const float* dsum, void* dk, void* dv, float scale_log2);
int faar_attention_tc_status(uint32_t* code_out);
int faar_launch_softquant_eval(faar_ctx*, const faar_shape*, const float* V, const uint8_t* code,
                               const uint8_t* scales, const float* s_global, float beta,
                               float* W_soft, float* h, __nv_bfloat16* W_soft_bf16,
                               float* W_operand_f32 = nullptr);
int faar_launch_act_fakequant(faar_ctx*, int T, int K, const void* X, int64_t ldx, float s_global_in, void* Xq,
                              int64_t ldq, float* s_global_out, uint8_t* packed, uint8_t* scales,
                              unsigned long long* amax_word);
int faar_launch_transpose_bf16(faar_ctx*, int rows, int cols, const void* in, int64_t ld_in, void* out,
                               int64_t ld_out);
int faar_launch_swizzle_scales(faar_ctx*, int rows, int cols, const uint8_t* in, uint8_t* out);
// Eq. 6's data terms: one partial per CTA, at most one CTA per token
int faar_launch_align_loss(faar_ctx*, int T, int vocab, int hidden, const void* Z_fp, const void* Z_q, int64_t ldz,
                           const void* H_fp, const void* H_q, int64_t ldh, float tau, float lambda_kl, void* dZ_q,
                           void* dH_q, float* kl_partials, float* mse_partials, int* n_partials);
int faar_launch_silu_mul(faar_ctx*, int rows, int cols, const void* gate, int64_t ldg, const void* up, int64_t ldu,
                         void* out, int64_t ldo);
int faar_launch_rmsnorm(faar_ctx*, int rows, int cols, const void* x, int64_t ldx, const void* b, int64_t ldb,
                        void* sum_out, int64_t lds, const float* g, float eps, void* y, int64_t ldy, float* rstd);
int faar_launch_rmsnorm_bwd(faar_ctx*, int rows, int cols, const void* dy, const void* dy2, const void* dy3, int64_t lddy,
                            const void* x, int64_t ldx, const float* g, const float* rstd, const void* add, int64_t ldadd,
                            void* dx, int64_t lddx);
int faar_launch_rope(faar_ctx*, int rows, int n_heads, int head_dim, const void* x, int64_t ldx, const int* pos, float theta,
                     int inverse, void* y, int64_t ldy);
int faar_launch_silu_mul_bwd(faar_ctx*, int rows, int cols, const void* dout, int64_t ldd, const void* gate, int64_t ldg,
                             const void* up, int64_t ldu, void* dgate, int64_t lddg, void* dup, int64_t lddu);
int faar_launch_embedding(faar_ctx*, int rows, int cols, int vocab, const void* table, int64_t ldt, const int* tokens,
                          void* out, int64_t ldo);
int faar_launch_add(faar_ctx*, int rows, int cols, const void* a, int64_t lda, const void* b, int64_t ldb, void* out,
                    int64_t ldo);
int faar_launch_attention_fwd(faar_ctx*, int B, int S, int H, int Hkv, int D, const void* q, int64_t ldq, const void* k,
                              const void* v, int64_t ldk, void* out, int64_t ldo, float* lse);
int faar_launch_attention_bwd(faar_ctx*, int B, int S, int H, int Hkv, int D, const void* q, int64_t ldq, const void* k,
                              const void* v, int64_t ldk, const void* out, const void* dout, int64_t ldo, const float* lse,
                              float* dsum, void* dq, void* dk, void* dv);
int faar_launch_nvfp4_gemm(faar_ctx*, int M, int N, int K, const uint8_t* A, const uint8_t* sfa, const float* sa,
                           const uint8_t* B, const uint8_t* sfb, const float* sb, void* C, int64_t ldc, uint32_t* status);
int faar_launch_round_partials(faar_ctx*, const float* V, int64_t N, float* partials, int* n_partials);
// out[0] = scale0 * sum(p0[0..n0)), out[1] = scale1 * sum(p1[0..n1)) (either may have n = 0 -> skipped)
int faar_launch_finalize(faar_ctx*, const float* p0, int n0, float scale0, float* out0, const float* p1,
                         int n1, float scale1, float* out1);
int faar_launch_harden_pack(faar_ctx*, const faar_shape*, const float* V, const uint8_t* code,
                            const uint8_t* scales, const float* s_global, uint8_t* packed,
                            uint8_t* scales_out, uint8_t* decisions, void* W_final, int wfinal_dtype);

enum { FAAR_GEMM_REF = 0, FAAR_GEMM_FWD = 1, FAAR_GEMM_BWD = 2 };

struct faar_gemm_args {
  int mode;
  int M, N, Kc;           // C[M,N] = A[M,Kc] * B[N,Kc]^T, both operands bf16 with Kc contiguous
  const void* A; int64_t lda;
  const void* B; int64_t ldb;
  int a_mn, b_mn;         // 1: the operand is stored with M (N) contiguous instead: A[Kc, M] (lda), B[Kc, N] (ldb)
  uint32_t* status;       // workspace status word
  // REF / FWD
  void* Yout; int yout_dtype; int64_t ldy;     // [N(T), M(O)] written transposed; nullable in FWD
  const void* Yref; int yref_dtype;            // FWD
  int yref_t;                                  // REF, FWD: Y stored transposed [O, ldy]
  __nv_bfloat16* dYt; int64_t ld_dyt;          // FWD: [M(O), ld_dyt]
  float mse2c;                                 // FWD: 2 * mse_scale
  float act_scale;                             // FWD, BWD: tensor scale of quantised activations (1 = none)
  float* partials;                             // FWD: sum r^2 partials; BWD: Round Loss partials
  // BWD: M = O, N = K
  float* V; const uint8_t* code; const uint8_t* scales; const float* s_global;
  float* adam_m; float* adam_u; float* dV;
  float beta, lam_over_n, lr, b1, b2, eps, inv_bc1, inv_bc2; int opt;
  // BWD, optional: also write the next step's BF16 operand W_soft(V', beta_next) (null = not wanted)
  __nv_bfloat16* wsoft_next; float beta_next;
  // BWD, optional: final loss sums by the last CTA (fin_out2 null = not wanted)
  uint32_t* fin_counter; const float* fin_mse_partials; int fin_n_mse; float fin_scale_mse, fin_scale_round;
  float* fin_out2;
};
// n_partials_out: number of floats written to args.partials
int faar_launch_gemm(faar_ctx*, const faar_gemm_args*, int* n_partials_out);
int faar_gemm_max_partials(const faar_ctx*, int M, int N);
int faar_launch_wait_selftest(faar_ctx*, uint32_t* status, unsigned long long limit_ns);

// ---- device helpers -----------------------------------------------------------
#ifdef __CUDACC__

// E2M1 magnitude of code c (0..7): 0, .5, 1, 1.5, 2, 3, 4, 6.
__device__ __forceinline__ float faar_node(int c) {
  int e = c >> 1, m = c & 1;
  // e == 0: m * 0.5 ; else (1 + m/2) * 2^(e-1)
  float normal = __uint_as_float(((uint32_t)(e + 126) << 23) | ((uint32_t)m << 22));
  return e == 0 ? 0.5f * (float)m : normal;
}

// width of interval k (0..6): .5 .5 .5 .5 1 1 2
__device__ __forceinline__ float faar_width(int k) { return k < 4 ? 0.5f : (k < 6 ? 1.0f : 2.0f); }

// FP8 E4M3 byte -> float (finite codes only).
__device__ __forceinline__ float faar_e4m3_to_float(uint32_t b) {
  uint32_t e = (b >> 3) & 0xF, m = b & 7;
  float sub = (float)m * 0.001953125f;  // m * 2^-9
  float nor = __uint_as_float(((e + 120u) << 23) | (m << 20));
  return e == 0 ? sub : nor;
}

// Non-negative finite float -> nearest finite E4M3 byte, ties to even, saturating at 448.
__device__ __forceinline__ uint32_t faar_float_to_e4m3(float q) {
  if (!(q < 448.0f)) return 0x7Eu;
  if (q < 0.015625f) {                       // below 2^-6: fixed quantum 2^-9
    return (uint32_t)__float2int_rn(q * 512.0f);   // 0..8; 8 is the smallest normal
  }
  uint32_t bits = __float_as_uint(q);
  uint32_t lsb = (bits >> 20) & 1u;
  bits += 0x7FFFFu + lsb;                    // round to nearest even at bit 20
  bits &= 0xFFF00000u;
  if (bits > 0x43E00000u) return 0x7Eu;      // above 448
  uint32_t e = (bits >> 23) - 120u;
  uint32_t m = (bits >> 20) & 7u;
  return (e << 3) | m;
}

// Eq. 3 in FP32 with a relative error of a few 1e-7 over the whole range of h, also where h is tiny.
// z = beta*(v-0.5) is kept as an unevaluated sum (v-0.5 is exact or off by < 2^-26; the product's
// rounding error is recovered with one FMA), -|z|*log2(e) likewise, so the argument of the hardware
// 2^x carries no error that grows with |z|; the low parts enter as a first-order correction.
__device__ __forceinline__ float faar_sigmoid_precise(float beta, float v) {
  const float d = __fsub_rn(v, 0.5f);
  const float zh = __fmul_rn(beta, d);
  const float zl = __fmaf_rn(beta, d, -zh);              // exact error of the product
  const float az = -fabsf(zh);
  const float sl = zh >= 0.f ? -zl : zl;                  // low part of -|z| (sign follows zh)
  const float L1 = 1.4426950216293335f;                   // float(log2 e)
  const float L2 = 1.9259629911266175e-8f;                // log2 e - L1
  const float th = __fmul_rn(az, L1);
  float tl = __fmaf_rn(az, L1, -th);
  tl = __fmaf_rn(az, L2, tl);
  tl = __fmaf_rn(sl, L1, tl);
  float e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(th));
  e = __fmaf_rn(e, tl * 0.6931471805599453f, e);          // 2^(th+tl) = 2^th (1 + tl ln 2)
  const float hs = __fdividef(1.0f, 1.0f + e);            // sigmoid(|z|)
  return zh >= 0.f ? hs : __fmul_rn(e, hs);               // sigmoid(-|z|) = e / (1 + e)
}

// Eq. 3 as the forward GEMM's BF16 operand is built (relative error below 3e-6):
// h = 1 / (1 + 2^(-z log2 e)), z = beta (v - 0.5), with beta log2(e) rounded once, the exponent formed
// in one FMA, hardware 2^x and reciprocal.  A 2^x that overflows (z < -88) gives h = 0, the value's
// rounding.  nbl = -(beta * log2 e), hbl = -nbl / 2 (faar_operand_consts).
__device__ __forceinline__ void faar_operand_consts(float beta, float* nbl, float* hbl) {
  *nbl = -__fmul_rn(beta, 1.4426950408889634f);
  *hbl = -0.5f * *nbl;
}
__device__ __forceinline__ float faar_sigmoid_operand(float nbl, float hbl, float v) {
  float e, h;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(fmaf(nbl, v, hbl)));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(h) : "f"(1.0f + e));
  return h;
}
// The operand value before its rounding to BF16: (lo + h * width) * s with the sign of w, in exactly
// these operations wherever it is produced (soft-weights kernel, dW epilogue), so that both give the
// same bits.  lo and width may carry the sign already (rounding is symmetric).
__device__ __forceinline__ float faar_operand_weight(float h, float lo, float width, float s) {
  return fmaf(h, width, lo) * s;
}

// Eq. 2 in FP32: sign * (lo + h * (hi - lo)) * s for the nibble (sign<<3 | k).
__device__ __forceinline__ float faar_soft_weight(float h, uint32_t nib, float s) {
  int k = nib & 7;
  float mag = __fmul_rn(__fmaf_rn(h, faar_width(k), faar_node(k)), s);
  return (nib & 8) ? -mag : mag;
}

// Programmatic dependent launch: the step's kernels are launched with stream serialisation relaxed, so
// that a kernel's CTAs may start (and run their set-up) on SMs that the previous kernel has already
// left.  faar_pdl_sync() lets the next kernel do the same and then waits until the previous kernel has
// completed and its memory is visible; nothing before it may touch global data.
__device__ __forceinline__ void faar_pdl_sync() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ float faar_warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

#endif  // __CUDACC__
