/*
 * faar.h -- C ABI of libfaar.so: one FAAR layer-wise rounding-optimisation step
 * for a linear layer, on one NVIDIA B200 (sm_100a).
 *
 * The operations are the ones the paper's Procedure table lists for Stage 1
 * (steps 2-13) and for hardening (steps 25-26); each entry point below cites
 * the step / equation it implements.
 *
 * Conventions
 *   - nn.Linear orientation: W[O,K] row-major (K contiguous), X[T,K], Y[T,O] = X W^T.
 *     N = O*K is the number of quantised weights of the layer.  NVFP4 scale
 *     blocks are 16 consecutive elements along K; K % 16 == 0 is required.
 *   - Every tensor argument is a caller-owned DEVICE pointer unless it says
 *     "host".  The library never allocates device memory: scratch comes from
 *     the caller's `workspace` (size from faar_workspace_size).  Hyper-
 *     parameters are passed by value in host structs.  Scalar results (losses,
 *     s_global) are written to device memory; no call synchronises the stream.
 *   - All work is enqueued on the context's stream.  A context is not
 *     thread-safe.  V, adam_m, adam_u are updated in place.
 *   - Every function returns an int status (FAAR_OK == 0).  Nothing throws or
 *     aborts.  On a device that is not sm_100 every compute call returns
 *     FAAR_ERR_ARCH; there is no CPU fallback.
 *   - The tensor-core kernels bound every wait on a barrier.  If a wait gives
 *     up, the kernel records a code in the workspace status word, releases its
 *     tensor memory and returns; faar_check_status reports it as
 *     FAAR_ERR_TIMEOUT after the caller has synchronised the stream.  The
 *     status word is sticky and the workspace's counters may be left half
 *     updated: after FAAR_ERR_TIMEOUT call faar_workspace_init before the
 *     workspace is used again (results of the call that timed out are invalid).
 *   - The soft weights of Eq. 2 are not generated inside the forward GEMM:
 *     each step a separate kernel (or the previous step's backward epilogue,
 *     see faar_hparams.beta_next) writes them once as a BF16 operand [O,K] into
 *     the workspace, and the forward GEMM reads that operand by TMA.  Generating
 *     the operand inside the GEMM would re-evaluate Eq. 3 once per token tile
 *     (T/256 times per weight), which costs more than the 2 bytes per weight of
 *     the round trip.
 *
 * Packed formats
 *   code   [O, K/2] u8: element 2j in bits 3:0, element 2j+1 in bits 7:4 of byte j;
 *          nibble = sign<<3 | k, k in 0..6 the index of the LOWER bracketing node
 *          in (0, 0.5, 1, 1.5, 2, 3, 4, 6) -- i.e. the E2M1 code of that node.
 *   scales [O, K/16] u8: FP8 E4M3 block scales, linear row-major.
 *   packed [O, K/2] u8: same nibble order, nibble = sign<<3 | (k + v_hat): the
 *          deployable E2M1 weight code.
 */
#ifndef FAAR_H_
#define FAAR_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define FAAR_API __attribute__((visibility("default")))
#else
#define FAAR_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
  FAAR_OK = 0,
  FAAR_ERR_INVALID_ARG = 1, /* null pointer, bad enum, bad hyper-parameter      */
  FAAR_ERR_SHAPE = 2,       /* O/K/T <= 0, K % 16 != 0, leading dim too small,
                               K > 268 435 455 in the backward / step calls      */
  FAAR_ERR_ALIGN = 3,       /* pointer not 16-byte aligned / ld not multiple of 8 */
  FAAR_ERR_DTYPE = 4,
  FAAR_ERR_WORKSPACE = 5,   /* workspace null, misaligned or too small          */
  FAAR_ERR_ARCH = 6,        /* device is not compute capability 10.x            */
  FAAR_ERR_CUDA = 7,        /* a CUDA call failed; see faar_last_cuda_error     */
  FAAR_ERR_TIMEOUT = 8      /* a bounded device-side wait gave up               */
};

typedef struct faar_ctx faar_ctx;

typedef enum { FAAR_BF16 = 0, FAAR_F32 = 1 } faar_dtype;

/* Hyper-parameters of one step (host struct, by pointer, read at call time).
 * beta: temperature of Eq. 3, 0 < beta <= 1024 in the forward / backward / step calls (the BF16
 *   operand is rounded from an FP32 evaluation of Eq. 2/3 whose relative error is at most
 *   6e-7 + 7.5e-8 beta: 3e-6 at beta = 32; beyond 1024 Eq. 3 is a step function at BF16 precision and
 *   the hardened weights are the thing to use).  lambda_round: weight of the Round Loss in Eq. 5.
 * mse_scale: factor c on the squared Frobenius norm (the paper's Eq. 5 has c = 1).
 * opt: 0 = gradient descent, 1 = Adam (bias-corrected, no weight decay).
 * step: 1-based step index (Adam bias correction). */
typedef struct {
  float beta, lambda_round, mse_scale;
  int opt;
  float lr, beta1, beta2, eps;
  int step;
  /* FP32 tensor scale of quantised activations (faar_act_fakequant): the activation matrix passed to
   * the forward / backward calls then holds X_q / act_scale, and Y_q and the weight gradient are
   * multiplied by act_scale in the GEMM epilogues.  0 (or 1) = activations as given. */
  float act_scale;
  /* Chaining of consecutive steps on one workspace (both 0 = every step stands alone).  Eq. 2 is a
   * function of each weight's own v, so the backward pass, which holds the updated v' in registers,
   * can build the next step's forward operand on the way out.
   * beta_next > 0: the backward pass also writes, into the workspace, the BF16 forward operand
   *   W_soft(V', beta_next) of the NEXT step.
   * wsoft_ready != 0: the caller states that the previous backward (or step) call on this workspace
   *   was given beta_next == this step's beta and that V has not been touched since; the forward pass
   *   then reads that operand instead of rebuilding it from V (the soft-weights kernel is skipped).
   *   The context remembers the workspace and beta_next of its last backward call: wsoft_ready with
   *   another workspace or another beta is refused with FAAR_ERR_INVALID_ARG (a V that the caller
   *   changed in between cannot be detected).
   * The values, and so every result, are the same bit for bit either way. */
  float beta_next;
  int wsoft_ready;
} faar_hparams;

/* Layer geometry.  Leading dimensions are in ELEMENTS.
 * ldw : row stride of W[O,K]          (>= K)
 * ldx : row stride of X[T,K]          (>= K, multiple of 8)
 * ldxt: row stride of Xt[K,T] = X^T   (>= T, multiple of 8)
 * ldy : row stride of Y_ref[T,O] and of the optional Y_q output (>= O); with yref_transposed != 0
 *       both are stored as [O, ldy] (one row per output feature), ldy >= T rounded up to 16, so that
 *       the forward epilogue reads its target values as 16-byte vectors
 * V, code, scales, adam_m, adam_u, dV are dense (row strides K, K/2, K/16, K). */
typedef struct {
  int O, K, T;
  int64_t ldw, ldx, ldxt, ldy;
  int w_dtype;    /* faar_dtype of W      */
  int yref_dtype; /* faar_dtype of Y_ref  */
  int yref_transposed; /* 0: Y_ref[T,O]; 1: Y_ref stored as [O, ldy] */
} faar_shape;

/* ---- context -------------------------------------------------------------- */

/* Creates a context bound to `device` and to `stream` (a cudaStream_t, may be 0).
 * Returns FAAR_ERR_ARCH if the device is not sm_100.  Host memory only. */
FAAR_API int faar_create(faar_ctx** out, int device, void* stream);
FAAR_API int faar_destroy(faar_ctx* ctx);
FAAR_API int faar_set_stream(faar_ctx* ctx, void* stream);
FAAR_API const char* faar_status_string(int status);
/* Last cudaError_t seen by this context (0 if none). */
FAAR_API int faar_last_cuda_error(const faar_ctx* ctx);

/* ---- GEMM tiling (no counterpart in the paper: tuning and introspection of this library) -------
 * The tensor-core kernels cover the output with 256-row tiles whose width is chosen per launch (a
 * multiple of 16 in [128, 256]): the widest unless the problem is too small to give every CTA pair a
 * tile.  faar_tune_tile_n forces a width for the following launches on this context
 * (0 = automatic again).  faar_last_gemm_config reports the width and the number of CTA pairs of the
 * most recent GEMM launch (host out-pointers). */
FAAR_API int faar_tune_tile_n(faar_ctx* ctx, int bn);
/* The last, partly empty wave of tiles: the trailing tile columns can be cut into half-width tiles so
 * that more CTA pairs share it and the final, un-overlapped epilogue is half as long.  The number of
 * columns cut is chosen per launch from a cost model; faar_tune_tail_split forces it (-1 = automatic,
 * 0 = none).  faar_last_tail_split reports what the most recent GEMM launch used. */
FAAR_API int faar_tune_tail_split(faar_ctx* ctx, int columns);
FAAR_API int faar_last_tail_split(const faar_ctx* ctx, int* columns);
FAAR_API int faar_last_gemm_config(const faar_ctx* ctx, int* bn, int* cta_pairs);
/* On request a launch takes 256 x 512 tiles: the pair's whole tensor memory as one accumulator, a quarter less
 * operand traffic per flop, no overlap of a tile's epilogue with the next tile's main loop, no tail split.
 * mode: 1 = whenever the output has more than 256 columns and 256-wide tiles would have been used; 0 and -1
 * (the default) = never: measured, they win by a few per cent only for the forward GEMM of a large layer in a
 * short job and lose elsewhere.  faar_last_gemm_config reports bn = 512 for such a launch.  The per-weight
 * results (dW, V, moments) do not depend on the tile shape. */
FAAR_API int faar_tune_wide_tiles(faar_ctx* ctx, int mode);

/* Bytes of workspace that any call on this shape needs (host out-pointer).
 * The workspace must be 256-byte aligned.  Its first 256 bytes hold the status
 * word; the caller zeroes them once (faar_workspace_init) before first use. */
FAAR_API int faar_workspace_size(const faar_shape* shape, size_t* bytes);
/* Enqueues the zeroing of the workspace header (status word, counters). */
FAAR_API int faar_workspace_init(faar_ctx* ctx, void* workspace, size_t workspace_bytes);
/* Synchronises the context's stream and returns FAAR_ERR_TIMEOUT if a kernel
 * recorded a wait that gave up (detail_out, host, nullable: the raw code),
 * FAAR_ERR_CUDA if the stream is in error, else FAAR_OK. */
FAAR_API int faar_check_status(faar_ctx* ctx, const void* workspace, uint32_t* detail_out);

/* Self-test of the bounded waits (no counterpart in the paper).  Launches one small kernel whose only
 * wait can never be satisfied and whose limit is `limit_us` microseconds (1 .. 1 000 000): the wait gives
 * up, records code 0x700 in the workspace status word and the kernel exits normally, so a following
 * faar_check_status returns FAAR_ERR_TIMEOUT with that code and the context stays usable.  Re-arm with
 * faar_workspace_init. */
FAAR_API int faar_selftest_wait_timeout(faar_ctx* ctx, void* workspace, size_t workspace_bytes, unsigned int limit_us);

/* ---- per-kernel timing -------------------------------------------------------
 * (No counterpart in the paper: instrumentation of this library.)
 * Between faar_profile_begin and faar_profile_end every kernel the context
 * launches is bracketed by a pair of CUDA events on the context's stream.
 * faar_profile_end synchronises the stream and writes, per kernel id that ran,
 * the number of launches and the summed device time (host array `out` of
 * `capacity` entries; *count receives the number written).  Events are host
 * resources; no device memory is allocated. */
enum {
  FAAR_K_AMAX = 0,           /* max |W| reduction (part 1, pass 1)                */
  FAAR_K_SOFTQUANT_INIT = 1, /* scales, bracket, V_init (part 1, pass 2)          */
  FAAR_K_SOFT_WEIGHTS = 2,   /* Eq. 2/3 -> FP32 view and/or BF16 GEMM operand     */
  FAAR_K_GEMM_REF = 3,       /* Y_fp = X W^T                                      */
  FAAR_K_GEMM_FWD = 4,       /* forward GEMM + residual + dY                      */
  FAAR_K_GEMM_BWD = 5,       /* dW GEMM + dV + update                             */
  FAAR_K_ROUND_LOSS = 6,     /* stand-alone Round Loss partial sums               */
  FAAR_K_FINALIZE = 7,       /* fixed-order final sums of the loss partials       */
  FAAR_K_HARDEN_PACK = 8,
  FAAR_K_TRANSPOSE = 9,
  FAAR_K_ACT_FAKEQUANT = 10, /* activations to NVFP4 values (the X_q of Eq. 5)          */
  FAAR_K_ALIGN_LOSS = 11,    /* Eq. 6: KL of the softmaxes + last-hidden error, gradients */
  FAAR_K_GLUE = 12,          /* element-wise pieces of a decoder block between the linears */
  FAAR_K_NVFP4_GEMM = 13,    /* block-scaled FP4 GEMM on the deployable operands            */
  FAAR_K_ATTENTION = 14,     /* causal attention, forward or backward                       */
  FAAR_K_COUNT = 15
};
typedef struct {
  int kernel;     /* one of FAAR_K_*          */
  int launches;
  float total_ms; /* summed over the launches */
} faar_kernel_time;
FAAR_API int faar_profile_begin(faar_ctx* ctx);
FAAR_API int faar_profile_end(faar_ctx* ctx, faar_kernel_time* out, int capacity, int* count);
FAAR_API const char* faar_kernel_name(int kernel);

/* ---- part 1: soft-quantisation set-up, once per layer ----------------------
 * Procedure steps 2-5, "NVFP4 Overview", Eq. 4.
 * Computes the FP32 tensor scale (s_global = amax|W| / (6*448) unless
 * s_global_in > 0 is given), the E4M3 block scales s_g = E4M3(amax_block /
 * (6*s_global)) (round to nearest even, saturating at 448), and per weight the
 * normalised magnitude w~ = |w| / (s_g*s_global) clamped to 6, the index k of
 * the lower bracketing node (intervals half-open, the last closed), the sign
 * bit, and V_init = (w~ - lo) / (hi - lo).  All arithmetic IEEE binary32, one
 * correctly rounded operation at a time, so the byte outputs are reproducible.
 *   W           in : [O,K] (w_dtype, ldw)
 *   scales      out: [O,K/16] u8      s_global_out out: 1 float (device)
 *   code        out: [O,K/2] u8       V_init       out: [O,K] float */
FAAR_API int faar_softquant_init(faar_ctx* ctx, const faar_shape* shape, const void* W, float s_global_in,
                        uint8_t* scales, float* s_global_out, uint8_t* code, float* V_init,
                        void* workspace, size_t workspace_bytes);

/* ---- part 2: soft weights, FP32 view ---------------------------------------
 * Procedure steps 6-7, Eq. 2 and Eq. 3:  h = sigmoid(beta*(v-0.5)),
 * W_soft = sign*(lo + h*(hi-lo))*s_g*s_global, evaluated in FP32.  W_soft_bf16
 * is that FP32 value rounded to nearest even: exactly the operand the forward
 * GEMM multiplies (faar_layer_fwd builds it with this same routine).  Any
 * output may be null.
 *   W_soft out: [O,K] float    h out: [O,K] float    W_soft_bf16 out: [O,K] bf16 */
FAAR_API int faar_softquant_eval(faar_ctx* ctx, const faar_shape* shape, const float* V, const uint8_t* code,
                        const uint8_t* scales, const float* s_global, float beta,
                        float* W_soft, float* h, void* W_soft_bf16);

/* Debug view of the forward GEMM's operand (no counterpart in the paper): the FP32 value of Eq. 2 that
 * the soft-weights kernel and the chained backward epilogue round to BF16, before that rounding.  It
 * comes from a cheaper evaluation of Eq. 3 than W_soft above (one FMA for the exponent, hardware 2^x and
 * reciprocal); its relative error against the exact value is at most 6e-7 + 7.5e-8 beta.
 *   W_operand out: [O,K] float */
FAAR_API int faar_softquant_operand_f32(faar_ctx* ctx, const faar_shape* shape, const float* V, const uint8_t* code,
                                        const uint8_t* scales, const float* s_global, float beta, float* W_operand);

/* ---- layout helper ----------------------------------------------------------
 * out[c, r] = in[r, c] for a BF16 matrix in[rows, cols] (ld_in) -> out[cols, rows]
 * (ld_out).  Used once per layer to build Xt = X^T, the K-major operand of the
 * dW GEMM (no counterpart in the paper: a storage choice of this library). */
FAAR_API int faar_transpose_bf16(faar_ctx* ctx, int rows, int cols, const void* in, int64_t ld_in,
                        void* out, int64_t ld_out);

/* ---- quantised activations -------------------------------------------------
 * The X_q of Eq. 5 ("Stage 1": the quantised output is X_q W_q).  The paper gives
 * no rule for X_q; reading taken: the weights' NVFP4 format and scale rule
 * (blocks of 16 along K, E4M3 block scales, FP32 tensor scale = amax / (6*448)
 * unless s_global_in > 0), every value to its nearest node, a tie to the larger
 * magnitude.  Xq_units receives sign * node * block scale (exact in BF16); the
 * quantised activations are Xq_units * *s_global_out.  Pass Xq_units (and its
 * transpose) as X / Xt and the tensor scale as faar_hparams.act_scale.
 *   X in: [T,K] bf16 (ldx, multiple of 8)      Xq_units out: [T,K] bf16 (ldq, multiple of 8)
 *   s_global_out out: 1 float (device)
 *   packed out: [T,K/2] u8 E2M1 codes, nullable   scales out: [T,K/16] u8 E4M3, nullable */
FAAR_API int faar_act_fakequant(faar_ctx* ctx, int T, int K, const void* X, int64_t ldx, float s_global_in,
                                void* Xq_units, int64_t ldq, float* s_global_out, uint8_t* packed,
                                uint8_t* scales, void* workspace, size_t workspace_bytes);

/* ---- frozen target ----------------------------------------------------------
 * Procedure step 8: Y_fp = X W^T with the original BF16 weights (w_dtype must
 * be FAAR_BF16, ldw multiple of 8), FP32 accumulation on the tensor cores,
 * written as yref_dtype to Y_ref[T,O] (ldy). */
FAAR_API int faar_layer_ref(faar_ctx* ctx, const faar_shape* shape, const void* X, const void* W, void* Y_ref,
                   void* workspace, size_t workspace_bytes);

/* ---- part 3: forward GEMM + MSE ---------------------------------------------
 * Procedure steps 6-10, first term of Eq. 5.  Builds W_soft (Eq. 2, rounded to
 * BF16), computes Y_q = X W_soft^T on the tensor cores with FP32 accumulation,
 * r = Y_q - Y_ref, L_MSE = mse_scale * sum r^2 and dY = 2*mse_scale*r.
 *   X        in : [T,K] bf16 (ldx)           Y_ref in: [T,O] (yref_dtype, ldy)
 *   dYt      out: [O, ceil8(T)] bf16, dY transposed (row stride = T rounded up to 8)
 *   loss_mse out: 1 float (device)           Y_q out: [T,O] bf16 (ldy), nullable */
FAAR_API int faar_layer_fwd(faar_ctx* ctx, const faar_shape* shape, const faar_hparams* hp, const void* X,
                   const void* Y_ref, const float* V, const uint8_t* code, const uint8_t* scales,
                   const float* s_global, void* dYt, float* loss_mse, void* Y_q,
                   void* workspace, size_t workspace_bytes);

/* ---- input gradient (towards full-model alignment) ----------------------------
 * Procedure steps 16-23 train the rounding variables of all layers through the
 * whole model; a layer must then also pass the gradient on to its input:
 * dX = dY W_soft (the derivative of Y_q = X W_soft^T, W_soft as in faar_layer_fwd).
 * Soft weights (into the workspace) and one tensor-core GEMM that reads them untransposed, with the
 * output-feature index as the contraction row.
 *   dY     in : [T,O] bf16 (ldy, multiple of 8)      dX out: [T,K] bf16 (ldx, multiple of 8)
 *   WsoftT: not used (earlier versions transposed the soft weights into it); may be null */
FAAR_API int faar_layer_dx(faar_ctx* ctx, const faar_shape* shape, float beta, const void* dY, const float* V,
                           const uint8_t* code, const uint8_t* scales, const float* s_global, void* WsoftT,
                           void* dX, void* workspace, size_t workspace_bytes);

/* The same input gradient from soft weights that already exist: within one alignment step (Procedure steps
 * 16-23) a layer's rounding variables change only in its own update, which follows its input gradient, so the
 * BF16 soft weights its forward product was formed with (faar_softquant_eval's W_soft_bf16) are still the ones
 * Eq. 2 gives, and dX = dY W_soft needs the GEMM alone.
 *   dY    in : [T,O] bf16 (ldy, multiple of 8)      Wsoft in: [O,K] bf16 (row stride ldw, multiple of 8), read
 *   dX    out: [T,K] bf16 (ldx, multiple of 8)                untransposed; caller-owned device memory
 * Errors as faar_layer_dx (null pointer, shape, alignment, workspace too small). */
FAAR_API int faar_layer_dx_operand(faar_ctx* ctx, const faar_shape* shape, const void* dY, const void* Wsoft,
                                   void* dX, void* workspace, size_t workspace_bytes);

/* ---- the MLP's gated product ---------------------------------------------------
 * Procedure step 1 runs Stage 1 "for each layer": the input of a block's down
 * projection is the frozen model's own activation silu(H W_gate^T) * (H W_up^T),
 * silu(x) = x / (1 + e^-x).  This call forms it from the two GEMM outputs
 * (faar_layer_ref) so that the calibration input never leaves the device.  FP32
 * arithmetic, BF16 in and out.
 *   gate, up in: [rows, cols] bf16 (ldg, ldu)     out: [rows, cols] bf16 (ldo); may alias gate or up
 * cols and the leading dimensions are multiples of 8, the bases 16-byte aligned. */
FAAR_API int faar_silu_mul(faar_ctx* ctx, int rows, int cols, const void* gate, int64_t ldg, const void* up,
                           int64_t ldu, void* out, int64_t ldo);

/* ---- part 4: Round Loss, backward, update -----------------------------------
 * Eq. 5, second term without lambda: L_round = (1/N) sum (1 - (2v-1)^2).
 *   V in: N floats     loss_round out: 1 float (device) */
FAAR_API int faar_round_loss(faar_ctx* ctx, const float* V, int64_t N, float* loss_round,
                    void* workspace, size_t workspace_bytes);

/* The same Round Loss for callers that cannot allocate device memory (no
 * counterpart in the paper: a deployment variant of faar_round_loss).  Meant for
 * code that is handed raw device pointers and nothing else -- a plugin inside
 * another runtime's memory pool, a serving loop in which cudaMalloc is forbidden
 * or would stall the device -- and so has no workspace to give.  The partial
 * sums live in a fixed 256 KB array inside the library's device image instead
 * (one copy per GPU that loads the library, held until the process exits); the
 * call allocates nothing, on the device or through any library.
 *   V in: N floats, 16-byte aligned     loss_round out: 1 float (device)
 * Limit: N <= faar_round_loss_static_max_n() (268 435 456 = 65536 partials x 4096
 * elements); a larger N returns FAAR_ERR_SHAPE and launches nothing.
 * The first call on each device looks up the array's device address
 * (cudaGetSymbolAddress, with that device current); make that first call before
 * any stream capture begins.  Every call on a device uses the same array and
 * overwrites the slots it later reads, so nothing needs clearing between calls,
 * but two calls that overlap on the GPU (different streams, no ordering between
 * them) race on it: order them.  One partial per 4096 consecutive elements, so
 * the result does not depend on the device's SM count. */
FAAR_API int faar_round_loss_static(faar_ctx* ctx, const float* V, int64_t N, float* loss_round);
FAAR_API int64_t faar_round_loss_static_max_n(void);

/* Procedure step 13 with the clip that Stage 1 prescribes.  G = dY^T X on the
 * tensor cores (contraction over T), then per weight
 *   dV = G*sign*s*(hi-lo)*beta*h*(1-h) + (lambda_round/N)*(4-8v)
 * (the derivative of Eq. 5 through Eq. 2 and Eq. 3), the optimiser update and
 * v <- clamp(v, 0, 1).  All of it at the pre-update V.
 *   dYt in: [O, ceil8(T)] bf16 (from faar_layer_fwd)   Xt in: [K,T] bf16 (ldxt)
 *   V in/out: [O,K] float    adam_m, adam_u in/out: [O,K] float (null for opt 0)
 *   dV out: [O,K] float, nullable */
FAAR_API int faar_layer_bwd(faar_ctx* ctx, const faar_shape* shape, const faar_hparams* hp, const void* dYt,
                   const void* Xt, float* V, const uint8_t* code, const uint8_t* scales,
                   const float* s_global, float* adam_m, float* adam_u, float* dV,
                   void* workspace, size_t workspace_bytes);

/* faar_layer_bwd on the operands as a model's backward pass holds them: dY [T, ldy] and X [T, ldx], one row
 * per token (BF16; shape->ldy >= O, shape->ldx >= K, both multiples of 8; bases 16-byte aligned), no transposed
 * copies.  The tensor cores read both operands with the token index as the contraction row.  Everything else
 * as faar_layer_bwd; the results are the same bits (each dW element is the same sum in the same order).  The
 * GEMM itself takes the same time as on transposed operands (measured on four decoder-block shapes at 8192
 * tokens), so what is saved is the two transposes: 17-30 % of a linear's backward pass. */
FAAR_API int faar_layer_bwd_rowmajor(faar_ctx* ctx, const faar_shape* shape, const faar_hparams* hp, const void* dY,
                   const void* X, float* V, const uint8_t* code, const uint8_t* scales,
                   const float* s_global, float* adam_m, float* adam_u, float* dV,
                   void* workspace, size_t workspace_bytes);

/* Forward, Round Loss and backward + update back to back: one pass of Procedure
 * steps 6-13.  loss_out2 (device) receives {L_MSE, L_round}, both at the
 * pre-update V.  dYt lives in the workspace.  With hp->beta_next / hp->wsoft_ready
 * (see faar_hparams) a loop of steps builds each step's soft weights inside the
 * previous step's backward pass: two kernels per step instead of three. */
FAAR_API int faar_layer_step(faar_ctx* ctx, const faar_shape* shape, const faar_hparams* hp, const void* X,
                    const void* Xt, const void* Y_ref, float* V, const uint8_t* code,
                    const uint8_t* scales, const float* s_global, float* adam_m, float* adam_u,
                    float* loss_out2, void* workspace, size_t workspace_bytes);

/* faar_layer_step for a calibration batch that lives in HOST memory (ideally
 * pinned): copies X_host[T,K] (ldx) and Y_ref_host (the layout the shape declares)
 * into the caller's device staging buffers X_dev / Yref_dev, rebuilds
 * Xt_dev = X^T [K, ldxt], runs the step, and copies {L_MSE, L_round} back to
 * loss_host2.  Y_ref_host may be null: the batch's frozen target is then computed
 * on the device from the copied X and the layer's original BF16 weights W [O,K]
 * (ldw; Procedure step 8, as faar_layer_ref) instead of crossing the bus, and W
 * must be given; with Y_ref_host given W is not read and may be null.
 * Everything is ordered with the context's stream; loss_host2 is valid after the
 * caller synchronises it.  Bytes moved: T*K*2 (+ T*O*sizeof(yref_dtype) with
 * Y_ref_host) in, 8 out.  Every argument is validated before the first copy is
 * enqueued, so a refused call leaves the staging buffers untouched.
 * The host-to-device copies run on a copy stream that the context creates on
 * the first call (with three events: host resources, no device memory).  A
 * caller that alternates between two sets of staging buffers (X_dev, Xt_dev,
 * Yref_dev) on consecutive calls gets the copy of batch n+1 overlapped with step
 * n; with a single set the copy waits for the previous step.  After a change of
 * the context's stream (faar_set_stream) synchronise before the next call. */
FAAR_API int faar_layer_step_host(faar_ctx* ctx, const faar_shape* shape, const faar_hparams* hp,
                                  const void* X_host, const void* Y_ref_host, const void* W, void* X_dev,
                                  void* Xt_dev, void* Yref_dev, float* V, const uint8_t* code, const uint8_t* scales,
                                  const float* s_global, float* adam_m, float* adam_u, float* loss_dev2,
                                  float* loss_host2, void* workspace, size_t workspace_bytes);

/* The inverse of faar_act_fakequant's packed output: out[r][c] = sign * E2M1 node * E4M3 block scale as BF16
 * (exact; the FP32 tensor scale stays outside), from packed [rows, K/2] nibbles (8-byte aligned) and scales
 * [rows, K/16] bytes, both dense.  out: [rows, ld] bf16, ld >= K, multiple of 8, 16-byte aligned.  K % 16 == 0. */
FAAR_API int faar_nvfp4_expand(faar_ctx* ctx, int rows, int K, const void* packed, const void* scales, void* out,
                               int64_t ld);

/* faar_layer_step_host for quantised activations (the X_q of Eq. 5): the batch crosses the bus as the packed
 * NVFP4 codes and block scales that faar_act_fakequant produced (4.5 bits per value instead of 16), together
 * with its frozen target Y_ref (computed from the unquantised X, Procedure step 8, so it cannot be rebuilt
 * from what arrives).  On the device the batch is expanded into Xq_dev [T, ldx] (faar_nvfp4_expand) and the
 * step runs on it with hp->act_scale = the batch's FP32 tensor scale (required, > 0); the dW GEMM reads
 * Xq_dev with the token index as its contraction row, so no transposed copy is built.
 *   Xpacked_host [T, K/2], Xscales_host [T, K/16]: host (ideally pinned), dense
 *   Xpacked_dev, Xscales_dev, Xq_dev, Yref_dev: the caller's device staging buffers (16-byte aligned)
 * Bytes moved: T*K*9/16 + T*O*sizeof(yref_dtype) in, 8 out.  Stream order, validation before the first copy
 * and the alternation of two staging sets are as for faar_layer_step_host. */
FAAR_API int faar_layer_step_host_nvfp4(faar_ctx* ctx, const faar_shape* shape, const faar_hparams* hp,
                   const void* Xpacked_host, const void* Xscales_host, const void* Y_ref_host,
                   void* Xpacked_dev, void* Xscales_dev, void* Xq_dev, void* Yref_dev, float* V,
                   const uint8_t* code, const uint8_t* scales, const float* s_global, float* adam_m,
                   float* adam_u, float* loss_dev2, float* loss_host2, void* workspace, size_t workspace_bytes);

/* ---- part 5: harden + pack ---------------------------------------------------
 * Procedure steps 25-26, Eq. 7: v_hat = (v >= 0.5); weight code = k + v_hat.
 *   packed     out: [O,K/2] u8           scales_out out: [O,K/16] u8 (copy; nullable)
 *   decisions  out: [O,K/8] u8 bitmask, element 8j+i in bit i of byte j (nullable)
 *   W_final    out: [O,K] of wfinal_dtype = sign*node*s_g*s_global (nullable) */
FAAR_API int faar_harden_pack(faar_ctx* ctx, const faar_shape* shape, const float* V, const uint8_t* code,
                     const uint8_t* scales, const float* s_global, uint8_t* packed,
                     uint8_t* scales_out, uint8_t* decisions, void* W_final, int wfinal_dtype);

/* ---- full-model alignment loss (towards Stage 2) --------------------------------
 * Eq. 6 / Procedure steps 18-20: P_fp = softmax(Z_fp / tau), P_q = softmax(Z_q / tau)
 * over the vocabulary; L_KL = KL(P_fp || P_q) summed over the vocabulary and averaged
 * over the T tokens (the paper gives no reduction over tokens); L_MSE = the squared
 * Frobenius norm of H_fp - H_q.  Also the gradients towards the quantised model's
 * outputs, which its backward pass starts from:
 *   dZ_q = lambda_kl (P_q - P_fp) / (tau T)      dH_q = 2 (H_q - H_fp)
 * (the Round Loss term of Eq. 6 is per layer: faar_round_loss / the backward epilogue).
 *   Z_fp, Z_q in : [T, vocab] bf16, row stride ldz      dZ_q out: same layout, nullable
 *   H_fp, H_q in : [T, hidden] bf16, row stride ldh     dH_q out: same layout, nullable
 *   loss_out2 out: {L_KL, L_MSE} (device)
 * ldz, ldh: multiples of 8 and at least the column count rounded up to 8 (the kernel
 * reads whole 16-byte vectors; padding columns are read, never written); all bases
 * 16-byte aligned.  The workspace (faar_align_loss_workspace_size, 256-byte aligned,
 * header zeroed once by faar_workspace_init) holds the per-CTA partial sums. */
FAAR_API int faar_align_loss_workspace_size(int T, int vocab, size_t* bytes);
FAAR_API int faar_align_loss(faar_ctx* ctx, int T, int vocab, int hidden, const void* Z_fp, const void* Z_q,
                             int64_t ldz, const void* H_fp, const void* H_q, int64_t ldh, float tau, float lambda_kl,
                             void* dZ_q, void* dH_q, float* loss_out2, void* workspace, size_t workspace_bytes);

/* ---- deployable scale-factor layout ---------------------------------------
 * "Hardening and Inference": the final weights are "directly deployable on NVFP4
 * hardware".  Block-scaled tensor-core GEMMs read the E4M3 block scales not
 * row-major but in 128-row x 4-column tiles of 512 bytes (tiles of a row band
 * one after another; byte (r, c) of a tile at (r%32)*16 + (r/32)*4 + c; the
 * matrix zero-padded to multiples of 128 rows and 4 columns).  This call
 * rewrites linear scales [rows, cols] (from faar_harden_pack or
 * faar_act_fakequant; cols = K/16) into that order.
 *   scales in: [rows, cols] u8      scales_tiled out: ceil(rows/128)*ceil(cols/4)*512 bytes
 *   (tiled_bytes: size of the output buffer; too small is FAAR_ERR_SHAPE) */
FAAR_API int faar_swizzle_scales(faar_ctx* ctx, int rows, int cols, const uint8_t* scales, uint8_t* scales_tiled,
                                 size_t tiled_bytes);

/* ---- element-wise pieces of a decoder block --------------------------------------
 * Procedure steps 16-23 run the whole quantised model forward and backward; between its linears sit the
 * block's own operations, which the paper takes from the model family (Llama 3 / Qwen 3).  These calls are
 * the ones that are not matrix products.  BF16 in and out, FP32 arithmetic; cols (and every leading
 * dimension) a multiple of 8, bases 16-byte aligned.
 *
 * faar_rmsnorm: y = x / sqrt(mean(x^2) + eps) * g over each row.
 *   x in: [rows, cols] bf16 (ldx)    g in: [cols] float    y out: [rows, cols] bf16 (ldy)
 *   rstd out: [rows] float = 1 / sqrt(mean(x^2) + eps), kept for the backward call (nullable)
 * faar_rmsnorm_bwd: gradient towards x (g is frozen): dx = rstd * (g dy - xh * mean(g dy xh)), xh = x rstd;
 *   `add` ([rows, cols] bf16, ldadd; nullable) is added to it: the gradient that reaches x past the norm, along
 *   the residual connection.  dx may alias add.
 * faar_add_rmsnorm: a residual connection followed by the next norm in one pass: sum = a + b (rounded to BF16
 *   and stored, [rows, cols] bf16, lds), y = rmsnorm(sum) from the rounded values, i.e. the results of faar_add
 *   followed by faar_rmsnorm bit for bit.  sum may alias a or b.
 * faar_rmsnorm_bwd_sum: faar_rmsnorm_bwd with dy = dy + dy2 + dy3 formed in FP32 (the gradients of the linears
 *   that read the norm's output meet here: q / k / v, gate / up); dy2, dy3 nullable ([rows, cols] bf16, same
 *   leading dimension lddy; dy3 without dy2 is FAAR_ERR_INVALID_ARG).
 * faar_rope: rotary position embedding, half-split pairing: in every head, element i < head_dim/2 pairs with
 *   element i + head_dim/2 and the pair of row t turns by positions[t] * theta^(-2 i / head_dim); inverse != 0
 *   turns the other way (the backward pass).  x, y: [rows, n_heads * head_dim]; y may alias x; head_dim % 16 == 0.
 * faar_silu_mul_bwd: gradients of faar_silu_mul: with s = sigmoid(gate), dgate = dout * up * s * (1 + gate (1 - s)),
 *   dup = dout * gate * s.  dgate may alias gate and dup may alias up.
 * faar_embedding: out[t, :] = table[tokens[t], :]; tokens are 32-bit ints on the device; a token outside
 *   [0, vocab) yields a row of zeros. */
FAAR_API int faar_rmsnorm(faar_ctx* ctx, int rows, int cols, const void* x, int64_t ldx, const float* g, float eps, void* y,
                          int64_t ldy, float* rstd);
FAAR_API int faar_rmsnorm_bwd(faar_ctx* ctx, int rows, int cols, const void* dy, int64_t lddy, const void* x, int64_t ldx,
                              const float* g, const float* rstd, const void* add, int64_t ldadd, void* dx, int64_t lddx);
FAAR_API int faar_add_rmsnorm(faar_ctx* ctx, int rows, int cols, const void* a, int64_t lda, const void* b, int64_t ldb,
                              void* sum, int64_t lds, const float* g, float eps, void* y, int64_t ldy, float* rstd);
FAAR_API int faar_rmsnorm_bwd_sum(faar_ctx* ctx, int rows, int cols, const void* dy, const void* dy2, const void* dy3,
                                  int64_t lddy, const void* x, int64_t ldx, const float* g, const float* rstd,
                                  const void* add, int64_t ldadd, void* dx, int64_t lddx);
FAAR_API int faar_rope(faar_ctx* ctx, int rows, int n_heads, int head_dim, const void* x, int64_t ldx, const int* positions,
                       float theta, int inverse, void* y, int64_t ldy);
FAAR_API int faar_silu_mul_bwd(faar_ctx* ctx, int rows, int cols, const void* dout, int64_t ldd, const void* gate,
                               int64_t ldg, const void* up, int64_t ldu, void* dgate, int64_t lddg, void* dup, int64_t lddu);
FAAR_API int faar_embedding(faar_ctx* ctx, int rows, int cols, int vocab, const void* table, int64_t ldt, const int* tokens,
                            void* out, int64_t ldo);

/* faar_add: out = a + b, element-wise on [rows, cols] BF16 matrices (residual connections; gradients that meet
 * at one tensor).  out may alias a or b. */
FAAR_API int faar_add(faar_ctx* ctx, int rows, int cols, const void* a, int64_t lda, const void* b, int64_t ldb, void* out,
                      int64_t ldo);

/* ---- attention of a decoder block -------------------------------------------------
 * Procedure steps 16-23 again: the model family's causal softmax attention with grouped key/value heads sits
 * between a block's q/k/v projections and its output projection, and Eq. 6's gradient passes through it.
 *   out[t, h, :] = sum over u <= t of the same sequence of softmax_u(q[t, h, :] . k[u, g, :] / sqrt(head_dim)) v[u, g, :]
 * with g = h / (n_heads / n_kv_heads).  Tokens of a sequence are contiguous rows: row = sequence * seq + position.
 *   q in: [batch*seq, n_heads*head_dim] bf16 (ldq)     k, v in: [batch*seq, n_kv_heads*head_dim] bf16 (ldkv)
 *   out: [batch*seq, n_heads*head_dim] bf16 (ldo)      lse out: [batch, n_heads, seq] float, log2 of each row's
 *   sum of 2^(score log2 e / sqrt(head_dim)): what the backward call recomputes the probabilities from.
 * faar_attention_bwd: from dout (layout of out) to dq (layout of q), dk, dv (layout of k, v); out and lse are the
 * forward call's; dsum is scratch, [batch, n_heads, seq] floats.  No matrix of seq x seq values is stored; results
 * are reproducible (no atomics).  head_dim is 64 or 128; leading dimensions multiples of 8, bases 16-byte aligned. */
/* Which kernels head_dim 64 takes (head_dim 128 always takes the third kind):
 *   0 (default): forward, dQ and dK / dV kernels on the tcgen05 tensor cores (scores in tensor memory, one query or
 *      key row per thread or pair of threads, gradients accumulated in tensor memory over the sweep);
 *   2: forward and backward with scores and probabilities in registers (mma.sync m16n8k16, one sweep over the
 *      keys with a running maximum);
 *   1: kernels that pass scores and probabilities through shared memory as 16 x 16 fragments (two sweeps in the
 *      forward pass).
 * The same mathematics in all three, used to test them against each other and the definition. */
FAAR_API int faar_tune_attention(faar_ctx* ctx, int mode);
/* The tcgen05 attention kernel bounds its barrier waits like the GEMM kernels; a wait that gave up is recorded in
 * a status word of the library, which this call reads and clears (after the caller has synchronised the stream):
 * FAAR_ERR_TIMEOUT with the raw code in detail_out (host, nullable), else FAAR_OK. */
FAAR_API int faar_attention_status(faar_ctx* ctx, uint32_t* detail_out);
FAAR_API int faar_attention_fwd(faar_ctx* ctx, int batch, int seq, int n_heads, int n_kv_heads, int head_dim, const void* q,
                                int64_t ldq, const void* k, const void* v, int64_t ldkv, void* out, int64_t ldo, float* lse);
FAAR_API int faar_attention_bwd(faar_ctx* ctx, int batch, int seq, int n_heads, int n_kv_heads, int head_dim, const void* q,
                                int64_t ldq, const void* k, const void* v, int64_t ldkv, const void* out, const void* dout,
                                int64_t ldo, const float* lse, float* dsum, void* dq, void* dk, void* dv);

/* ---- GEMM on the deployable operands -----------------------------------------
 * "Hardening and Inference": the hardened weights are NVFP4 tensors that the hardware multiplies as they
 * are.  This call does that on the block-scaled FP4 tensor-core path: C = (sA sB) A B^T, every element of A
 * and B being sign * E2M1 node * E4M3 block scale (blocks of 16 along K), FP32 accumulation, BF16 result.
 * With A = the quantised activations (faar_act_fakequant: packed, scales, s_global_out) and B = the
 * hardened weights (faar_harden_pack: packed, scales_out; s_global of faar_softquant_init), both scale
 * arrays rewritten by faar_swizzle_scales, C[T,O] is the quantised layer's output X_q W_final^T.
 *   A_packed in: [M, K/2] u8      A_scales_tiled in: ceil(M/128)*ceil(K/64)*512 bytes      A_s_global in: 1 float (device)
 *   B_packed in: [N, K/2] u8      B_scales_tiled in: ceil(N/128)*ceil(K/64)*512 bytes      B_s_global in: 1 float (device)
 *   C out: [M, N] bf16, row stride ldc >= N
 * K must be a multiple of 32 (rows of K/2 bytes are read by TMA: 16-byte row pitch); all four operand
 * arrays 16-byte aligned.  The workspace needs the 256-byte header only (status word of the bounded waits). */
FAAR_API int faar_nvfp4_gemm(faar_ctx* ctx, int M, int N, int K, const uint8_t* A_packed, const uint8_t* A_scales_tiled,
                             const float* A_s_global, const uint8_t* B_packed, const uint8_t* B_scales_tiled,
                             const float* B_s_global, void* C, int64_t ldc, void* workspace, size_t workspace_bytes);

#ifdef __cplusplus
}
#endif
#endif /* FAAR_H_ */
