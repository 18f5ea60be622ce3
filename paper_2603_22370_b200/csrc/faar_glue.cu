// Element-wise pieces of a decoder block that sit between the linears: what the layer-wise driver needs
// to produce each linear's calibration input on the device (the MLP's SiLU-gated product feeds down_proj),
// and what full-model alignment (Eq. 6, Procedure steps 15-23) needs around the tensor-core GEMMs.
// All of them are HBM-bound: BF16 in and out as 16-byte vectors, FP32 arithmetic in registers.
#include <math.h>

#include "faar_internal.cuh"

namespace {

constexpr int GL_THREADS = 256;

__device__ __forceinline__ void unpack8(const uint4& raw, float (&x)[8]) {
  const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    x[2 * i] = __uint_as_float(r[i] << 16);
    x[2 * i + 1] = __uint_as_float(r[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ uint4 pack8(const float (&x)[8]) {
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 p2 = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
    o[i] = *reinterpret_cast<uint32_t*>(&p2);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}

// sigmoid(x) in FP32: 1 / (1 + e^-x) with the library exponential (relative error ~1e-7) and an IEEE
// division; e^-x overflowing to +inf gives 0, the limit.
__device__ __forceinline__ float sigmoid_f32(float x) { return __fdiv_rn(1.0f, 1.0f + expf(-x)); }

// out = silu(gate) * up, silu(x) = x * sigmoid(x)
__global__ void __launch_bounds__(GL_THREADS)
silu_mul_kernel(const __nv_bfloat16* __restrict__ gate, int64_t ldg, const __nv_bfloat16* __restrict__ up, int64_t ldu,
                __nv_bfloat16* __restrict__ out, int64_t ldo, int rows, int cols) {
  const uint32_t groups_per_row = cols / 8;
  const int64_t total = (int64_t)rows * groups_per_row;
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = g / groups_per_row;
    const int col = (int)(g - row * groups_per_row) * 8;
    float a[8], b[8], y[8];
    unpack8(*reinterpret_cast<const uint4*>(gate + row * ldg + col), a);
    unpack8(*reinterpret_cast<const uint4*>(up + row * ldu + col), b);
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = a[i] * sigmoid_f32(a[i]) * b[i];
    *reinterpret_cast<uint4*>(out + row * ldo + col) = pack8(y);
  }
}

// ---- RMSNorm: y = x / sqrt(mean(x^2) + eps) * g, one warp per row ---------------------------------
// The row is read twice (sum of squares, then the scaled output); the second read hits L1/L2.
__global__ void __launch_bounds__(GL_THREADS)
rmsnorm_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, const float* __restrict__ g, float eps,
               __nv_bfloat16* __restrict__ y, int64_t ldy, float* __restrict__ rstd_out, int rows, int cols) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int n_groups = cols / 8;
  for (int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; row < rows; row += warps) {
    const __nv_bfloat16* xr = x + (int64_t)row * ldx;
    float ss = 0.f;
    for (int c = lane; c < n_groups; c += 32) {
      float a[8];
      unpack8(*reinterpret_cast<const uint4*>(xr + 8 * c), a);
#pragma unroll
      for (int i = 0; i < 8; ++i) ss = fmaf(a[i], a[i], ss);
    }
    ss = faar_warp_sum(ss);
    const float rstd = 1.0f / sqrtf(ss / (float)cols + eps);
    if (lane == 0 && rstd_out) rstd_out[row] = rstd;
    __nv_bfloat16* yr = y + (int64_t)row * ldy;
    for (int c = lane; c < n_groups; c += 32) {
      float a[8], o[8];
      unpack8(*reinterpret_cast<const uint4*>(xr + 8 * c), a);
      const float4 g0 = *reinterpret_cast<const float4*>(g + 8 * c), g1 = *reinterpret_cast<const float4*>(g + 8 * c + 4);
      const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) o[i] = a[i] * rstd * gg[i];
      *reinterpret_cast<uint4*>(yr + 8 * c) = pack8(o);
    }
  }
}

// Backward of RMSNorm towards x (the norm weights are frozen): with xh = x * rstd and w = g * dy,
// dx = rstd * (w - xh * mean(w * xh)), optionally added to `add` (the residual branch's gradient).
__global__ void __launch_bounds__(GL_THREADS)
rmsnorm_bwd_kernel(const __nv_bfloat16* __restrict__ dy, int64_t lddy, const __nv_bfloat16* __restrict__ x, int64_t ldx,
                   const float* __restrict__ g, const float* __restrict__ rstd_in, const __nv_bfloat16* __restrict__ add,
                   int64_t ldadd, __nv_bfloat16* __restrict__ dx, int64_t lddx, int rows, int cols) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int n_groups = cols / 8;
  for (int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; row < rows; row += warps) {
    const __nv_bfloat16* xr = x + (int64_t)row * ldx;
    const __nv_bfloat16* dr = dy + (int64_t)row * lddy;
    const float rstd = rstd_in[row];
    float dot = 0.f;
    for (int c = lane; c < n_groups; c += 32) {
      float a[8], d[8];
      unpack8(*reinterpret_cast<const uint4*>(xr + 8 * c), a);
      unpack8(*reinterpret_cast<const uint4*>(dr + 8 * c), d);
      const float4 g0 = *reinterpret_cast<const float4*>(g + 8 * c), g1 = *reinterpret_cast<const float4*>(g + 8 * c + 4);
      const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) dot = fmaf(d[i] * gg[i], a[i] * rstd, dot);
    }
    dot = faar_warp_sum(dot) / (float)cols;
    for (int c = lane; c < n_groups; c += 32) {
      float a[8], d[8], o[8], r[8];
      unpack8(*reinterpret_cast<const uint4*>(xr + 8 * c), a);
      unpack8(*reinterpret_cast<const uint4*>(dr + 8 * c), d);
      const float4 g0 = *reinterpret_cast<const float4*>(g + 8 * c), g1 = *reinterpret_cast<const float4*>(g + 8 * c + 4);
      const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
      if (add) unpack8(*reinterpret_cast<const uint4*>(add + (int64_t)row * ldadd + 8 * c), r);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        o[i] = rstd * fmaf(-(a[i] * rstd), dot, d[i] * gg[i]);
        if (add) o[i] += r[i];
      }
      *reinterpret_cast<uint4*>(dx + (int64_t)row * lddx + 8 * c) = pack8(o);
    }
  }
}

// ---- rotary position embedding, half-split pairing ----------------------------------------------
// Inside every head, element i (i < head_dim / 2) pairs with element i + head_dim / 2; the pair of token t is
// rotated by pos[t] * theta^(-2 i / head_dim) (by the negative angle with inverse != 0: the backward pass of
// an orthogonal map).  One thread takes 8 consecutive i of one head of one token.
__global__ void __launch_bounds__(GL_THREADS)
rope_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, const int* __restrict__ pos, __nv_bfloat16* __restrict__ y,
            int64_t ldy, int rows, int n_heads, int head_dim, float log2_theta, int inverse) {
  const int half = head_dim / 2, gph = half / 8;                    // 8-element groups per half head
  const int64_t total = (int64_t)rows * n_heads * gph;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
    const int gi = (int)(t % gph);
    const int head = (int)((t / gph) % n_heads);
    const int64_t row = t / ((int64_t)gph * n_heads);
    const int64_t off = (int64_t)head * head_dim + 8 * gi;
    float a[8], b[8], oa[8], ob[8];
    unpack8(*reinterpret_cast<const uint4*>(x + row * ldx + off), a);
    unpack8(*reinterpret_cast<const uint4*>(x + row * ldx + off + half), b);
    const float p = (float)pos[row];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float inv_freq = exp2f(-2.0f * (float)(8 * gi + i) / (float)head_dim * log2_theta);
      float sn, cs;
      sincosf(p * inv_freq, &sn, &cs);
      if (inverse) sn = -sn;
      oa[i] = a[i] * cs - b[i] * sn;
      ob[i] = b[i] * cs + a[i] * sn;
    }
    *reinterpret_cast<uint4*>(y + row * ldy + off) = pack8(oa);
    *reinterpret_cast<uint4*>(y + row * ldy + off + half) = pack8(ob);
  }
}

// ---- backward of the gated product: with s = sigmoid(g),  dg = d u s (1 + g (1 - s)),  du = d g s -----
__global__ void __launch_bounds__(GL_THREADS)
silu_mul_bwd_kernel(const __nv_bfloat16* __restrict__ dout, int64_t ldd, const __nv_bfloat16* __restrict__ gate, int64_t ldg,
                    const __nv_bfloat16* __restrict__ up, int64_t ldu, __nv_bfloat16* __restrict__ dgate, int64_t lddg,
                    __nv_bfloat16* __restrict__ dup, int64_t lddu, int rows, int cols) {
  const uint32_t groups_per_row = cols / 8;
  const int64_t total = (int64_t)rows * groups_per_row;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = t / groups_per_row;
    const int col = (int)(t - row * groups_per_row) * 8;
    float d[8], g[8], u[8], og[8], ou[8];
    unpack8(*reinterpret_cast<const uint4*>(dout + row * ldd + col), d);
    unpack8(*reinterpret_cast<const uint4*>(gate + row * ldg + col), g);
    unpack8(*reinterpret_cast<const uint4*>(up + row * ldu + col), u);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float sg = sigmoid_f32(g[i]);
      og[i] = d[i] * u[i] * sg * fmaf(g[i], 1.0f - sg, 1.0f);
      ou[i] = d[i] * g[i] * sg;
    }
    *reinterpret_cast<uint4*>(dgate + row * lddg + col) = pack8(og);
    *reinterpret_cast<uint4*>(dup + row * lddu + col) = pack8(ou);
  }
}

// ---- embedding: out[t, :] = table[tokens[t], :]; a token outside [0, vocab) gives a row of zeros --------
__global__ void __launch_bounds__(GL_THREADS)
embedding_kernel(const __nv_bfloat16* __restrict__ table, int64_t ldt, const int* __restrict__ tokens, int vocab,
                 __nv_bfloat16* __restrict__ out, int64_t ldo, int rows, int cols) {
  const uint32_t groups_per_row = cols / 8;
  const int64_t total = (int64_t)rows * groups_per_row;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = t / groups_per_row;
    const int col = (int)(t - row * groups_per_row) * 8;
    const int tok = tokens[row];
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (tok >= 0 && tok < vocab) v = *reinterpret_cast<const uint4*>(table + (int64_t)tok * ldt + col);
    *reinterpret_cast<uint4*>(out + row * ldo + col) = v;
  }
}

// ---- out = a + b (residual connections and the sums of gradients that meet at one tensor) -----------
__global__ void __launch_bounds__(GL_THREADS)
add_kernel(const __nv_bfloat16* __restrict__ a, int64_t lda, const __nv_bfloat16* __restrict__ b, int64_t ldb,
           __nv_bfloat16* __restrict__ out, int64_t ldo, int rows, int cols) {
  const uint32_t groups_per_row = cols / 8;
  const int64_t total = (int64_t)rows * groups_per_row;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = t / groups_per_row;
    const int col = (int)(t - row * groups_per_row) * 8;
    float x[8], y[8], o[8];
    unpack8(*reinterpret_cast<const uint4*>(a + row * lda + col), x);
    unpack8(*reinterpret_cast<const uint4*>(b + row * ldb + col), y);
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] = x[i] + y[i];
    *reinterpret_cast<uint4*>(out + row * ldo + col) = pack8(o);
  }
}

int glue_grid(const faar_ctx* ctx, int64_t items) {
  int64_t blocks = (items + GL_THREADS - 1) / GL_THREADS;
  const int64_t cap = (int64_t)ctx->num_sms * 8;
  if (blocks > cap) blocks = cap;
  return (int)(blocks < 1 ? 1 : blocks);
}

}  // namespace

int faar_launch_silu_mul(faar_ctx* ctx, int rows, int cols, const void* gate, int64_t ldg, const void* up, int64_t ldu,
                         void* out, int64_t ldo) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  silu_mul_kernel<<<glue_grid(ctx, (int64_t)rows * (cols / 8)), GL_THREADS, 0, ctx->stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(gate), ldg, reinterpret_cast<const __nv_bfloat16*>(up), ldu,
      reinterpret_cast<__nv_bfloat16*>(out), ldo, rows, cols);
  return (int)cudaGetLastError();
}

int faar_launch_rmsnorm(faar_ctx* ctx, int rows, int cols, const void* x, int64_t ldx, const float* g, float eps, void* y,
                        int64_t ldy, float* rstd) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  rmsnorm_kernel<<<glue_grid(ctx, (int64_t)rows * 32), GL_THREADS, 0, ctx->stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(x), ldx, g, eps, reinterpret_cast<__nv_bfloat16*>(y), ldy, rstd, rows, cols);
  return (int)cudaGetLastError();
}

int faar_launch_rmsnorm_bwd(faar_ctx* ctx, int rows, int cols, const void* dy, int64_t lddy, const void* x, int64_t ldx,
                            const float* g, const float* rstd, const void* add, int64_t ldadd, void* dx, int64_t lddx) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  rmsnorm_bwd_kernel<<<glue_grid(ctx, (int64_t)rows * 32), GL_THREADS, 0, ctx->stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(dy), lddy, reinterpret_cast<const __nv_bfloat16*>(x), ldx, g, rstd,
      reinterpret_cast<const __nv_bfloat16*>(add), ldadd, reinterpret_cast<__nv_bfloat16*>(dx), lddx, rows, cols);
  return (int)cudaGetLastError();
}

int faar_launch_rope(faar_ctx* ctx, int rows, int n_heads, int head_dim, const void* x, int64_t ldx, const int* pos, float theta,
                     int inverse, void* y, int64_t ldy) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  rope_kernel<<<glue_grid(ctx, (int64_t)rows * n_heads * (head_dim / 16)), GL_THREADS, 0, ctx->stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(x), ldx, pos, reinterpret_cast<__nv_bfloat16*>(y), ldy, rows, n_heads, head_dim,
      log2f(theta), inverse);
  return (int)cudaGetLastError();
}

int faar_launch_silu_mul_bwd(faar_ctx* ctx, int rows, int cols, const void* dout, int64_t ldd, const void* gate, int64_t ldg,
                             const void* up, int64_t ldu, void* dgate, int64_t lddg, void* dup, int64_t lddu) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  silu_mul_bwd_kernel<<<glue_grid(ctx, (int64_t)rows * (cols / 8)), GL_THREADS, 0, ctx->stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(dout), ldd, reinterpret_cast<const __nv_bfloat16*>(gate), ldg,
      reinterpret_cast<const __nv_bfloat16*>(up), ldu, reinterpret_cast<__nv_bfloat16*>(dgate), lddg,
      reinterpret_cast<__nv_bfloat16*>(dup), lddu, rows, cols);
  return (int)cudaGetLastError();
}

int faar_launch_embedding(faar_ctx* ctx, int rows, int cols, int vocab, const void* table, int64_t ldt, const int* tokens,
                          void* out, int64_t ldo) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  embedding_kernel<<<glue_grid(ctx, (int64_t)rows * (cols / 8)), GL_THREADS, 0, ctx->stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(table), ldt, tokens, vocab, reinterpret_cast<__nv_bfloat16*>(out), ldo, rows, cols);
  return (int)cudaGetLastError();
}

int faar_launch_add(faar_ctx* ctx, int rows, int cols, const void* a, int64_t lda, const void* b, int64_t ldb, void* out,
                    int64_t ldo) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  add_kernel<<<glue_grid(ctx, (int64_t)rows * (cols / 8)), GL_THREADS, 0, ctx->stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(a), lda, reinterpret_cast<const __nv_bfloat16*>(b), ldb,
      reinterpret_cast<__nv_bfloat16*>(out), ldo, rows, cols);
  return (int)cudaGetLastError();
}
