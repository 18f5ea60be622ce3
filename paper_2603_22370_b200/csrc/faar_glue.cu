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

// sigmoid(x) in FP32: 1 / (1 + e^-x) with the library exponential (relative error ~1e-7) and the hardware
// reciprocal (rcp.approx: relative error below 2^-22); e^-x overflowing to +inf gives 0, the limit.
__device__ __forceinline__ float sigmoid_f32(float x) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + expf(-x)));
  return r;
}

// Work split of the [rows, 8-element groups] kernels: threadIdx.x / blockIdx.x run over the groups of a row,
// threadIdx.y / blockIdx.y over rows (grid-stride), so no thread divides its index by the row length.
struct Split { dim3 grid, block; };
__device__ __forceinline__ int split_group() { return blockIdx.x * blockDim.x + threadIdx.x; }
__device__ __forceinline__ int split_row0() { return blockIdx.y * blockDim.y + threadIdx.y; }
__device__ __forceinline__ int split_row_step() { return gridDim.y * blockDim.y; }

// out = silu(gate) * up, silu(x) = x * sigmoid(x); two rows per thread in flight
__global__ void __launch_bounds__(GL_THREADS)
silu_mul_kernel(const __nv_bfloat16* gate, int64_t ldg, const __nv_bfloat16* up, int64_t ldu, __nv_bfloat16* out, int64_t ldo,
                int rows, int groups) {
  const int cg = split_group();
  if (cg >= groups) return;
  const int col = 8 * cg, step = split_row_step();
  for (int row = split_row0(); row < rows; row += 2 * step) {
    const int row1 = row + step;
    const bool two = row1 < rows;
    const uint4 ga = *reinterpret_cast<const uint4*>(gate + (int64_t)row * ldg + col);
    const uint4 ua = *reinterpret_cast<const uint4*>(up + (int64_t)row * ldu + col);
    uint4 gb = ga, ub = ua;
    if (two) {
      gb = *reinterpret_cast<const uint4*>(gate + (int64_t)row1 * ldg + col);
      ub = *reinterpret_cast<const uint4*>(up + (int64_t)row1 * ldu + col);
    }
    float a[8], b[8], y[8];
    unpack8(ga, a); unpack8(ua, b);
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = a[i] * sigmoid_f32(a[i]) * b[i];
    *reinterpret_cast<uint4*>(out + (int64_t)row * ldo + col) = pack8(y);
    if (two) {
      unpack8(gb, a); unpack8(ub, b);
#pragma unroll
      for (int i = 0; i < 8; ++i) y[i] = a[i] * sigmoid_f32(a[i]) * b[i];
      *reinterpret_cast<uint4*>(out + (int64_t)row1 * ldo + col) = pack8(y);
    }
  }
}

// ---- RMSNorm: y = x / sqrt(mean(x^2) + eps) * g, one warp per row ---------------------------------
// Rows of up to 8 * 32 * NV elements stay in registers between the sum of squares and the scaled output (NV
// 16-byte vectors per lane); NV = 0 is the form for longer rows, which reads the row a second time (L1 / L2).
// With `b` the row is first formed as the BF16-rounded sum x + b and written to `sum_out` (a residual
// connection followed by the next norm): the same values as faar_add followed by faar_rmsnorm.
template <int NV>
__global__ void __launch_bounds__(GL_THREADS)
rmsnorm_kernel(const __nv_bfloat16* x, int64_t ldx, const __nv_bfloat16* b, int64_t ldb, __nv_bfloat16* sum_out, int64_t lds,
               const float* __restrict__ g, float eps, __nv_bfloat16* y, int64_t ldy, float* __restrict__ rstd_out, int rows,
               int cols) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int n_groups = cols / 8;
  for (int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; row < rows; row += warps) {
    const __nv_bfloat16* xr = x + (int64_t)row * ldx;
    const __nv_bfloat16* br = b ? b + (int64_t)row * ldb : nullptr;
    __nv_bfloat16* sr = b ? sum_out + (int64_t)row * lds : nullptr;
    __nv_bfloat16* yr = y + (int64_t)row * ldy;
    float ss = 0.f;
    if constexpr (NV > 0) {
      uint4 v[NV];
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int c = lane + 32 * k;
        if (c < n_groups) v[k] = *reinterpret_cast<const uint4*>(xr + 8 * c);
      }
      if (br) {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
          const int c = lane + 32 * k;
          if (c < n_groups) {
            float a[8], r[8];
            unpack8(v[k], a);
            unpack8(*reinterpret_cast<const uint4*>(br + 8 * c), r);
#pragma unroll
            for (int i = 0; i < 8; ++i) a[i] += r[i];
            v[k] = pack8(a);
            *reinterpret_cast<uint4*>(sr + 8 * c) = v[k];
          }
        }
      }
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        if (lane + 32 * k < n_groups) {
          float a[8];
          unpack8(v[k], a);
#pragma unroll
          for (int i = 0; i < 8; ++i) ss = fmaf(a[i], a[i], ss);
        }
      }
      ss = faar_warp_sum(ss);
      const float rstd = 1.0f / sqrtf(ss / (float)cols + eps);
      if (lane == 0 && rstd_out) rstd_out[row] = rstd;
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        const int c = lane + 32 * k;
        if (c < n_groups) {
          float a[8], o[8];
          unpack8(v[k], a);
          const float4 g0 = *reinterpret_cast<const float4*>(g + 8 * c), g1 = *reinterpret_cast<const float4*>(g + 8 * c + 4);
          const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
          for (int i = 0; i < 8; ++i) o[i] = a[i] * rstd * gg[i];
          *reinterpret_cast<uint4*>(yr + 8 * c) = pack8(o);
        }
      }
    } else {
      for (int c = lane; c < n_groups; c += 32) {
        float a[8];
        unpack8(*reinterpret_cast<const uint4*>(xr + 8 * c), a);
        if (br) {
          float r[8];
          unpack8(*reinterpret_cast<const uint4*>(br + 8 * c), r);
#pragma unroll
          for (int i = 0; i < 8; ++i) a[i] += r[i];
          const uint4 sum = pack8(a);
          *reinterpret_cast<uint4*>(sr + 8 * c) = sum;
          unpack8(sum, a);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) ss = fmaf(a[i], a[i], ss);
      }
      ss = faar_warp_sum(ss);
      const float rstd = 1.0f / sqrtf(ss / (float)cols + eps);
      if (lane == 0 && rstd_out) rstd_out[row] = rstd;
      const __nv_bfloat16* src = br ? sr : xr;          // this lane wrote the groups it reads back
      for (int c = lane; c < n_groups; c += 32) {
        float a[8], o[8];
        unpack8(*reinterpret_cast<const uint4*>(src + 8 * c), a);
        const float4 g0 = *reinterpret_cast<const float4*>(g + 8 * c), g1 = *reinterpret_cast<const float4*>(g + 8 * c + 4);
        const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) o[i] = a[i] * rstd * gg[i];
        *reinterpret_cast<uint4*>(yr + 8 * c) = pack8(o);
      }
    }
  }
}

// Backward of RMSNorm towards x (the norm weights are frozen): with xh = x * rstd and w = g * dy,
// dx = rstd * (w - xh * mean(w * xh)), optionally added to `add` (the residual branch's gradient).  dy is the
// FP32 sum of up to three BF16 tensors (the gradients of the linears that read the norm's output).  One warp
// per row; the row is read twice (the dot product, then the result), the second time from L1 / L2.  (Keeping
// x and w of a 2048-element row in registers between the passes takes 134 registers per thread and was three
// times slower.)
__global__ void __launch_bounds__(GL_THREADS)
rmsnorm_bwd_kernel(const __nv_bfloat16* dy, const __nv_bfloat16* dy2, const __nv_bfloat16* dy3, int64_t lddy,
                   const __nv_bfloat16* x, int64_t ldx, const float* __restrict__ g, const float* __restrict__ rstd_in,
                   const __nv_bfloat16* add, int64_t ldadd, __nv_bfloat16* dx, int64_t lddx, int rows, int cols) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  const int n_groups = cols / 8;
  for (int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; row < rows; row += warps) {
    const __nv_bfloat16* xr = x + (int64_t)row * ldx;
    const int64_t doff = (int64_t)row * lddy;
    const float rstd = rstd_in[row];
    // w = g * (dy + dy2 + dy3) of one group
    auto load_w = [&](int c, float (&w)[8]) {
      unpack8(*reinterpret_cast<const uint4*>(dy + doff + 8 * c), w);
      if (dy2) {
        float t[8];
        unpack8(*reinterpret_cast<const uint4*>(dy2 + doff + 8 * c), t);
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] += t[i];
      }
      if (dy3) {
        float t[8];
        unpack8(*reinterpret_cast<const uint4*>(dy3 + doff + 8 * c), t);
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] += t[i];
      }
      const float4 g0 = *reinterpret_cast<const float4*>(g + 8 * c), g1 = *reinterpret_cast<const float4*>(g + 8 * c + 4);
      const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) w[i] *= gg[i];
    };
    float dot = 0.f;
    for (int c = lane; c < n_groups; c += 32) {
      float a[8], w[8];
      unpack8(*reinterpret_cast<const uint4*>(xr + 8 * c), a);
      load_w(c, w);
#pragma unroll
      for (int i = 0; i < 8; ++i) dot = fmaf(w[i], a[i] * rstd, dot);
    }
    dot = faar_warp_sum(dot) / (float)cols;
    for (int c = lane; c < n_groups; c += 32) {
      float a[8], w[8], o[8];
      unpack8(*reinterpret_cast<const uint4*>(xr + 8 * c), a);
      load_w(c, w);
#pragma unroll
      for (int i = 0; i < 8; ++i) o[i] = rstd * fmaf(-(a[i] * rstd), dot, w[i]);
      if (add) {
        float r[8];
        unpack8(*reinterpret_cast<const uint4*>(add + (int64_t)row * ldadd + 8 * c), r);
#pragma unroll
        for (int i = 0; i < 8; ++i) o[i] += r[i];
      }
      *reinterpret_cast<uint4*>(dx + (int64_t)row * lddx + 8 * c) = pack8(o);
    }
  }
}

// ---- rotary position embedding, half-split pairing ----------------------------------------------
// Inside every head, element i (i < head_dim / 2) pairs with element i + head_dim / 2; the pair of token t is
// rotated by pos[t] * theta^(-2 i / head_dim) (by the negative angle with inverse != 0: the backward pass of
// an orthogonal map).  One thread takes 8 consecutive i of HPT heads of one token (the angle does not depend
// on the head, so its sine and cosine serve all of them), for a stride of tokens.
template <int HPT>
__global__ void __launch_bounds__(GL_THREADS)
rope_kernel(const __nv_bfloat16* x, int64_t ldx, const int* __restrict__ pos, __nv_bfloat16* y, int64_t ldy, int rows,
            int groups, int head_dim, float log2_theta, int inverse) {
  const int cg = split_group();
  if (cg >= groups) return;
  const int half = head_dim / 2, gph = half / 8;                    // 8-element groups per half head
  const int chunk = cg / gph, gi = cg - chunk * gph;
  const int64_t off = (int64_t)chunk * HPT * head_dim + 8 * gi;
  float inv_freq[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) inv_freq[i] = exp2f(-2.0f * (float)(8 * gi + i) / (float)head_dim * log2_theta);
  for (int row = split_row0(); row < rows; row += split_row_step()) {
    const __nv_bfloat16* xr = x + (int64_t)row * ldx + off;
    __nv_bfloat16* yr = y + (int64_t)row * ldy + off;
    uint4 ra[HPT], rb[HPT];
#pragma unroll
    for (int h = 0; h < HPT; ++h) {
      ra[h] = *reinterpret_cast<const uint4*>(xr + h * head_dim);
      rb[h] = *reinterpret_cast<const uint4*>(xr + h * head_dim + half);
    }
    const float p = (float)pos[row];
    float sn[8], cs[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      sincosf(p * inv_freq[i], &sn[i], &cs[i]);
      if (inverse) sn[i] = -sn[i];
    }
#pragma unroll
    for (int h = 0; h < HPT; ++h) {
      float a[8], b[8], oa[8], ob[8];
      unpack8(ra[h], a);
      unpack8(rb[h], b);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        oa[i] = a[i] * cs[i] - b[i] * sn[i];
        ob[i] = b[i] * cs[i] + a[i] * sn[i];
      }
      *reinterpret_cast<uint4*>(yr + h * head_dim) = pack8(oa);
      *reinterpret_cast<uint4*>(yr + h * head_dim + half) = pack8(ob);
    }
  }
}

// ---- backward of the gated product: with s = sigmoid(g),  dg = d u s (1 + g (1 - s)),  du = d g s -----
__global__ void __launch_bounds__(GL_THREADS)
silu_mul_bwd_kernel(const __nv_bfloat16* dout, int64_t ldd, const __nv_bfloat16* gate, int64_t ldg, const __nv_bfloat16* up,
                    int64_t ldu, __nv_bfloat16* dgate, int64_t lddg, __nv_bfloat16* dup, int64_t lddu, int rows, int groups) {
  const int cg = split_group();
  if (cg >= groups) return;
  const int col = 8 * cg;
  for (int row = split_row0(); row < rows; row += split_row_step()) {
    float d[8], g[8], u[8], og[8], ou[8];
    unpack8(*reinterpret_cast<const uint4*>(dout + (int64_t)row * ldd + col), d);
    unpack8(*reinterpret_cast<const uint4*>(gate + (int64_t)row * ldg + col), g);
    unpack8(*reinterpret_cast<const uint4*>(up + (int64_t)row * ldu + col), u);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float sg = sigmoid_f32(g[i]);
      og[i] = d[i] * u[i] * sg * fmaf(g[i], 1.0f - sg, 1.0f);
      ou[i] = d[i] * g[i] * sg;
    }
    *reinterpret_cast<uint4*>(dgate + (int64_t)row * lddg + col) = pack8(og);
    *reinterpret_cast<uint4*>(dup + (int64_t)row * lddu + col) = pack8(ou);
  }
}

// ---- embedding: out[t, :] = table[tokens[t], :]; a token outside [0, vocab) gives a row of zeros --------
__global__ void __launch_bounds__(GL_THREADS)
embedding_kernel(const __nv_bfloat16* __restrict__ table, int64_t ldt, const int* __restrict__ tokens, int vocab,
                 __nv_bfloat16* __restrict__ out, int64_t ldo, int rows, int groups) {
  const int cg = split_group();
  if (cg >= groups) return;
  const int col = 8 * cg;
  for (int row = split_row0(); row < rows; row += split_row_step()) {
    const int tok = tokens[row];
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (tok >= 0 && tok < vocab) v = *reinterpret_cast<const uint4*>(table + (int64_t)tok * ldt + col);
    *reinterpret_cast<uint4*>(out + (int64_t)row * ldo + col) = v;
  }
}

// ---- out = a + b (residual connections and the sums of gradients that meet at one tensor) -----------
__global__ void __launch_bounds__(GL_THREADS)
add_kernel(const __nv_bfloat16* a, int64_t lda, const __nv_bfloat16* b, int64_t ldb, __nv_bfloat16* out, int64_t ldo, int rows,
           int groups) {
  const int cg = split_group();
  if (cg >= groups) return;
  const int col = 8 * cg;
  for (int row = split_row0(); row < rows; row += split_row_step()) {
    float x[8], y[8], o[8];
    unpack8(*reinterpret_cast<const uint4*>(a + (int64_t)row * lda + col), x);
    unpack8(*reinterpret_cast<const uint4*>(b + (int64_t)row * ldb + col), y);
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] = x[i] + y[i];
    *reinterpret_cast<uint4*>(out + (int64_t)row * ldo + col) = pack8(o);
  }
}

// Launch shape for the kernels above: 256 threads as (groups of a row) x (rows), the row extent of the grid
// capped at eight blocks per SM.
Split glue_split(const faar_ctx* ctx, int rows, int groups) {
  int tx = 4;                                   // short rows: several rows per warp
  while (tx < GL_THREADS && tx < groups) tx *= 2;
  const int ty = GL_THREADS / tx;
  const int gx = (groups + tx - 1) / tx;
  int64_t gy = ((int64_t)rows + ty - 1) / ty;
  const int64_t cap = ((int64_t)ctx->num_sms * 8 + gx - 1) / gx;
  if (gy > cap) gy = cap;
  if (gy > 65535) gy = 65535;
  if (gy < 1) gy = 1;
  Split s;
  s.grid = dim3((unsigned)gx, (unsigned)gy, 1);
  s.block = dim3((unsigned)tx, (unsigned)ty, 1);
  return s;
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
  const Split sp = glue_split(ctx, (rows + 1) / 2, cols / 8);
  silu_mul_kernel<<<sp.grid, sp.block, 0, ctx->stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(gate), ldg, reinterpret_cast<const __nv_bfloat16*>(up), ldu,
      reinterpret_cast<__nv_bfloat16*>(out), ldo, rows, cols / 8);
  return (int)cudaGetLastError();
}

// b / sum_out null: y = rmsnorm(x).  Otherwise sum_out = x + b (BF16) and y = rmsnorm(sum_out).
int faar_launch_rmsnorm(faar_ctx* ctx, int rows, int cols, const void* x, int64_t ldx, const void* b, int64_t ldb,
                        void* sum_out, int64_t lds, const float* g, float eps, void* y, int64_t ldy, float* rstd) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  const int grid = glue_grid(ctx, (int64_t)rows * 32);
  auto* xp = reinterpret_cast<const __nv_bfloat16*>(x);
  auto* bp = reinterpret_cast<const __nv_bfloat16*>(b);
  auto* sp = reinterpret_cast<__nv_bfloat16*>(sum_out);
  auto* yp = reinterpret_cast<__nv_bfloat16*>(y);
  if (cols <= 8 * 32 * 8)
    rmsnorm_kernel<8><<<grid, GL_THREADS, 0, ctx->stream>>>(xp, ldx, bp, ldb, sp, lds, g, eps, yp, ldy, rstd, rows, cols);
  else
    rmsnorm_kernel<0><<<grid, GL_THREADS, 0, ctx->stream>>>(xp, ldx, bp, ldb, sp, lds, g, eps, yp, ldy, rstd, rows, cols);
  return (int)cudaGetLastError();
}

// dy2 / dy3 nullable: further gradients (same leading dimension as dy) summed with dy before the norm's backward.
int faar_launch_rmsnorm_bwd(faar_ctx* ctx, int rows, int cols, const void* dy, const void* dy2, const void* dy3, int64_t lddy,
                            const void* x, int64_t ldx, const float* g, const float* rstd, const void* add, int64_t ldadd,
                            void* dx, int64_t lddx) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  const int grid = glue_grid(ctx, (int64_t)rows * 32);
  auto* d1 = reinterpret_cast<const __nv_bfloat16*>(dy);
  auto* d2 = reinterpret_cast<const __nv_bfloat16*>(dy2);
  auto* d3 = reinterpret_cast<const __nv_bfloat16*>(dy3);
  auto* xp = reinterpret_cast<const __nv_bfloat16*>(x);
  auto* ap = reinterpret_cast<const __nv_bfloat16*>(add);
  auto* op = reinterpret_cast<__nv_bfloat16*>(dx);
  rmsnorm_bwd_kernel<<<grid, GL_THREADS, 0, ctx->stream>>>(d1, d2, d3, lddy, xp, ldx, g, rstd, ap, ldadd, op, lddx, rows, cols);
  return (int)cudaGetLastError();
}

int faar_launch_rope(faar_ctx* ctx, int rows, int n_heads, int head_dim, const void* x, int64_t ldx, const int* pos, float theta,
                     int inverse, void* y, int64_t ldy) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  const bool four = n_heads % 4 == 0;                                 // four heads per thread share one sine / cosine
  const int groups = (four ? n_heads / 4 : n_heads) * (head_dim / 16);
  const Split sp = glue_split(ctx, rows, groups);
  auto* xp = reinterpret_cast<const __nv_bfloat16*>(x);
  auto* yp = reinterpret_cast<__nv_bfloat16*>(y);
  if (four)
    rope_kernel<4><<<sp.grid, sp.block, 0, ctx->stream>>>(xp, ldx, pos, yp, ldy, rows, groups, head_dim, log2f(theta), inverse);
  else
    rope_kernel<1><<<sp.grid, sp.block, 0, ctx->stream>>>(xp, ldx, pos, yp, ldy, rows, groups, head_dim, log2f(theta), inverse);
  return (int)cudaGetLastError();
}

int faar_launch_silu_mul_bwd(faar_ctx* ctx, int rows, int cols, const void* dout, int64_t ldd, const void* gate, int64_t ldg,
                             const void* up, int64_t ldu, void* dgate, int64_t lddg, void* dup, int64_t lddu) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  const Split sp = glue_split(ctx, rows, cols / 8);
  silu_mul_bwd_kernel<<<sp.grid, sp.block, 0, ctx->stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(dout), ldd, reinterpret_cast<const __nv_bfloat16*>(gate), ldg,
      reinterpret_cast<const __nv_bfloat16*>(up), ldu, reinterpret_cast<__nv_bfloat16*>(dgate), lddg,
      reinterpret_cast<__nv_bfloat16*>(dup), lddu, rows, cols / 8);
  return (int)cudaGetLastError();
}

int faar_launch_embedding(faar_ctx* ctx, int rows, int cols, int vocab, const void* table, int64_t ldt, const int* tokens,
                          void* out, int64_t ldo) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  const Split sp = glue_split(ctx, rows, cols / 8);
  embedding_kernel<<<sp.grid, sp.block, 0, ctx->stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(table), ldt, tokens, vocab, reinterpret_cast<__nv_bfloat16*>(out), ldo, rows,
      cols / 8);
  return (int)cudaGetLastError();
}

int faar_launch_add(faar_ctx* ctx, int rows, int cols, const void* a, int64_t lda, const void* b, int64_t ldb, void* out,
                    int64_t ldo) {
  faar_prof_scope ps(ctx, FAAR_K_GLUE);
  const Split sp = glue_split(ctx, rows, cols / 8);
  add_kernel<<<sp.grid, sp.block, 0, ctx->stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(a), lda, reinterpret_cast<const __nv_bfloat16*>(b), ldb,
      reinterpret_cast<__nv_bfloat16*>(out), ldo, rows, cols / 8);
  return (int)cudaGetLastError();
}
