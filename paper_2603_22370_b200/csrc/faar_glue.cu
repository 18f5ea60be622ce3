// Element-wise pieces of a decoder block that sit between the linears: what the layer-wise driver needs
// to produce each linear's calibration input on the device (the MLP's SiLU-gated product feeds down_proj),
// and what full-model alignment (Eq. 6, Procedure steps 15-23) needs around the tensor-core GEMMs.
// All of them are HBM-bound: BF16 in and out as 16-byte vectors, FP32 arithmetic in registers.
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
