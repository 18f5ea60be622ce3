// HBM-bound kernels of the FAAR layer step: soft-quantisation set-up (scales,
// bracket, V_init), the FP32 soft-weight view, the BF16 soft-weight operand,
// Round Loss reduction, hardening + packing, and a BF16 transpose.
//
// Work decomposition used by all per-weight kernels: one thread owns 8
// consecutive weights of a row (half a scale block), so V moves as two float4,
// the code as one 32-bit word and BF16 data as one 16-byte vector; the two
// threads of a block exchange their maxima with one shuffle.
#include "faar_internal.cuh"

namespace {

constexpr int EW_THREADS = 256;

__device__ __forceinline__ void load8(const void* W, int w_dtype, int64_t idx, float (&w)[8]) {
  if (w_dtype == FAAR_BF16) {
    uint4 raw = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(W) + idx);
    const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      w[2 * i] = __uint_as_float(r[i] << 16);
      w[2 * i + 1] = __uint_as_float(r[i] & 0xFFFF0000u);
    }
  } else {
    const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(W) + idx);
    float4 a = p[0], b = p[1];
    w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
    w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
  }
}

// Element offset in W of 8-element group g.  Dense rows (ldw == K) need no division; otherwise the
// row comes from a 32-bit division (the host checks that the group count fits).
__device__ __forceinline__ int64_t w_offset(int64_t g, uint32_t groups_per_row, int64_t ldw, bool dense) {
  if (dense) return g * 8;
  const uint32_t row = (uint32_t)g / groups_per_row;
  return (int64_t)row * ldw + (int64_t)((uint32_t)g - row * groups_per_row) * 8;
}

// ---- pass 1: max |W| over the tensor -----------------------------------------
__global__ void __launch_bounds__(EW_THREADS)
amax_kernel(const void* __restrict__ W, int w_dtype, int O, int K, int64_t ldw, uint32_t* amax_word) {
  const uint32_t groups_per_row = K / 8;
  const int64_t total = (int64_t)O * groups_per_row;
  const bool dense = ldw == K;
  float amax = 0.f;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  // four independent 16-byte (32-byte for FP32) loads in flight per thread
  for (; g + 3 * stride < total; g += 4 * stride) {
    float w[4][8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      load8(W, w_dtype, w_offset(g + j * stride, groups_per_row, ldw, dense), w[j]);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(w[j][i]));
  }
  for (; g < total; g += stride) {
    float w[8];
    load8(W, w_dtype, w_offset(g, groups_per_row, ldw, dense), w);
#pragma unroll
    for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(w[i]));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  __shared__ float s_max[EW_THREADS / 32];
  if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = 0.f;
    for (int i = 0; i < EW_THREADS / 32; ++i) m = fmaxf(m, s_max[i]);
    atomicMax(amax_word, __float_as_uint(m));   // non-negative floats order like their bit patterns
  }
}

// ---- pass 2: block scales, bracket, V_init -------------------------------------
__global__ void __launch_bounds__(EW_THREADS)
softquant_init_kernel(const void* __restrict__ W, int w_dtype, int O, int K, int64_t ldw,
                      float s_global_in, const uint32_t* __restrict__ amax_word,
                      uint8_t* __restrict__ scales, float* __restrict__ s_global_out,
                      uint8_t* __restrict__ code, float* __restrict__ V) {
  float s_global;
  if (s_global_in > 0.f) {
    s_global = s_global_in;
  } else {
    float amax_t = __uint_as_float(*amax_word);
    s_global = amax_t == 0.f ? 1.0f : __fdiv_rn(amax_t, 2688.0f);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *s_global_out = s_global;
  const float d = __fmul_rn(s_global, 6.0f);

  const uint32_t groups_per_row = K / 8;
  const int64_t total = (int64_t)O * groups_per_row;
  const bool dense = ldw == K;
  // the grid is sized so that every warp is either fully inside or the tail is padded with idle lanes
  for (int64_t g0 = (int64_t)blockIdx.x * blockDim.x; g0 < total; g0 += (int64_t)gridDim.x * blockDim.x) {
    int64_t g = g0 + threadIdx.x;
    bool valid = g < total;
    int64_t gc = valid ? g : total - 1;
    float w[8];
    load8(W, w_dtype, w_offset(gc, groups_per_row, ldw, dense), w);
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(w[i]));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));   // partner holds the other half-block
    const uint32_t sb = faar_float_to_e4m3(__fdiv_rn(amax, d));
    const float s = __fmul_rn(faar_e4m3_to_float(sb), s_global);
    uint32_t cw = 0;
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float wt = s > 0.f ? __fdiv_rn(fabsf(w[i]), s) : 0.f;
      wt = fminf(wt, 6.0f);
      // From 1 upwards the nodes are the floats with a one-bit mantissa, so the bits of w~ give the bracket:
      // lower node = w~ with the mantissa cut to its top bit, interval index = (bits >> 22) - 252
      // ([1,1.5) -> 2, [1.5,2) -> 3, [2,3) -> 4, [3,4) -> 5, [4,6) -> 6), 1 / width = 2^(1 - exponent).
      // Below 1 the nodes 0, 0.5, 1 are 0.5 apart.  w~ = 6 (the clamp) closes the last interval: k = 6, v = 1.
      const uint32_t wb = __float_as_uint(wt);
      const bool ge1 = wt >= 1.0f, geh = wt >= 0.5f;
      const float lo = ge1 ? __uint_as_float(wb & 0xFFC00000u) : (geh ? 0.5f : 0.0f);
      const float inv_w = ge1 ? __uint_as_float(0x7F800000u - (wb & 0x7F800000u)) : 2.0f;      // 2, 1, 0.5
      uint32_t k = ge1 ? (wb >> 22) - 252u : (geh ? 1u : 0u);
      float vi = __fmul_rn(__fsub_rn(wt, lo), inv_w);
      if (wt >= 6.0f) { k = 6u; vi = 1.0f; }
      v[i] = vi;
      cw |= (k | (w[i] < 0.f ? 8u : 0u)) << (4 * i);                  // -0.0 counts as positive
    }
    if (valid) {
      const int64_t e = g * 8;                 // V, code, scales are dense
      const bool first_half = (g & 1) == 0;    // K % 16 == 0: even groups start a scale block
      float4* vp = reinterpret_cast<float4*>(V + e);
      vp[0] = make_float4(v[0], v[1], v[2], v[3]);
      vp[1] = make_float4(v[4], v[5], v[6], v[7]);
      *reinterpret_cast<uint32_t*>(code + e / 2) = cw;
      if (first_half) scales[e / 16] = (uint8_t)sb;
    }
  }
}

// ---- activation fake-quantisation: the X_q of Eq. 5 --------------------------------------------
// Same format and scale rule as the weights; each value goes to the nearest node, a tie to the larger
// magnitude (Eq. 7 applied to the initial position).  The output holds sign * node * block scale, which
// needs at most 7 significant bits and is therefore exact in BF16; the FP32 tensor scale stays outside
// (X_q = Xq_units * s_global) and is applied by the GEMM epilogues.
__global__ void __launch_bounds__(EW_THREADS)
act_fakequant_kernel(const __nv_bfloat16* __restrict__ X, int T, int K, int64_t ldx, float s_global_in,
                     const uint32_t* __restrict__ amax_word, __nv_bfloat16* __restrict__ Xq, int64_t ldq,
                     float* __restrict__ s_global_out, uint8_t* __restrict__ packed, uint8_t* __restrict__ scales) {
  float s_global;
  if (s_global_in > 0.f) {
    s_global = s_global_in;
  } else {
    float amax_t = __uint_as_float(*amax_word);
    s_global = amax_t == 0.f ? 1.0f : __fdiv_rn(amax_t, 2688.0f);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *s_global_out = s_global;
  const float d = __fmul_rn(s_global, 6.0f);
  const uint32_t groups_per_row = K / 8;
  const int64_t total = (int64_t)T * groups_per_row;
  for (int64_t g0 = (int64_t)blockIdx.x * blockDim.x; g0 < total; g0 += (int64_t)gridDim.x * blockDim.x) {
    int64_t g = g0 + threadIdx.x;
    bool valid = g < total;
    int64_t gc = valid ? g : total - 1;
    const uint32_t row = (uint32_t)gc / groups_per_row, col = ((uint32_t)gc - row * groups_per_row) * 8;
    float w[8];
    load8(X, FAAR_BF16, (int64_t)row * ldx + col, w);
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(w[i]));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));   // partner holds the other half-block
    const uint32_t sb = faar_float_to_e4m3(__fdiv_rn(amax, d));
    const float sg = faar_e4m3_to_float(sb);
    const float s = __fmul_rn(sg, s_global);
    uint32_t cw = 0;
    float q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float wt = s > 0.f ? __fdiv_rn(fabsf(w[i]), s) : 0.f;
      wt = fminf(wt, 6.0f);
      // Nearest node, a tie to the larger one.  From 1 upwards the nodes are the floats with a one-bit
      // mantissa: add a quarter of the binade and cut the mantissa to its top bit (5 -> 6, 3.5 -> 4,
      // 1.25 -> 1.5; 6 stays 6).  Below 1 the nodes 0, 0.5, 1 are 0.5 apart.
      const uint32_t rb = (__float_as_uint(wt) + 0x00200000u) & 0xFFC00000u;
      const float node = wt >= 1.0f ? __uint_as_float(rb) : (wt >= 0.75f ? 1.0f : (wt >= 0.25f ? 0.5f : 0.0f));
      // E2M1 magnitude code of the node: 0, 0.5 -> 0, 1; from 1 upwards exponent and mantissa bit count on
      const int c = node >= 1.0f ? (int)(__float_as_uint(node) >> 22) - 252 : (node > 0.0f ? 1 : 0);
      const float mag = __fmul_rn(node, sg);                      // exact: 2 x 4 significant bits
      const bool neg = w[i] < 0.f;
      q[i] = neg ? -mag : mag;
      cw |= ((uint32_t)c | (neg ? 8u : 0u)) << (4 * i);
    }
    if (valid) {
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 p2 = __floats2bfloat162_rn(q[2 * i], q[2 * i + 1]);
        o[i] = *reinterpret_cast<uint32_t*>(&p2);
      }
      *reinterpret_cast<uint4*>(Xq + (int64_t)row * ldq + col) = make_uint4(o[0], o[1], o[2], o[3]);
      const int64_t e = g * 8;                 // packed and scales are dense
      if (packed) *reinterpret_cast<uint32_t*>(packed + e / 2) = cw;
      if (scales && (g & 1) == 0) scales[e / 16] = (uint8_t)sb;
    }
  }
}

// ---- Eq. 2 / Eq. 3 -----------------------------------------------------------------------------
// FP32 outputs (W_soft, H): the parity view, relative error below 1e-6.
// BF16 output: the operand of the forward GEMM.  It is rounded from a cheaper FP32 evaluation whose
// relative error is below 3e-6 for beta <= 32 (beta*log2(e) rounded once, the exponent formed in one
// FMA, hardware 2^x and reciprocal), far inside the BF16 spacing of 2^-8; it can differ from the rounding of the exact
// value only where that value lies within 3e-6 of a BF16 rounding boundary.
// Per nibble (sign<<3 | k) the signed lower node and the signed interval width come from a
// 16-entry table in shared memory: mag = lo + h*width needs one 8-byte load.
__global__ void __launch_bounds__(EW_THREADS)
softquant_eval_kernel(const float* __restrict__ V, const uint8_t* __restrict__ code,
                      const uint8_t* __restrict__ scales, const float* __restrict__ s_global_p,
                      float beta, int64_t n_groups, float* __restrict__ W_soft, float* __restrict__ H,
                      __nv_bfloat16* __restrict__ W_bf16, float* __restrict__ W_operand_f32) {
  __shared__ float2 lut[16];
  if (threadIdx.x < 16) {
    const int k = threadIdx.x & 7;
    const float sgn = (threadIdx.x & 8) ? -1.f : 1.f;
    lut[threadIdx.x] = make_float2(sgn * faar_node(k), sgn * faar_width(k));
  }
  __syncthreads();
  faar_pdl_sync();                                   // V comes from the previous step's backward kernel
  const float s_global = *s_global_p;
  float nbl, hbl;
  faar_operand_consts(beta, &nbl, &hbl);
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < n_groups;
       g += (int64_t)gridDim.x * blockDim.x) {
    int64_t e = g * 8;
    const float4* vp = reinterpret_cast<const float4*>(V + e);
    float4 a = vp[0], b = vp[1];
    float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint32_t cw = *reinterpret_cast<const uint32_t*>(code + e / 2);
    float s = __fmul_rn(faar_e4m3_to_float(scales[e / 16]), s_global);
    if (W_soft || H) {
      float ws[8], h[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        uint32_t nib = (cw >> (4 * i)) & 0xF;
        h[i] = faar_sigmoid_precise(beta, v[i]);
        ws[i] = faar_soft_weight(h[i], nib, s);
      }
      if (W_soft) {
        float4* p = reinterpret_cast<float4*>(W_soft + e);
        p[0] = make_float4(ws[0], ws[1], ws[2], ws[3]);
        p[1] = make_float4(ws[4], ws[5], ws[6], ws[7]);
      }
      if (H) {
        float4* p = reinterpret_cast<float4*>(H + e);
        p[0] = make_float4(h[0], h[1], h[2], h[3]);
        p[1] = make_float4(h[4], h[5], h[6], h[7]);
      }
    }
    if (W_bf16 || W_operand_f32) {
      float wf[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float2 nw = lut[(cw >> (4 * i)) & 0xF];
        wf[i] = faar_operand_weight(faar_sigmoid_operand(nbl, hbl, v[i]), nw.x, nw.y, s);
      }
      if (W_operand_f32) {                              // debug view: the operand before its rounding to BF16
        float4* p = reinterpret_cast<float4*>(W_operand_f32 + e);
        p[0] = make_float4(wf[0], wf[1], wf[2], wf[3]);
        p[1] = make_float4(wf[4], wf[5], wf[6], wf[7]);
      }
      if (!W_bf16) continue;
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 p2 = __floats2bfloat162_rn(wf[2 * i], wf[2 * i + 1]);
        o[i] = *reinterpret_cast<uint32_t*>(&p2);
      }
      *reinterpret_cast<uint4*>(W_bf16 + e) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

// ---- Round Loss partial sums ------------------------------------------------------------
__global__ void __launch_bounds__(EW_THREADS)
round_partials_kernel(const float* __restrict__ V, int64_t N, float* __restrict__ partials) {
  float acc = 0.f;
  const int64_t n4 = N / 4;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
       i += (int64_t)gridDim.x * blockDim.x) {
    float4 a = reinterpret_cast<const float4*>(V)[i];
    float t0 = 2.f * a.x - 1.f, t1 = 2.f * a.y - 1.f, t2 = 2.f * a.z - 1.f, t3 = 2.f * a.w - 1.f;
    acc += (1.f - t0 * t0) + (1.f - t1 * t1) + (1.f - t2 * t2) + (1.f - t3 * t3);
  }
  if (blockIdx.x == 0 && threadIdx.x < (int)(N - n4 * 4)) {
    float t = 2.f * V[n4 * 4 + threadIdx.x] - 1.f;
    acc += 1.f - t * t;
  }
  acc = faar_warp_sum(acc);
  __shared__ float s_sum[EW_THREADS / 32];
  if ((threadIdx.x & 31) == 0) s_sum[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int i = 0; i < EW_THREADS / 32; ++i) t += s_sum[i];
    partials[blockIdx.x] = t;
  }
}

// Fixed-order final sums (one block; double accumulation).
__global__ void __launch_bounds__(256)
finalize_kernel(const float* __restrict__ p0, int n0, float scale0, float* out0,
                const float* __restrict__ p1, int n1, float scale1, float* out1) {
  __shared__ double sh[256];
  for (int which = 0; which < 2; ++which) {
    const float* p = which ? p1 : p0;
    int n = which ? n1 : n0;
    float* out = which ? out1 : out0;
    if (n <= 0 || out == nullptr) continue;
    double acc = 0.0;
    for (int i = threadIdx.x; i < n; i += 256) acc += (double)p[i];
    sh[threadIdx.x] = acc;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
      if (threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
      __syncthreads();
    }
    if (threadIdx.x == 0) *out = (float)(sh[0] * (double)(which ? scale1 : scale0));
    __syncthreads();
  }
}

// ---- Eq. 7: harden + pack ---------------------------------------------------------------
__global__ void __launch_bounds__(EW_THREADS)
harden_pack_kernel(const float* __restrict__ V, const uint8_t* __restrict__ code,
                   const uint8_t* __restrict__ scales, const float* __restrict__ s_global_p,
                   int64_t n_groups, uint8_t* __restrict__ packed, uint8_t* __restrict__ scales_out,
                   uint8_t* __restrict__ decisions, void* __restrict__ W_final, int wfinal_dtype) {
  const float s_global = W_final ? *s_global_p : 0.f;
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < n_groups;
       g += (int64_t)gridDim.x * blockDim.x) {
    int64_t e = g * 8;
    const float4* vp = reinterpret_cast<const float4*>(V + e);
    float4 a = vp[0], b = vp[1];
    float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint32_t cw = *reinterpret_cast<const uint32_t*>(code + e / 2);
    uint32_t dec = 0, add = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      uint32_t up = v[i] >= 0.5f ? 1u : 0u;
      dec |= up << i;
      add |= up << (4 * i);
    }
    uint32_t pw = cw + add;      // k <= 6, so k + 1 never carries into the sign bit
    *reinterpret_cast<uint32_t*>(packed + e / 2) = pw;
    if (decisions) decisions[g] = (uint8_t)dec;
    if (scales_out && (g & 1) == 0) scales_out[e / 16] = scales[e / 16];
    if (W_final) {
      float s = __fmul_rn(faar_e4m3_to_float(scales[e / 16]), s_global);
      float wf[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        uint32_t nib = (pw >> (4 * i)) & 0xF;
        float mag = __fmul_rn(faar_node(nib & 7), s);
        wf[i] = (nib & 8) ? -mag : mag;
      }
      if (wfinal_dtype == FAAR_F32) {
        float4* p = reinterpret_cast<float4*>(reinterpret_cast<float*>(W_final) + e);
        p[0] = make_float4(wf[0], wf[1], wf[2], wf[3]);
        p[1] = make_float4(wf[4], wf[5], wf[6], wf[7]);
      } else {
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          __nv_bfloat162 p2 = __floats2bfloat162_rn(wf[2 * i], wf[2 * i + 1]);
          o[i] = *reinterpret_cast<uint32_t*>(&p2);
        }
        *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(W_final) + e) = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
  }
}

// ---- block scales into the tiled order of block-scaled tensor-core GEMMs ----------------------------
// Output: 128 x 4 tiles of 512 bytes, tiles of a row band first; byte (r, c) of a tile at
// (r % 32) * 16 + (r / 32) * 4 + c; rows and columns beyond the matrix are zero.  One thread per output
// 4-byte word (the four columns of one row of one tile).
__global__ void __launch_bounds__(EW_THREADS)
swizzle_scales_kernel(const uint8_t* __restrict__ in, int rows, int cols, uint32_t* __restrict__ out, int64_t n_words) {
  const int col_tiles = (cols + 3) / 4;
  for (int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; w < n_words; w += (int64_t)gridDim.x * blockDim.x) {
    const int64_t tile = w >> 7;
    const int in_tile = (int)(w & 127);                 // (r % 32) * 4 + r / 32
    const int r = (int)(tile / col_tiles) * 128 + (in_tile & 3) * 32 + (in_tile >> 2);
    const int c0 = (int)(tile % col_tiles) * 4;
    uint32_t v = 0;
    if (r < rows) {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (c0 + j < cols) v |= (uint32_t)in[(int64_t)r * cols + c0 + j] << (8 * j);
    }
    out[w] = v;
  }
}

// ---- BF16 transpose through shared memory -----------------------------------------------
__global__ void __launch_bounds__(256)
transpose_bf16_kernel(const uint16_t* __restrict__ in, int rows, int cols, int64_t ld_in,
                      uint16_t* __restrict__ out, int64_t ld_out) {
  __shared__ uint16_t tile[64][66];
  const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;   // 64 x 4
  for (int i = ty; i < 64; i += 4) {
    int r = r0 + i, c = c0 + tx;
    tile[i][tx] = (r < rows && c < cols) ? in[(int64_t)r * ld_in + c] : (uint16_t)0;
  }
  __syncthreads();
  for (int i = ty; i < 64; i += 4) {
    int c = c0 + i, r = r0 + tx;
    if (c < cols && r < rows) out[(int64_t)c * ld_out + r] = tile[tx][i];
  }
}

// The same transpose with 16-byte global accesses, for the aligned case (cols, ld_in, ld_out multiples
// of 8, 16-byte aligned bases, ld_out >= rows rounded up to 8).  A thread reads 8 columns of two
// consecutive rows, pairs the values column by column (element r in the low half, r + 1 in the high half)
// and stores the eight 32-bit pairs into tile[column][row pair]; a row of the tile is then a run of the
// output row and leaves as 16-byte vectors.  Rows beyond the matrix enter as zeros and may be written
// into the padding of the output rows.
__global__ void __launch_bounds__(256)
transpose_bf16_vec_kernel(const uint16_t* __restrict__ in, int rows, int cols, int64_t ld_in,
                          uint16_t* __restrict__ out, int64_t ld_out) {
  __shared__ __align__(16) uint32_t tile[64][36];
  const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
  {
    const int rp = threadIdx.x & 31, cc = threadIdx.x >> 5;          // row pair, 8-column chunk
    const int r = r0 + 2 * rp, c = c0 + 8 * cc;
    uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
    if (c < cols) {
      if (r < rows) a = *reinterpret_cast<const uint4*>(in + (int64_t)r * ld_in + c);
      if (r + 1 < rows) b = *reinterpret_cast<const uint4*>(in + (int64_t)(r + 1) * ld_in + c);
    }
    const uint32_t x[4] = {a.x, a.y, a.z, a.w}, y[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      tile[8 * cc + 2 * j][rp] = __byte_perm(x[j], y[j], 0x5410);     // column 2j: low halves
      tile[8 * cc + 2 * j + 1][rp] = __byte_perm(x[j], y[j], 0x7632); // column 2j + 1: high halves
    }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int idx = threadIdx.x + 256 * i;
    const int cl = idx >> 3, q = idx & 7;                             // output row of the tile, 8-element chunk
    const int c = c0 + cl, r = r0 + 8 * q;
    if (c < cols && r < rows)
      *reinterpret_cast<uint4*>(out + (int64_t)c * ld_out + r) = *reinterpret_cast<const uint4*>(&tile[cl][4 * q]);
  }
}

int grid_for(const faar_ctx* ctx, int64_t work_items, int per_sm) {
  int64_t blocks = (work_items + EW_THREADS - 1) / EW_THREADS;
  int64_t cap = (int64_t)ctx->num_sms * per_sm;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

}  // namespace

int faar_launch_softquant_init(faar_ctx* ctx, const faar_shape* s, const void* W, float s_global_in,
                               uint8_t* scales, float* s_global_out, uint8_t* code, float* V,
                               uint32_t* amax_word) {
  const int64_t groups = (int64_t)s->O * (s->K / 8);
  const int grid = grid_for(ctx, groups, 8);
  if (!(s_global_in > 0.f)) {
    cudaError_t e = cudaMemsetAsync(amax_word, 0, sizeof(uint32_t), ctx->stream);
    if (e != cudaSuccess) return (int)e;
    faar_prof_scope ps(ctx, FAAR_K_AMAX);
    amax_kernel<<<grid, EW_THREADS, 0, ctx->stream>>>(W, s->w_dtype, s->O, s->K, s->ldw, amax_word);
  }
  faar_prof_scope ps(ctx, FAAR_K_SOFTQUANT_INIT);
  softquant_init_kernel<<<grid, EW_THREADS, 0, ctx->stream>>>(W, s->w_dtype, s->O, s->K, s->ldw, s_global_in,
                                                               amax_word, scales, s_global_out, code, V);
  return (int)cudaGetLastError();
}

int faar_launch_act_fakequant(faar_ctx* ctx, int T, int K, const void* X, int64_t ldx, float s_global_in, void* Xq,
                              int64_t ldq, float* s_global_out, uint8_t* packed, uint8_t* scales, uint32_t* amax_word) {
  const int64_t groups = (int64_t)T * (K / 8);
  const int grid = grid_for(ctx, groups, 8);
  if (!(s_global_in > 0.f)) {
    cudaError_t e = cudaMemsetAsync(amax_word, 0, sizeof(uint32_t), ctx->stream);
    if (e != cudaSuccess) return (int)e;
    faar_prof_scope ps(ctx, FAAR_K_AMAX);
    amax_kernel<<<grid, EW_THREADS, 0, ctx->stream>>>(X, FAAR_BF16, T, K, ldx, amax_word);
  }
  faar_prof_scope ps(ctx, FAAR_K_ACT_FAKEQUANT);
  act_fakequant_kernel<<<grid, EW_THREADS, 0, ctx->stream>>>(reinterpret_cast<const __nv_bfloat16*>(X), T, K, ldx,
                                                            s_global_in, amax_word, reinterpret_cast<__nv_bfloat16*>(Xq),
                                                            ldq, s_global_out, packed, scales);
  return (int)cudaGetLastError();
}

int faar_launch_softquant_eval(faar_ctx* ctx, const faar_shape* s, const float* V, const uint8_t* code,
                               const uint8_t* scales, const float* s_global, float beta, float* W_soft,
                               float* h, __nv_bfloat16* W_bf16, float* W_operand_f32) {
  const int64_t groups = (int64_t)s->O * (s->K / 8);
  faar_prof_scope ps(ctx, FAAR_K_SOFT_WEIGHTS);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(grid_for(ctx, groups, 8), 1, 1);
  cfg.blockDim = dim3(EW_THREADS, 1, 1);
  cfg.stream = ctx->stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, softquant_eval_kernel, V, code, scales, s_global, beta, (int64_t)groups, W_soft,
                                     h, W_bf16, W_operand_f32);
  if (e != cudaSuccess) return (int)e;
  return (int)cudaGetLastError();
}

int faar_launch_transpose_bf16(faar_ctx* ctx, int rows, int cols, const void* in, int64_t ld_in, void* out,
                               int64_t ld_out) {
  dim3 grid((cols + 63) / 64, (rows + 63) / 64);
  faar_prof_scope ps(ctx, FAAR_K_TRANSPOSE);
  const bool vec = cols % 8 == 0 && ld_in % 8 == 0 && ld_out % 8 == 0 && ld_out >= (int64_t)(rows + 7) / 8 * 8 &&
                   ((uintptr_t)in & 15) == 0 && ((uintptr_t)out & 15) == 0;
  if (vec) {
    transpose_bf16_vec_kernel<<<grid, 256, 0, ctx->stream>>>(reinterpret_cast<const uint16_t*>(in), rows, cols, ld_in,
                                                             reinterpret_cast<uint16_t*>(out), ld_out);
    return (int)cudaGetLastError();
  }
  transpose_bf16_kernel<<<grid, 256, 0, ctx->stream>>>(reinterpret_cast<const uint16_t*>(in), rows, cols, ld_in,
                                                       reinterpret_cast<uint16_t*>(out), ld_out);
  return (int)cudaGetLastError();
}

int faar_launch_swizzle_scales(faar_ctx* ctx, int rows, int cols, const uint8_t* in, uint8_t* out) {
  const int64_t n_words = (int64_t)((rows + 127) / 128) * ((cols + 3) / 4) * 128;
  faar_prof_scope ps(ctx, FAAR_K_HARDEN_PACK);
  swizzle_scales_kernel<<<grid_for(ctx, n_words, 8), EW_THREADS, 0, ctx->stream>>>(in, rows, cols,
                                                                                  reinterpret_cast<uint32_t*>(out), n_words);
  return (int)cudaGetLastError();
}

int faar_launch_round_partials(faar_ctx* ctx, const float* V, int64_t N, float* partials, int* n_partials) {
  int grid = grid_for(ctx, (N + 3) / 4, 4);
  if (grid > FAAR_MAX_PARTIALS) grid = FAAR_MAX_PARTIALS;
  faar_prof_scope ps(ctx, FAAR_K_ROUND_LOSS);
  round_partials_kernel<<<grid, EW_THREADS, 0, ctx->stream>>>(V, N, partials);
  *n_partials = grid;
  return (int)cudaGetLastError();
}

int faar_launch_finalize(faar_ctx* ctx, const float* p0, int n0, float scale0, float* out0, const float* p1,
                         int n1, float scale1, float* out1) {
  faar_prof_scope ps(ctx, FAAR_K_FINALIZE);
  finalize_kernel<<<1, 256, 0, ctx->stream>>>(p0, n0, scale0, out0, p1, n1, scale1, out1);
  return (int)cudaGetLastError();
}

int faar_launch_harden_pack(faar_ctx* ctx, const faar_shape* s, const float* V, const uint8_t* code,
                            const uint8_t* scales, const float* s_global, uint8_t* packed,
                            uint8_t* scales_out, uint8_t* decisions, void* W_final, int wfinal_dtype) {
  const int64_t groups = (int64_t)s->O * (s->K / 8);
  faar_prof_scope ps(ctx, FAAR_K_HARDEN_PACK);
  harden_pack_kernel<<<grid_for(ctx, groups, 8), EW_THREADS, 0, ctx->stream>>>(
      V, code, scales, s_global, groups, packed, scales_out, decisions, W_final, wfinal_dtype);
  return (int)cudaGetLastError();
}
