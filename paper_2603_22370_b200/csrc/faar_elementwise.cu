// HBM-bound kernels of the FAAR layer step: soft-quantisation set-up (scales,
// bracket, V_init), the FP32 soft-weight view, the BF16 soft-weight operand,
// Round Loss reduction, hardening + packing, and a BF16 transpose.
//
// Work decomposition used by all per-weight kernels: one thread owns 8
// consecutive weights of a row (half a scale block), so V moves as two float4,
// the code as one 32-bit word and BF16 data as one 16-byte vector; the two
// threads of a block exchange their maxima with one shuffle.
#include "faar_internal.cuh"

#include <atomic>

namespace {

constexpr int EW_THREADS = 256;

// Element offset in W of 8-element group g.  Dense rows (ldw == K) need no division; otherwise the
// row comes from a 32-bit division (the host checks that the group count fits).
__device__ __forceinline__ int64_t w_offset(int64_t g, uint32_t groups_per_row, int64_t ldw, bool dense) {
  if (dense) return g * 8;
  const uint32_t row = (uint32_t)g / groups_per_row;
  return (int64_t)row * ldw + (int64_t)((uint32_t)g - row * groups_per_row) * 8;
}

// ---- pass 1: max |W| over the tensor -----------------------------------------
// One thread takes 8-value groups g, g + stride, ...; eight 16-byte loads (FP32: sixteen) are in flight per
// thread and iteration, the ragged end re-reads the last group instead of branching.  BF16 values are
// compared as packed pairs.
template <bool BF16IN>
__global__ void __launch_bounds__(EW_THREADS)
amax_kernel(const void* __restrict__ W, int O, int K, int64_t ldw, unsigned long long* amax_word, uint32_t epoch) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel waits for this one's end itself
  const uint32_t groups_per_row = K / 8;
  const int64_t total = (int64_t)O * groups_per_row;
  const bool dense = ldw == K;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  constexpr int DEPTH = 8;
  float amax = 0.f;
  __nv_bfloat162 mx2 = __float2bfloat162_rn(0.f);
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += DEPTH * stride) {
    if (BF16IN) {
      uint4 raw[DEPTH];
#pragma unroll
      for (int j = 0; j < DEPTH; ++j) {
        const int64_t gj = min(g + j * stride, total - 1);
        raw[j] = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(W) +
                                                 w_offset(gj, groups_per_row, ldw, dense));
      }
#pragma unroll
      for (int j = 0; j < DEPTH; ++j) {
        const uint32_t r[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) mx2 = __hmax2(mx2, __habs2(*reinterpret_cast<const __nv_bfloat162*>(&r[i])));
      }
    } else {
      float4 raw[DEPTH][2];
#pragma unroll
      for (int j = 0; j < DEPTH; ++j) {
        const int64_t gj = min(g + j * stride, total - 1);
        const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(W) +
                                                          w_offset(gj, groups_per_row, ldw, dense));
        raw[j][0] = p[0];
        raw[j][1] = p[1];
      }
#pragma unroll
      for (int j = 0; j < DEPTH; ++j)
#pragma unroll
        for (int h = 0; h < 2; ++h)
          amax = fmaxf(fmaxf(amax, fabsf(raw[j][h].x)),
                       fmaxf(fmaxf(fabsf(raw[j][h].y), fabsf(raw[j][h].z)), fabsf(raw[j][h].w)));
    }
  }
  if (BF16IN) amax = fmaxf(__low2float(mx2), __high2float(mx2));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  __shared__ float s_max[EW_THREADS / 32];
  if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = 0.f;
    for (int i = 0; i < EW_THREADS / 32; ++i) m = fmaxf(m, s_max[i]);
    // non-negative floats order like their bit patterns; the call's serial number on top makes a value left
    // by an earlier call lose against any value of this one, so the word is never cleared between calls
    atomicMax(amax_word, ((unsigned long long)epoch << 32) | __float_as_uint(m));
  }
}

// ---- one thread, one 16-element scale block -----------------------------------------------------
// The set-up and activation kernels give each thread a whole scale block: the block maximum needs no
// exchange, the E4M3 scale is formed once per 16 values, and all 16 quotients w / s share one
// reciprocal.  Outputs wider than the input (V: 64 bytes per thread) pass through shared memory so that
// every global store instruction of a warp covers one contiguous run.
//
// These kernels are bound by the SM's integer/logic pipe (compares, selects, min/max, shifts and
// bit operations issue at half the rate of FP32 multiply-add), so the per-value work is phrased in
// exact FP32 arithmetic wherever that is possible: the region of the node grid comes from two
// saturating multiply-adds, floor() from an addition that rounds down, the nibbles of eight values
// are summed as small integers in FP32.  Every such operation is exact, so the results equal those
// of the compare-and-select formulation bit for bit.

// The 16 values of a block as loaded: 32 bytes of BF16 (in r[0..7]) or 64 bytes of FP32.
struct block_raw {
  uint32_t r[16];
};
template <bool BF16IN>
__device__ __forceinline__ block_raw load_block(const void* W, int64_t idx) {
  block_raw raw;
  if (BF16IN) {
    const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(W) + idx);
    const uint4 r0 = p[0], r1 = p[1];
    raw.r[0] = r0.x; raw.r[1] = r0.y; raw.r[2] = r0.z; raw.r[3] = r0.w;
    raw.r[4] = r1.x; raw.r[5] = r1.y; raw.r[6] = r1.z; raw.r[7] = r1.w;
  } else {
    const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(W) + idx);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint4 r = p[j];
      raw.r[4 * j] = r.x; raw.r[4 * j + 1] = r.y; raw.r[4 * j + 2] = r.z; raw.r[4 * j + 3] = r.w;
    }
  }
  return raw;
}

// Values as binary32, the block maximum of |w|, and whether some magnitude is below 2^-80 (zero included):
// such a block takes the division instruction instead of the shared reciprocal (see block_quotients).
// BF16 input: maximum and minimum run on the packed pairs, two values per instruction.
template <bool BF16IN>
__device__ __forceinline__ float unpack_block(const block_raw& raw, float (&w)[16], bool* has_minute) {
  if (BF16IN) {
    __nv_bfloat162 mx = __habs2(*reinterpret_cast<const __nv_bfloat162*>(&raw.r[0]));
    __nv_bfloat162 mn = mx;
#pragma unroll
    for (int i = 1; i < 8; ++i) {
      const __nv_bfloat162 a = __habs2(*reinterpret_cast<const __nv_bfloat162*>(&raw.r[i]));
      mx = __hmax2(mx, a);
      mn = __hmin2(mn, a);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      w[2 * i] = __uint_as_float(raw.r[i] << 16);
      w[2 * i + 1] = __uint_as_float(raw.r[i] & 0xFFFF0000u);
    }
    *has_minute = fminf(__low2float(mn), __high2float(mn)) < 0x1p-80f;
    return fmaxf(__low2float(mx), __high2float(mx));
  } else {
    float amax = 0.f;
    bool minute = false;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      w[i] = __uint_as_float(raw.r[i]);
      amax = fmaxf(amax, fabsf(w[i]));
      minute |= fabsf(w[i]) < 0x1p-80f;
    }
    *has_minute = minute;
    return amax;
  }
}

// q[i] = w[i] / s, correctly rounded (the result of a binary32 division; rounding to nearest is
// symmetric, so the sign rides along), for the 16 values of a block.
// FAST: r = RN(1/s) once, then per value q0 = RN(w r) and two residual corrections
// e = w - q s (one FMA), q <- RN(q + e r).  After the first correction q is within half a unit of
// w / s plus 2^-47 relative, hence a faithful rounding; the residual of a faithful quotient is exact in
// one FMA, and a faithful quotient corrected once more with the correctly rounded reciprocal is the
// correctly rounded quotient (Markstein's theorem), provided nothing under- or overflows.  The caller
// secures that proviso: s and the block maximum within [2^-40, 2^40] and no magnitude below 2^-80
// keep every quotient, product and residual a normal number.  The corrections run as packed pairs
// (two binary32 lanes per instruction).
// Otherwise (a zero or minute value, an extreme scale): the division instruction sequence.
template <bool FAST>
__device__ __forceinline__ void block_quotients(const float (&w)[16], float s, float (&q)[16]) {
  if (FAST) {
    const float r = __frcp_rn(s);
    const float2 r2 = make_float2(r, r), ns2 = make_float2(-s, -s);
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
      const float2 w2 = make_float2(w[i], w[i + 1]);
      float2 qq = __fmul2_rn(w2, r2);
      float2 e = __ffma2_rn(qq, ns2, w2);
      qq = __ffma2_rn(e, r2, qq);
      e = __ffma2_rn(qq, ns2, w2);
      qq = __ffma2_rn(e, r2, qq);
      q[i] = qq.x;
      q[i + 1] = qq.y;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) q[i] = s > 0.f ? __fdiv_rn(w[i], s) : 0.f;
  }
}

// Position of one scaled magnitude q = min(|w| / s, 6) on the node grid {0, .5, 1, 1.5, 2, 3, 4, 6}.
// The grid has three regions of constant spacing: [0, 2] by 0.5, [2, 4] by 1, [4, 6] by 2 (a value on
// a shared end point gets the same answer from either side).  With t1 = [q > 2], t2 = [q > 4] as 0 / 1
// (q - 2 and q - 4 are multiples of 2^-22 there, so a saturating FMA by 2^22 gives exactly 0 or 1),
//   m = 1 / spacing = 2 - t1 - t2 / 2,  u = q m,  j = floor(u)  (j = 2 throughout the last region:
//   it is a single interval that includes its upper end 6),
//   interval index k = j + 2 t1 + 2 t2,   v = u - j = (q - lower node) / spacing, in [0, 1].
struct grid_pos {
  float k, j, v, t1, t2;
};
__device__ __forceinline__ grid_pos locate(float q_signed) {
  grid_pos g;
  const float q = fminf(fabsf(q_signed), 6.0f);
  g.t1 = __saturatef(__fmaf_rn(q, 0x1p22f, -0x1p23f));
  g.t2 = __saturatef(__fmaf_rn(q, 0x1p22f, -0x1p24f));
  const float m = __fmaf_rn(-0.5f, g.t2, __fsub_rn(2.0f, g.t1));
  const float u = __fmul_rn(q, m);
  const float fl = __fsub_rn(__fadd_rd(u, 0x1p23f), 0x1p23f);      // floor(u): the sum has unit spacing, rounded down
  g.j = __fmaf_rn(g.t2, __fsub_rn(2.0f, fl), fl);
  g.v = __fsub_rn(u, g.j);
  g.k = __fmaf_rn(2.0f, __fadd_rn(g.t1, g.t2), g.j);
  return g;
}

// 1 for a negative value, 0 otherwise (-0.0 counts as positive).  FAST: the quotient is a normal number
// of magnitude at least 2^-120, so its product with -2^126 saturates to 0 or 1.
template <bool FAST>
__device__ __forceinline__ float negative_flag(float w, float q_signed) {
  return FAST ? __saturatef(__fmul_rn(q_signed, -0x1p126f)) : (w < 0.f ? 1.0f : 0.0f);
}

// Eight nibbles given as FP32 integers 0..15 -> one 32-bit word, nibble i at bits 4i.  Four nibbles sum
// exactly in FP32 (below 2^16); adding 2^23 leaves that integer in the low mantissa bits.
__device__ __forceinline__ uint32_t pack_nibbles(const float (&n)[8]) {
  const float lo = __fmaf_rn(n[3], 4096.f, __fmaf_rn(n[2], 256.f, __fmaf_rn(n[1], 16.f, n[0])));
  const float hi = __fmaf_rn(n[7], 4096.f, __fmaf_rn(n[6], 256.f, __fmaf_rn(n[5], 16.f, n[4])));
  return __byte_perm(__float_as_uint(__fadd_rn(lo, 0x1p23f)), __float_as_uint(__fadd_rn(hi, 0x1p23f)), 0x5410);
}

// A warp's threads each hold CH 16-byte chunks that are consecutive in the output (thread t: chunks
// t*CH .. t*CH+CH-1 of the warp's run).  Pass them through the warp's slice of shared memory so that
// store instruction i writes chunks 32 i .. 32 i + 31.  The chunk position inside a thread's group is
// XOR-ed with a few bits of the thread index: without it the 8 threads of a quarter-warp, CH chunks
// apart, would fall on the same banks.
template <int CH>
__device__ __forceinline__ void warp_store_chunks(uint4* stage_warp, const uint4 (&mine)[CH], uint4* out_warp,
                                                  int valid_threads) {
  const int lane = threadIdx.x & 31;
  constexpr int G = 8 / CH;
#pragma unroll
  for (int j = 0; j < CH; ++j) stage_warp[lane * CH + (j ^ ((lane / G) & (CH - 1)))] = mine[j];
  __syncwarp();
#pragma unroll
  for (int i = 0; i < CH; ++i) {
    const int c = i * 32 + lane, t = c / CH, j = c % CH;
    const uint4 x = stage_warp[t * CH + (j ^ ((t / G) & (CH - 1)))];
    if (t < valid_threads) out_warp[c] = x;
  }
  __syncwarp();
}

// Element offset in a row-major tensor of 16-element block b.
__device__ __forceinline__ int64_t block_offset(int64_t b, uint32_t blocks_per_row, int64_t ld, bool dense) {
  if (dense) return b * 16;
  const uint32_t row = (uint32_t)b / blocks_per_row;
  return (int64_t)row * ld + (int64_t)((uint32_t)b - row * blocks_per_row) * 16;
}

__device__ __forceinline__ float tensor_scale(float s_global_in, const unsigned long long* amax_word) {
  if (s_global_in > 0.f) return s_global_in;
  const float amax_t = __uint_as_float((uint32_t)*amax_word);      // low half: the maximum's bits
  return amax_t == 0.f ? 1.0f : __fdiv_rn(amax_t, 2688.0f);
}

__device__ __forceinline__ bool fast_division_ok(float s, float amax, bool has_minute) {
  return s >= 0x1p-40f && s <= 0x1p40f && amax <= 0x1p40f && !has_minute;
}

// ---- pass 2: block scales, bracket, V_init -------------------------------------
// Bracket of w~ = min(|w| / s, 6): interval index k (lower node = node k) and V_init = (w~ - lower node) / width.
template <bool FAST>
__device__ __forceinline__ void bracket_block(const float (&w)[16], float s, float (&v)[16], uint32_t (&cw)[2]) {
  float q[16];
  block_quotients<FAST>(w, s, q);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    float n[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const grid_pos g = locate(q[8 * h + i]);
      v[8 * h + i] = g.v;
      n[i] = __fmaf_rn(8.0f, negative_flag<FAST>(w[8 * h + i], q[8 * h + i]), g.k);
    }
    cw[h] = pack_nibbles(n);
  }
}

template <bool BF16IN>
__global__ void __launch_bounds__(EW_THREADS, 3)
softquant_init_kernel(const void* __restrict__ W, int O, int K, int64_t ldw,
                      float s_global_in, const unsigned long long* __restrict__ amax_word,
                      uint8_t* __restrict__ scales, float* __restrict__ s_global_out,
                      uint8_t* __restrict__ code, float* __restrict__ V) {
  __shared__ uint4 stage[EW_THREADS * 4];
  asm volatile("griddepcontrol.wait;" ::: "memory");      // the maximum (and W itself) may come from the kernel before
  const float s_global = tensor_scale(s_global_in, amax_word);
  if (blockIdx.x == 0 && threadIdx.x == 0) *s_global_out = s_global;
  const float d = __fmul_rn(s_global, 6.0f);

  const uint32_t blocks_per_row = K / 16;
  const int64_t total = (int64_t)O * blocks_per_row;
  const bool dense = ldw == K;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  uint4* stage_warp = stage + (threadIdx.x & ~31) * 4;
  int64_t b0 = (int64_t)blockIdx.x * blockDim.x;
  if (b0 >= total) return;
  // the next block's values are requested before this block's arithmetic starts
  block_raw next = load_block<BF16IN>(W, block_offset(min(b0 + threadIdx.x, total - 1), blocks_per_row, ldw, dense));
  for (; b0 < total; b0 += stride) {
    const int64_t b = b0 + threadIdx.x;
    const bool valid = b < total;
    const block_raw raw = next;
    if (b0 + stride < total)
      next = load_block<BF16IN>(W, block_offset(min(b + stride, total - 1), blocks_per_row, ldw, dense));
    float w[16];
    bool has_minute;
    const float amax = unpack_block<BF16IN>(raw, w, &has_minute);
    const uint32_t sb = faar_float_to_e4m3(__fdiv_rn(amax, d));
    const float s = __fmul_rn(faar_e4m3_to_float(sb), s_global);
    uint32_t cw[2];
    uint4 vq[4];
    float(&v)[16] = *reinterpret_cast<float(*)[16]>(vq);
    if (fast_division_ok(s, amax, has_minute)) bracket_block<true>(w, s, v, cw);
    else bracket_block<false>(w, s, v, cw);
    const int64_t warp_first = b0 + (threadIdx.x & ~31);
    if (warp_first < total) {
      const int64_t left = total - warp_first;
      warp_store_chunks<4>(stage_warp, vq, reinterpret_cast<uint4*>(V + warp_first * 16), left < 32 ? (int)left : 32);
    }
    if (valid) {
      *reinterpret_cast<uint2*>(code + b * 8) = make_uint2(cw[0], cw[1]);
      scales[b] = (uint8_t)sb;
    }
  }
}

// ---- activation fake-quantisation: the X_q of Eq. 5 --------------------------------------------
// Same format and scale rule as the weights; each value goes to the nearest node, a tie to the larger
// magnitude (Eq. 7 applied to the initial position).  The output holds sign * node * block scale, which
// needs at most 7 significant bits and is therefore exact in BF16; the FP32 tensor scale stays outside
// (X_q = Xq_units * s_global) and is applied by the GEMM epilogues.
// From the bracket: t = [v >= 0.5] (v - 0.5 is a multiple of 2^-25, so a saturating FMA by 2^25 gives 0 or 1),
// node = (j + t) * spacing, magnitude code = k + t.
template <bool FAST>
__device__ __forceinline__ void nearest_block(const float (&w)[16], float s, float sg, uint32_t (&o)[8], uint32_t (&cw)[2]) {
  float q[16];
  block_quotients<FAST>(w, s, q);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    float n[8];
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
      float out[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int x = 8 * h + i + e;
        const grid_pos g = locate(q[x]);
        const float t = __saturatef(__fmaf_rn(g.v, 0x1p25f, 1.0f - 0x1p24f));
        const float neg = negative_flag<FAST>(w[x], q[x]);
        n[i + e] = __fmaf_rn(8.0f, neg, __fadd_rn(g.k, t));
        const float spacing_sg = __fmul_rn(__fmaf_rn(0.5f, g.t1, __fadd_rn(0.5f, g.t2)), sg);   // {.5, 1, 2} * sg
        const float mag = __fmul_rn(__fadd_rn(g.j, t), spacing_sg);                          // exact: 3 x 4 bits at most
        out[e] = __fmul_rn(mag, __fmaf_rn(-2.0f, neg, 1.0f));
      }
      // both values have zero low halves: the BF16 pair is the two high halves
      o[(8 * h + i) >> 1] = __byte_perm(__float_as_uint(out[0]), __float_as_uint(out[1]), 0x7632);
    }
    cw[h] = pack_nibbles(n);
  }
}

__global__ void __launch_bounds__(EW_THREADS, 3)
act_fakequant_kernel(const __nv_bfloat16* __restrict__ X, int T, int K, int64_t ldx, float s_global_in,
                     const unsigned long long* __restrict__ amax_word, __nv_bfloat16* __restrict__ Xq, int64_t ldq,
                     float* __restrict__ s_global_out, uint8_t* __restrict__ packed, uint8_t* __restrict__ scales) {
  __shared__ uint4 stage[EW_THREADS * 2];
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const float s_global = tensor_scale(s_global_in, amax_word);
  if (blockIdx.x == 0 && threadIdx.x == 0) *s_global_out = s_global;
  const float d = __fmul_rn(s_global, 6.0f);
  const uint32_t blocks_per_row = K / 16;
  const int64_t total = (int64_t)T * blocks_per_row;
  const bool dense_in = ldx == K, dense_out = ldq == K;
  uint4* stage_warp = stage + (threadIdx.x & ~31) * 2;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t b0 = (int64_t)blockIdx.x * blockDim.x;
  if (b0 >= total) return;
  block_raw next = load_block<true>(X, block_offset(min(b0 + threadIdx.x, total - 1), blocks_per_row, ldx, dense_in));
  for (; b0 < total; b0 += stride) {
    const int64_t b = b0 + threadIdx.x;
    const bool valid = b < total;
    const block_raw raw = next;
    if (b0 + stride < total)
      next = load_block<true>(X, block_offset(min(b + stride, total - 1), blocks_per_row, ldx, dense_in));
    float w[16];
    bool has_minute;
    const float amax = unpack_block<true>(raw, w, &has_minute);
    const uint32_t sb = faar_float_to_e4m3(__fdiv_rn(amax, d));
    const float sg = faar_e4m3_to_float(sb);
    const float s = __fmul_rn(sg, s_global);
    uint32_t cw[2];
    uint4 oq[2];
    uint32_t(&o)[8] = *reinterpret_cast<uint32_t(*)[8]>(oq);
    if (fast_division_ok(s, amax, has_minute)) nearest_block<true>(w, s, sg, o, cw);
    else nearest_block<false>(w, s, sg, o, cw);
    if (dense_out) {
      const int64_t warp_first = b0 + (threadIdx.x & ~31);
      if (warp_first < total) {
        const int64_t left = total - warp_first;
        warp_store_chunks<2>(stage_warp, oq, reinterpret_cast<uint4*>(Xq + warp_first * 16), left < 32 ? (int)left : 32);
      }
    } else if (valid) {
      uint4* p = reinterpret_cast<uint4*>(Xq + block_offset(b, blocks_per_row, ldq, false));
      p[0] = oq[0];
      p[1] = oq[1];
    }
    if (valid) {
      if (packed) *reinterpret_cast<uint2*>(packed + b * 8) = make_uint2(cw[0], cw[1]);
      if (scales) scales[b] = (uint8_t)sb;
    }
  }
}

// ---- packed NVFP4 activations back to the BF16 operand: the inverse of the kernel above -------------------
// out[r][c] = sign * node(code) * block scale (the FP32 tensor scale stays outside, as in act_fakequant's X_q):
// exactly the values act_fakequant wrote, from 4.5 bits per value instead of 16.  One thread per 16-value block.
__global__ void __launch_bounds__(EW_THREADS)
nvfp4_expand_kernel(const uint8_t* __restrict__ packed, const uint8_t* __restrict__ scales, int rows, int K,
                    __nv_bfloat16* __restrict__ out, int64_t ld) {
  const uint32_t blocks_per_row = K / 16;
  const int64_t total = (int64_t)rows * blocks_per_row;
  for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < total; b += (int64_t)gridDim.x * blockDim.x) {
    const uint2 cw = *reinterpret_cast<const uint2*>(packed + b * 8);
    const float sg = faar_e4m3_to_float(scales[b]);
    const uint32_t w[2] = {cw.x, cw.y};
    uint32_t o[8];
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
      uint32_t h[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const uint32_t nib = (w[(i + e) >> 3] >> (4 * ((i + e) & 7))) & 0xFu;
        const float mag = __fmul_rn(faar_node(nib & 7), sg);            // exact: 2 x 4 significant bits
        h[e] = __float_as_uint(mag) | ((nib & 8u) << 28);
      }
      o[i >> 1] = __byte_perm(h[0], h[1], 0x7632);                       // the two high halves: a BF16 pair
    }
    uint4* dst = reinterpret_cast<uint4*>(out + block_offset(b, blocks_per_row, ld, ld == K));
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
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

// Launch with stream serialisation relaxed: the kernel's CTAs may be scheduled while the kernel before
// it drains; the kernel itself waits (griddepcontrol.wait) before it touches global memory.
template <typename... KArgs, typename... Args>
static cudaError_t launch_relaxed(faar_ctx* ctx, void (*kernel)(KArgs...), int grid, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(EW_THREADS, 1, 1);
  cfg.stream = ctx->stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Serial number of a tensor-maximum pass, shared by all contexts of the process (a workspace may pass from one
// context to another).  0 is what a freshly initialised workspace header holds and is skipped.
static std::atomic<uint32_t> g_amax_epoch{0};

static int launch_amax(faar_ctx* ctx, bool bf16, const void* W, int rows, int K, int64_t ld,
                       unsigned long long* amax_word) {
  uint32_t epoch = ++g_amax_epoch;
  if (epoch == 0) {                                        // the counter wrapped: start over from a cleared word
    cudaError_t e = cudaMemsetAsync(amax_word, 0, sizeof(unsigned long long), ctx->stream);
    if (e != cudaSuccess) return (int)e;
    epoch = ++g_amax_epoch;
  }
  const int64_t groups = (int64_t)rows * (K / 8);
  faar_prof_scope ps(ctx, FAAR_K_AMAX);
  const int grid = grid_for(ctx, (groups + 7) / 8, 8);
  if (bf16) amax_kernel<true><<<grid, EW_THREADS, 0, ctx->stream>>>(W, rows, K, ld, amax_word, epoch);
  else amax_kernel<false><<<grid, EW_THREADS, 0, ctx->stream>>>(W, rows, K, ld, amax_word, epoch);
  return (int)cudaGetLastError();
}

int faar_launch_softquant_init(faar_ctx* ctx, const faar_shape* s, const void* W, float s_global_in,
                               uint8_t* scales, float* s_global_out, uint8_t* code, float* V,
                               unsigned long long* amax_word) {
  const int64_t blocks = (int64_t)s->O * (s->K / 16);
  if (!(s_global_in > 0.f)) {
    int e = launch_amax(ctx, s->w_dtype == FAAR_BF16, W, s->O, s->K, s->ldw, amax_word);
    if (e) return e;
  }
  faar_prof_scope ps(ctx, FAAR_K_SOFTQUANT_INIT);
  cudaError_t e = launch_relaxed(ctx, s->w_dtype == FAAR_BF16 ? softquant_init_kernel<true> : softquant_init_kernel<false>,
                                 grid_for(ctx, blocks, 3), W, s->O, s->K, s->ldw, s_global_in,
                                 (const unsigned long long*)amax_word, scales, s_global_out, code, V);
  if (e != cudaSuccess) return (int)e;
  return (int)cudaGetLastError();
}

int faar_launch_act_fakequant(faar_ctx* ctx, int T, int K, const void* X, int64_t ldx, float s_global_in, void* Xq,
                              int64_t ldq, float* s_global_out, uint8_t* packed, uint8_t* scales,
                              unsigned long long* amax_word) {
  const int64_t blocks = (int64_t)T * (K / 16);
  if (!(s_global_in > 0.f)) {
    int e = launch_amax(ctx, true, X, T, K, ldx, amax_word);
    if (e) return e;
  }
  faar_prof_scope ps(ctx, FAAR_K_ACT_FAKEQUANT);
  cudaError_t e = launch_relaxed(ctx, act_fakequant_kernel, grid_for(ctx, blocks, 3),
                                 reinterpret_cast<const __nv_bfloat16*>(X), T, K, ldx, s_global_in,
                                 (const unsigned long long*)amax_word, reinterpret_cast<__nv_bfloat16*>(Xq), ldq,
                                 s_global_out, packed, scales);
  if (e != cudaSuccess) return (int)e;
  return (int)cudaGetLastError();
}

int faar_launch_nvfp4_expand(faar_ctx* ctx, int rows, int K, const uint8_t* packed, const uint8_t* scales, void* out,
                             int64_t ld) {
  const int64_t blocks = (int64_t)rows * (K / 16);
  faar_prof_scope ps(ctx, FAAR_K_ACT_FAKEQUANT);
  nvfp4_expand_kernel<<<grid_for(ctx, blocks, 8), EW_THREADS, 0, ctx->stream>>>(packed, scales, rows, K,
                                                                               reinterpret_cast<__nv_bfloat16*>(out), ld);
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
