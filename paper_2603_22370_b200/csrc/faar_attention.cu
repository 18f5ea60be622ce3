// Causal softmax attention with grouped key/value heads, forward and backward, for full-model alignment
// (Eq. 6, Procedure steps 16-23: the loss is back-propagated through the whole quantised model, and between a
// block's q/k/v projections and its output projection sits the model family's attention).
//
//   out[t, h, :] = sum_{u <= t, same sequence} softmax_u(q[t, h, :] . k[u, g, :] / sqrt(D)) v[u, g, :],   g = h / (H / Hkv)
//
// q, out: [B*S, H*D]; k, v: [B*S, Hkv*D]; BF16, tokens of a sequence contiguous.  Tiles of 64 queries x 64 keys;
// every matrix product runs on the tensor cores through the warp-level 16 x 16 x 16 BF16 fragments (FP32
// accumulation), every intermediate (scores, probabilities) goes through shared memory between two products.
// Nothing of size S x S touches global memory: the forward pass makes two sweeps over the keys (row maximum and
// sum first, then the normalised probabilities times V), which keeps the output accumulators free of rescaling,
// and stores one number per query row, lse = log2 sum_u 2^(score_u), for the backward pass.  The backward pass
// recomputes the probabilities from lse in two kernels, each accumulating its own result in registers and writing
// it once: dK, dV per key tile (loop over the query tiles at or below it and over the query heads of the group),
// dQ per query tile (loop over the key tiles at or above it).  No atomics: results are reproducible.
#include <mma.h>

#include "faar_internal.cuh"

namespace {

using namespace nvcuda;

constexpr int AT = 64;                       // queries / keys per tile
constexpr int ATT_THREADS = 128;             // 4 warps, each owning 16 rows of the tile
constexpr float LOG2E = 1.4426950408889634f;

struct AttnParams {
  const __nv_bfloat16* q; const __nv_bfloat16* k; const __nv_bfloat16* v;
  __nv_bfloat16* out; float* lse;            // lse: [B, H, S], log2 domain
  const __nv_bfloat16* dout; const float* dsum;   // backward: dO and rowsum(dO * O) [B, H, S]
  __nv_bfloat16* dq; __nv_bfloat16* dk; __nv_bfloat16* dv;
  long long ldq, ldk, ldo;                   // row strides (elements) of q / dq, of k / v / dk / dv, of out / dout
  int B, S, H, Hkv;
  float scale_log2;                          // log2(e) / sqrt(D)
};

// rows [row0, row0 + 64) x D of a [.., ld] BF16 matrix (column offset col0) into shared memory tile[64][D + 8];
// rows at or beyond row_end are zero.
template <int D>
__device__ __forceinline__ void load_tile(__nv_bfloat16 (*tile)[D + 8], const __nv_bfloat16* src, long long ld, long long row0,
                                          long long row_end, int col0) {
  for (int i = threadIdx.x; i < AT * (D / 8); i += ATT_THREADS) {
    const int r = i / (D / 8), c = (i % (D / 8)) * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row0 + r < row_end) v = *reinterpret_cast<const uint4*>(src + (row0 + r) * ld + col0 + c);
    *reinterpret_cast<uint4*>(&tile[r][c]) = v;
  }
}

// ---- forward ---------------------------------------------------------------------------------------------
// grid (query tiles, H, B).  Warp w owns query rows 16 w .. 16 w + 15 of the tile; two lanes share a row in the
// element-wise phases (lane = 2 * row + half, 32 of the 64 key columns each).
template <int D>
__global__ void __launch_bounds__(ATT_THREADS)
attn_fwd_kernel(const AttnParams p) {
  extern __shared__ __align__(128) uint8_t att_smem[];
  auto Qs = reinterpret_cast<__nv_bfloat16(*)[D + 8]>(att_smem);
  auto Ks = reinterpret_cast<__nv_bfloat16(*)[D + 8]>(att_smem + AT * (D + 8) * 2);
  auto Vs = reinterpret_cast<__nv_bfloat16(*)[D + 8]>(att_smem + 2 * AT * (D + 8) * 2);
  float* Sall = reinterpret_cast<float*>(att_smem + 3 * AT * (D + 8) * 2);              // [4 warps][16][64 + 4]
  __nv_bfloat16* Pall = reinterpret_cast<__nv_bfloat16*>(Sall + 4 * 16 * (AT + 4));     // [4 warps][16][64 + 8]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* Sw = Sall + warp * 16 * (AT + 4);
  __nv_bfloat16* Pw = Pall + warp * 16 * (AT + 8);
  const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int g = h / (p.H / p.Hkv);
  const long long seq0 = (long long)b * p.S;
  const int q0 = qt * AT;
  load_tile<D>(Qs, p.q, p.ldq, seq0 + q0, seq0 + p.S, h * D);
  const int row = lane >> 1, half = lane & 1;            // this lane's row of the warp's 16 and its 32 columns
  const int qi = q0 + 16 * warp + row;                   // position of that query in its sequence
  float m_run = -INFINITY, l_run = 0.f;
  wmma::fragment<wmma::accumulator, 16, 16, 16, float> oacc[D / 16];
#pragma unroll
  for (int n = 0; n < D / 16; ++n) wmma::fill_fragment(oacc[n], 0.f);

  __syncthreads();
  wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::row_major> qf[D / 16];      // this warp's queries, kept
#pragma unroll
  for (int kk = 0; kk < D / 16; ++kk) wmma::load_matrix_sync(qf[kk], &Qs[16 * warp][16 * kk], D + 8);

  for (int pass = 0; pass < 2; ++pass) {
    for (int kt = 0; kt <= qt; ++kt) {
      const int k0 = kt * AT;
      __syncthreads();                                    // the previous tile's readers are done
      load_tile<D>(Ks, p.k, p.ldk, seq0 + k0, seq0 + p.S, g * D);
      if (pass == 1) load_tile<D>(Vs, p.v, p.ldk, seq0 + k0, seq0 + p.S, g * D);
      __syncthreads();
      // scores of this warp's 16 queries against the 64 keys
      {
        wmma::fragment<wmma::accumulator, 16, 16, 16, float> sacc[AT / 16];
#pragma unroll
        for (int n = 0; n < AT / 16; ++n) wmma::fill_fragment(sacc[n], 0.f);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
#pragma unroll
          for (int n = 0; n < AT / 16; ++n) {
            wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::col_major> bf;
            wmma::load_matrix_sync(bf, &Ks[16 * n][16 * kk], D + 8);
            wmma::mma_sync(sacc[n], qf[kk], bf, sacc[n]);
          }
        }
#pragma unroll
        for (int n = 0; n < AT / 16; ++n) wmma::store_matrix_sync(Sw + 16 * n, sacc[n], AT + 4, wmma::mem_row_major);
      }
      __syncwarp();
      // element-wise phase: this lane takes the columns half, half + 2, ... of its row (two lanes interleave,
      // so that a warp's accesses spread over the shared-memory banks)
      float* srow = Sw + row * (AT + 4) + half;
      if (pass == 0) {
        float mx = -INFINITY;
#pragma unroll 8
        for (int c = 0; c < 32; ++c) {
          const int kj = k0 + half + 2 * c;
          const float s = (kj <= qi && kj < p.S) ? srow[2 * c] * p.scale_log2 : -INFINITY;
          srow[2 * c] = s;
          mx = fmaxf(mx, s);
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        const float m_new = fmaxf(m_run, mx);
        float sum = 0.f;
        if (m_new > -INFINITY) {
#pragma unroll 8
          for (int c = 0; c < 32; ++c) sum += exp2f(srow[2 * c] - m_new);
        }
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        l_run = (m_run > -INFINITY ? l_run * exp2f(m_run - m_new) : 0.f) + sum;
        m_run = m_new;
      } else {
        const float inv_l = l_run > 0.f ? 1.0f / l_run : 0.f;
        __nv_bfloat16* prow = Pw + row * (AT + 8) + half;
#pragma unroll 8
        for (int c = 0; c < 32; ++c) {
          const int kj = k0 + half + 2 * c;
          const float pr = (kj <= qi && kj < p.S) ? exp2f(srow[2 * c] * p.scale_log2 - m_run) * inv_l : 0.f;
          prow[2 * c] = __float2bfloat16_rn(pr);
        }
        __syncwarp();
#pragma unroll
        for (int kk = 0; kk < AT / 16; ++kk) {
          wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::row_major> a;
          wmma::load_matrix_sync(a, Pw + 16 * kk, AT + 8);
#pragma unroll
          for (int n = 0; n < D / 16; ++n) {
            wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::row_major> bf;
            wmma::load_matrix_sync(bf, &Vs[16 * kk][16 * n], D + 8);
            wmma::mma_sync(oacc[n], a, bf, oacc[n]);
          }
        }
      }
      __syncwarp();
    }
  }
  // output rows of this warp: fragments -> shared (FP32) -> BF16 -> global
  __syncthreads();
  float* Ow = reinterpret_cast<float*>(att_smem) + warp * 16 * (D + 4);      // reuses the Q / K tiles' space
#pragma unroll
  for (int n = 0; n < D / 16; ++n) wmma::store_matrix_sync(Ow + 16 * n, oacc[n], D + 4, wmma::mem_row_major);
  __syncwarp();
  if (qi < p.S) {
    __nv_bfloat16* orow = p.out + (seq0 + qi) * p.ldo + h * D + (D / 2) * half;
    const float* src = Ow + row * (D + 4) + (D / 2) * half;
#pragma unroll
    for (int c = 0; c < D / 2; c += 2) {
      __nv_bfloat162 v2 = __floats2bfloat162_rn(src[c], src[c + 1]);
      *reinterpret_cast<__nv_bfloat162*>(orow + c) = v2;
    }
    if (half == 0) p.lse[((long long)b * p.H + h) * p.S + qi] = m_run + log2f(l_run);
  }
}

// ---- backward, step 0: dsum[b, h, t] = sum_d dO[t, h, d] * O[t, h, d] ------------------------------------------
// D / 8 lanes share one (token, head) row, 16 bytes of O and of dO each, so a warp takes 256 / D consecutive tokens
// of one head per pass; consecutive warps take the heads of the same tokens (whole rows of O and dO are read
// together), and a warp's results are consecutive floats of dsum.
template <int D>
__global__ void __launch_bounds__(ATT_THREADS)
attn_dsum_kernel(const AttnParams p, float* dsum) {
  constexpr int LPR = D / 8, RPW = 32 / LPR;                 // lanes per row, rows per warp
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPR, c = (lane % LPR) * 8;
  const int nq = (p.S + RPW - 1) / RPW;
  const long long total = (long long)p.B * p.H * nq;
  for (long long i = (long long)blockIdx.x * (ATT_THREADS / 32) + warp; i < total; i += (long long)gridDim.x * (ATT_THREADS / 32)) {
    const int h = (int)(i % p.H);
    const long long r = i / p.H;
    const int tq = (int)(r % nq);
    const long long b = r / nq;
    const int sidx = tq * RPW + sub;
    float acc = 0.f;
    if (sidx < p.S) {
      const long long off = (b * p.S + sidx) * p.ldo + h * D + c;
      const uint4 ov = *reinterpret_cast<const uint4*>(p.out + off);
      const uint4 dv = *reinterpret_cast<const uint4*>(p.dout + off);
      const uint32_t ow[4] = {ov.x, ov.y, ov.z, ov.w}, dw[4] = {dv.x, dv.y, dv.z, dv.w};
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        acc = fmaf(__uint_as_float(ow[k] << 16), __uint_as_float(dw[k] << 16), acc);
        acc = fmaf(__uint_as_float(ow[k] & 0xFFFF0000u), __uint_as_float(dw[k] & 0xFFFF0000u), acc);
      }
    }
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (lane % LPR == 0 && sidx < p.S) dsum[(b * p.H + h) * p.S + sidx] = acc;
  }
}

// ---- backward, dK and dV of one key tile --------------------------------------------------------------------
// grid (key tiles, Hkv, B).  Warp w owns keys 16 w .. 16 w + 15 of the tile: it forms the 64 x 16 slices of the
// scores, probabilities and their gradients that belong to its keys and accumulates dV[16 x D] += P^T dO and
// dK[16 x D] += dS^T Q over the query tiles at or below the key tile and over the query heads of the group.
// In the element-wise phase a lane owns two query rows (lane, lane + 32) and the 16 keys of its warp.
template <int D>
__global__ void __launch_bounds__(ATT_THREADS)
attn_dkv_kernel(const AttnParams p) {
  extern __shared__ __align__(128) uint8_t att_smem[];
  constexpr int TILE = AT * (D + 8) * 2;
  auto Ks = reinterpret_cast<__nv_bfloat16(*)[D + 8]>(att_smem);
  auto Vs = reinterpret_cast<__nv_bfloat16(*)[D + 8]>(att_smem + TILE);
  auto Qs = reinterpret_cast<__nv_bfloat16(*)[D + 8]>(att_smem + 2 * TILE);
  auto Ds = reinterpret_cast<__nv_bfloat16(*)[D + 8]>(att_smem + 3 * TILE);                 // dO tile
  float* Sall = reinterpret_cast<float*>(att_smem + 4 * TILE);                              // P, FP32: [4 warps][64][20]
  float* Gall = Sall + 4 * AT * 20;                                                         // dP, FP32: [4 warps][64][20]
  __nv_bfloat16* Pall = reinterpret_cast<__nv_bfloat16*>(Gall + 4 * AT * 20);               // P then dS, BF16: [4][64][24]
  float* rowv = reinterpret_cast<float*>(Pall + 4 * AT * 24);                               // lse[64], dsum[64]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* Sw = Sall + warp * AT * 20;
  float* Gw = Gall + warp * AT * 20;
  __nv_bfloat16* Pw = Pall + warp * AT * 24;
  const int kt = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int rep = p.H / p.Hkv;
  const long long seq0 = (long long)b * p.S;
  const int k0 = kt * AT;
  const int n_qt = (p.S + AT - 1) / AT;
  load_tile<D>(Ks, p.k, p.ldk, seq0 + k0, seq0 + p.S, g * D);
  load_tile<D>(Vs, p.v, p.ldk, seq0 + k0, seq0 + p.S, g * D);
  wmma::fragment<wmma::accumulator, 16, 16, 16, float> dkacc[D / 16], dvacc[D / 16];
#pragma unroll
  for (int n = 0; n < D / 16; ++n) { wmma::fill_fragment(dkacc[n], 0.f); wmma::fill_fragment(dvacc[n], 0.f); }
  const float inv_sqrt_d = p.scale_log2 / LOG2E;

  for (int hh = 0; hh < rep; ++hh) {
    const int h = g * rep + hh;
    for (int qt = kt; qt < n_qt; ++qt) {
      const int q0 = qt * AT;
      __syncthreads();
      load_tile<D>(Qs, p.q, p.ldq, seq0 + q0, seq0 + p.S, h * D);
      load_tile<D>(Ds, p.dout, p.ldo, seq0 + q0, seq0 + p.S, h * D);
      if (threadIdx.x < AT) {
        const int qi = q0 + threadIdx.x;
        const long long o = ((long long)b * p.H + h) * p.S + qi;
        rowv[threadIdx.x] = qi < p.S ? p.lse[o] : 0.f;
        rowv[AT + threadIdx.x] = qi < p.S ? p.dsum[o] : 0.f;
      }
      __syncthreads();
      // S = Q K^T and dP = dO V^T for [64 queries][this warp's 16 keys]
#pragma unroll
      for (int m = 0; m < AT / 16; ++m) {
        wmma::fragment<wmma::accumulator, 16, 16, 16, float> sacc, gacc;
        wmma::fill_fragment(sacc, 0.f);
        wmma::fill_fragment(gacc, 0.f);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::row_major> a;
          wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::col_major> bf;
          wmma::load_matrix_sync(a, &Qs[16 * m][16 * kk], D + 8);
          wmma::load_matrix_sync(bf, &Ks[16 * warp][16 * kk], D + 8);
          wmma::mma_sync(sacc, a, bf, sacc);
          wmma::load_matrix_sync(a, &Ds[16 * m][16 * kk], D + 8);
          wmma::load_matrix_sync(bf, &Vs[16 * warp][16 * kk], D + 8);
          wmma::mma_sync(gacc, a, bf, gacc);
        }
        wmma::store_matrix_sync(Sw + 16 * m * 20, sacc, 20, wmma::mem_row_major);
        wmma::store_matrix_sync(Gw + 16 * m * 20, gacc, 20, wmma::mem_row_major);
      }
      __syncwarp();
      // P = 2^(score - lse) under the causal mask -> BF16 for dV
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const int r = lane + 32 * rr, qi = q0 + r;
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          const int kj = k0 + 16 * warp + c;
          const float pr = (kj <= qi && qi < p.S) ? exp2f(Sw[r * 20 + c] * p.scale_log2 - rowv[r]) : 0.f;
          Sw[r * 20 + c] = pr;
          Pw[r * 24 + c] = __float2bfloat16_rn(pr);
        }
      }
      __syncwarp();
#pragma unroll
      for (int kk = 0; kk < AT / 16; ++kk) {                   // dV += P^T dO
        wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::col_major> a;      // A[key][query] = P[query][key]
        wmma::load_matrix_sync(a, Pw + 16 * kk * 24, 24);
#pragma unroll
        for (int n = 0; n < D / 16; ++n) {
          wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::row_major> bf;
          wmma::load_matrix_sync(bf, &Ds[16 * kk][16 * n], D + 8);
          wmma::mma_sync(dvacc[n], a, bf, dvacc[n]);
        }
      }
      __syncwarp();
      // dS = P (dP - dsum) / sqrt(D) -> BF16 for dK
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const int r = lane + 32 * rr;
#pragma unroll
        for (int c = 0; c < 16; ++c)
          Pw[r * 24 + c] = __float2bfloat16_rn(Sw[r * 20 + c] * (Gw[r * 20 + c] - rowv[AT + r]) * inv_sqrt_d);
      }
      __syncwarp();
#pragma unroll
      for (int kk = 0; kk < AT / 16; ++kk) {                   // dK += dS^T Q
        wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::col_major> a;
        wmma::load_matrix_sync(a, Pw + 16 * kk * 24, 24);
#pragma unroll
        for (int n = 0; n < D / 16; ++n) {
          wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::row_major> bf;
          wmma::load_matrix_sync(bf, &Qs[16 * kk][16 * n], D + 8);
          wmma::mma_sync(dkacc[n], a, bf, dkacc[n]);
        }
      }
      __syncwarp();
    }
  }
  // this warp's 16 keys of dK and dV: fragments -> shared (FP32) -> BF16 -> global
  __syncthreads();
  float* Ow = reinterpret_cast<float*>(att_smem + 2 * TILE) + warp * 16 * (D + 4);          // the Q / dO tiles' space
  const int r = lane >> 1, half = lane & 1;
  const int kj = k0 + 16 * warp + r;
  for (int which = 0; which < 2; ++which) {
#pragma unroll
    for (int n = 0; n < D / 16; ++n)
      wmma::store_matrix_sync(Ow + 16 * n, which ? dvacc[n] : dkacc[n], D + 4, wmma::mem_row_major);
    __syncwarp();
    if (kj < p.S) {
      __nv_bfloat16* dst = (which ? p.dv : p.dk) + (seq0 + kj) * p.ldk + g * D + (D / 2) * half;
      const float* src = Ow + r * (D + 4) + (D / 2) * half;
#pragma unroll
      for (int c = 0; c < D / 2; c += 2) *reinterpret_cast<__nv_bfloat162*>(dst + c) = __floats2bfloat162_rn(src[c], src[c + 1]);
    }
    __syncwarp();
  }
}

// ---- backward, dQ of one query tile --------------------------------------------------------------------------
// grid (query tiles, H, B).  Warp w owns queries 16 w .. 16 w + 15: scores and dP against every key tile up to
// its own, dS, and dQ[16 x D] += dS K.  Two lanes share a row in the element-wise phase, as in the forward.
template <int D>
__global__ void __launch_bounds__(ATT_THREADS)
attn_dq_kernel(const AttnParams p) {
  extern __shared__ __align__(128) uint8_t att_smem[];
  constexpr int TILE = AT * (D + 8) * 2;
  auto Qs = reinterpret_cast<__nv_bfloat16(*)[D + 8]>(att_smem);
  auto Ds = reinterpret_cast<__nv_bfloat16(*)[D + 8]>(att_smem + TILE);
  auto Ks = reinterpret_cast<__nv_bfloat16(*)[D + 8]>(att_smem + 2 * TILE);
  auto Vs = reinterpret_cast<__nv_bfloat16(*)[D + 8]>(att_smem + 3 * TILE);
  float* Sall = reinterpret_cast<float*>(att_smem + 4 * TILE);                              // [4 warps][16][68]
  float* Gall = Sall + 4 * 16 * (AT + 4);
  __nv_bfloat16* Pall = reinterpret_cast<__nv_bfloat16*>(Gall + 4 * 16 * (AT + 4));         // dS, BF16: [4][16][72]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* Sw = Sall + warp * 16 * (AT + 4);
  float* Gw = Gall + warp * 16 * (AT + 4);
  __nv_bfloat16* Pw = Pall + warp * 16 * (AT + 8);
  const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int g = h / (p.H / p.Hkv);
  const long long seq0 = (long long)b * p.S;
  const int q0 = qt * AT;
  load_tile<D>(Qs, p.q, p.ldq, seq0 + q0, seq0 + p.S, h * D);
  load_tile<D>(Ds, p.dout, p.ldo, seq0 + q0, seq0 + p.S, h * D);
  const int row = lane >> 1, half = lane & 1;
  const int qi = q0 + 16 * warp + row;
  const long long ro = ((long long)b * p.H + h) * p.S + qi;
  const float lse = qi < p.S ? p.lse[ro] : 0.f;
  const float dsum = qi < p.S ? p.dsum[ro] : 0.f;
  const float inv_sqrt_d = p.scale_log2 / LOG2E;
  wmma::fragment<wmma::accumulator, 16, 16, 16, float> dqacc[D / 16];
#pragma unroll
  for (int n = 0; n < D / 16; ++n) wmma::fill_fragment(dqacc[n], 0.f);

  for (int kt = 0; kt <= qt; ++kt) {
    const int k0 = kt * AT;
    __syncthreads();
    load_tile<D>(Ks, p.k, p.ldk, seq0 + k0, seq0 + p.S, g * D);
    load_tile<D>(Vs, p.v, p.ldk, seq0 + k0, seq0 + p.S, g * D);
    __syncthreads();
#pragma unroll
    for (int n = 0; n < AT / 16; ++n) {
      wmma::fragment<wmma::accumulator, 16, 16, 16, float> sacc, gacc;
      wmma::fill_fragment(sacc, 0.f);
      wmma::fill_fragment(gacc, 0.f);
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::row_major> a;
        wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::col_major> bf;
        wmma::load_matrix_sync(a, &Qs[16 * warp][16 * kk], D + 8);
        wmma::load_matrix_sync(bf, &Ks[16 * n][16 * kk], D + 8);
        wmma::mma_sync(sacc, a, bf, sacc);
        wmma::load_matrix_sync(a, &Ds[16 * warp][16 * kk], D + 8);
        wmma::load_matrix_sync(bf, &Vs[16 * n][16 * kk], D + 8);
        wmma::mma_sync(gacc, a, bf, gacc);
      }
      wmma::store_matrix_sync(Sw + 16 * n, sacc, AT + 4, wmma::mem_row_major);
      wmma::store_matrix_sync(Gw + 16 * n, gacc, AT + 4, wmma::mem_row_major);
    }
    __syncwarp();
    {
      const float* srow = Sw + row * (AT + 4) + 32 * half;
      const float* grow = Gw + row * (AT + 4) + 32 * half;
      __nv_bfloat16* prow = Pw + row * (AT + 8) + 32 * half;
#pragma unroll 8
      for (int c = 0; c < 32; ++c) {
        const int kj = k0 + 32 * half + c;
        const float pr = (kj <= qi && qi < p.S) ? exp2f(srow[c] * p.scale_log2 - lse) : 0.f;
        prow[c] = __float2bfloat16_rn(pr * (grow[c] - dsum) * inv_sqrt_d);
      }
    }
    __syncwarp();
#pragma unroll
    for (int kk = 0; kk < AT / 16; ++kk) {                     // dQ += dS K
      wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::row_major> a;
      wmma::load_matrix_sync(a, Pw + 16 * kk, AT + 8);
#pragma unroll
      for (int n = 0; n < D / 16; ++n) {
        wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::row_major> bf;
        wmma::load_matrix_sync(bf, &Ks[16 * kk][16 * n], D + 8);
        wmma::mma_sync(dqacc[n], a, bf, dqacc[n]);
      }
    }
    __syncwarp();
  }
  __syncthreads();
  float* Ow = reinterpret_cast<float*>(att_smem + 2 * TILE) + warp * 16 * (D + 4);          // the K / V tiles' space
#pragma unroll
  for (int n = 0; n < D / 16; ++n) wmma::store_matrix_sync(Ow + 16 * n, dqacc[n], D + 4, wmma::mem_row_major);
  __syncwarp();
  if (qi < p.S) {
    __nv_bfloat16* dst = p.dq + (seq0 + qi) * p.ldq + h * D + (D / 2) * half;
    const float* src = Ow + row * (D + 4) + (D / 2) * half;
#pragma unroll
    for (int c = 0; c < D / 2; c += 2) *reinterpret_cast<__nv_bfloat162*>(dst + c) = __floats2bfloat162_rn(src[c], src[c + 1]);
  }
}

// =====================================================================================================
// head_dim 64: the same three kernels with every intermediate kept in registers.  The matrix products are
// mma.sync m16n8k16 (BF16 in, FP32 accumulate) whose accumulator layout is documented: lane l holds, of a
// 16 x 8 tile, rows l / 4 and l / 4 + 8, columns 2 (l % 4) and 2 (l % 4) + 1.  Two neighbouring accumulator
// tiles are exactly the A operand of the next product (rows the same, 16 contraction columns), so the scores
// become probabilities and then the left operand of P V without leaving the register file; row maxima and sums
// are reduced over the four lanes that share a row.  Operands come from shared memory through ldmatrix (rows
// of D + 8 elements: 16-byte aligned and conflict-free); the forward pass makes one sweep over the keys with a
// running maximum (the output accumulators are rescaled in place).
// =====================================================================================================
constexpr int HD = 64;                       // head_dim of this path
constexpr int LDS = HD + 8;                  // shared-memory row stride (elements)

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void* ptr) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(ptr);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], const void* ptr) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(ptr);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
// D[16 x 8] += A[16 x 16] B[16 x 8]
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
// A operand (16 rows of `tile` from row0, contraction columns 16 kk ..): a0 rows 0-7 / k 0-7, a1 rows 8-15 / k 0-7,
// a2 rows 0-7 / k 8-15, a3 rows 8-15 / k 8-15.
__device__ __forceinline__ void load_a(uint32_t (&a)[4], const __nv_bfloat16 (*tile)[LDS], int row0, int kk, int lane) {
  ldsm_x4(a, &tile[row0 + (lane & 15)][16 * kk + 8 * (lane >> 4)]);
}
// B operands for two neighbouring 8-column tiles when B[k][n] = tile[n][k] (the tile's rows are the output
// columns: Q K^T style): r0, r1 for columns n0 .. n0 + 7, r2, r3 for n0 + 8 .. n0 + 15; contraction 16 kk ..
__device__ __forceinline__ void load_b_rows(uint32_t (&r)[4], const __nv_bfloat16 (*tile)[LDS], int n0, int kk, int lane) {
  ldsm_x4(r, &tile[n0 + (lane & 7) + 8 * (lane >> 4)][16 * kk + 8 * ((lane >> 3) & 1)]);
}
// B operands for two neighbouring 8-column tiles when B[k][n] = tile[k][n] (the tile's rows are contracted:
// P V style): contraction rows k0 .. k0 + 15, r0, r1 for columns n0 .. n0 + 7, r2, r3 for n0 + 8 .. n0 + 15.
__device__ __forceinline__ void load_b_cols(uint32_t (&r)[4], const __nv_bfloat16 (*tile)[LDS], int k0, int n0, int lane) {
  ldsm_x4_t(r, &tile[k0 + (lane & 7) + 8 * ((lane >> 3) & 1)][n0 + 8 * (lane >> 4)]);
}

// S[16 x 64] = A-rows (fragments af[4], contraction over head_dim) times tile^T
__device__ __forceinline__ void scores_16x64(float (&acc)[8][4], const uint32_t (&af)[HD / 16][4], const __nv_bfloat16 (*tile)[LDS],
                                             int lane) {
#pragma unroll
  for (int n = 0; n < 8; ++n) { acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f; }
#pragma unroll
  for (int kk = 0; kk < HD / 16; ++kk) {
#pragma unroll
    for (int n2 = 0; n2 < 4; ++n2) {
      uint32_t b[4];
      load_b_rows(b, tile, 16 * n2, kk, lane);
      mma16816(acc[2 * n2], af[kk], b[0], b[1]);
      mma16816(acc[2 * n2 + 1], af[kk], b[2], b[3]);
    }
  }
}
// out[16 x 64] += P[16 x 64] (as A fragments pf[4]) times tile (rows contracted)
__device__ __forceinline__ void accumulate_16x64(float (&out)[8][4], const uint32_t (&pf)[4][4], const __nv_bfloat16 (*tile)[LDS], int lane) {
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
    for (int n2 = 0; n2 < 4; ++n2) {
      uint32_t b[4];
      load_b_cols(b, tile, 16 * kk, 16 * n2, lane);
      mma16816(out[2 * n2], pf[kk], b[0], b[1]);
      mma16816(out[2 * n2 + 1], pf[kk], b[2], b[3]);
    }
  }
}
// accumulator tiles -> A fragments of the next product
__device__ __forceinline__ void to_a_frags(uint32_t (&pf)[4][4], const float (&acc)[8][4]) {
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
    pf[kk][0] = pack2(acc[2 * kk][0], acc[2 * kk][1]);
    pf[kk][1] = pack2(acc[2 * kk][2], acc[2 * kk][3]);
    pf[kk][2] = pack2(acc[2 * kk + 1][0], acc[2 * kk + 1][1]);
    pf[kk][3] = pack2(acc[2 * kk + 1][2], acc[2 * kk + 1][3]);
  }
}
// a warp's 16 x 64 accumulator as BF16 rows of a [.., ld] matrix (rows row0 + l/4 and + 8, valid below row_end)
__device__ __forceinline__ void store_16x64(__nv_bfloat16* base, long long ld, long long row0, long long row_end, int col0,
                                            const float (&acc)[8][4], float s0, float s1, int lane) {
  const long long r0 = row0 + (lane >> 2), r1 = r0 + 8;
#pragma unroll
  for (int n = 0; n < 8; ++n) {
    const int c = col0 + 8 * n + 2 * (lane & 3);
    if (r0 < row_end) *reinterpret_cast<uint32_t*>(base + r0 * ld + c) = pack2(acc[n][0] * s0, acc[n][1] * s0);
    if (r1 < row_end) *reinterpret_cast<uint32_t*>(base + r1 * ld + c) = pack2(acc[n][2] * s1, acc[n][3] * s1);
  }
}

// ---- asynchronous tile copies (cp.async, 16 bytes each; rows at or beyond row_end arrive as zeros) ------------
__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool valid) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
  const int n = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// ROWS x 64 BF16 tile of `src` (rows row0 .., columns col0 ..) into tile[ROWS][LDS], by NT threads
template <int ROWS, int NT>
__device__ __forceinline__ void tile_async(__nv_bfloat16 (*tile)[LDS], const __nv_bfloat16* src, long long ld, long long row0,
                                           long long row_end, int col0) {
  for (int i = threadIdx.x; i < ROWS * (HD / 8); i += NT) {
    const int r = i >> 3, c = (i & 7) * 8;
    const bool valid = row0 + r < row_end;
    cp_async16(&tile[r][c], src + (valid ? row0 + r : row0) * ld + col0 + c, valid);
  }
}

// ---- forward, head_dim 64: grid (128-query tiles, H, B); 8 warps, warp w owns queries 16 w .. 16 w + 15 ----------
// Key / value tiles of 64 keys run through a three-stage cp.async ring (the copy of tile t + 2 is issued before
// the products of tile t), one block-wide barrier per tile.  The query tile first sits in the ring's third
// stage; once every warp holds its query fragments the stage joins the ring.  A warp skips key tiles that lie
// wholly above its rows' diagonal and masks only where a tile crosses it (or the sequence end).
constexpr int FQ = 128;
constexpr int FWD_THREADS = 256;
constexpr int STAGE_ELEMS = 2 * AT * LDS;            // a K tile and a V tile; equals one 128-row query tile
constexpr int FWD64_SMEM = 3 * STAGE_ELEMS * 2;
__global__ void __launch_bounds__(FWD_THREADS, 2)
attn_fwd64_kernel(const AttnParams p) {
  extern __shared__ __align__(128) uint8_t att_smem[];
  auto stage_k = [&](int s) { return reinterpret_cast<__nv_bfloat16(*)[LDS]>(att_smem) + (size_t)s * 2 * AT; };
  auto stage_v = [&](int s) { return stage_k(s) + AT; };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;      // longest tiles first
  const int h = blockIdx.y, b = blockIdx.z;
  const int g = h / (p.H / p.Hkv);
  const long long seq0 = (long long)b * p.S;
  const int q0 = qt * FQ;
  const int last_q = min(q0 + FQ, p.S) - 1;
  const int n_kt = last_q / AT + 1;                          // key tiles that some query of this tile sees
  auto load_kv = [&](int kt) {
    if (kt < n_kt) {
      tile_async<AT, FWD_THREADS>(stage_k(kt % 3), p.k, p.ldk, seq0 + kt * AT, seq0 + p.S, g * HD);
      tile_async<AT, FWD_THREADS>(stage_v(kt % 3), p.v, p.ldk, seq0 + kt * AT, seq0 + p.S, g * HD);
    }
    cp_async_commit();
  };
  auto Qs = stage_k(2);                                      // 128 rows
  tile_async<FQ, FWD_THREADS>(Qs, p.q, p.ldq, seq0 + q0, seq0 + p.S, h * HD);
  cp_async_commit();
  load_kv(0);
  load_kv(1);
  cp_async_wait<2>();                                        // the query tile has landed
  __syncthreads();
  uint32_t qf[HD / 16][4];
#pragma unroll
  for (int kk = 0; kk < HD / 16; ++kk) load_a(qf[kk], Qs, 16 * warp, kk, lane);
  const int r_first = q0 + 16 * warp;                        // this warp's first query
  const int qi0 = r_first + (lane >> 2), qi1 = qi0 + 8;      // this lane's two query rows
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  float o[8][4];
#pragma unroll
  for (int n = 0; n < 8; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }

  for (int kt = 0; kt < n_kt; ++kt) {
    const int k0 = kt * AT;
    cp_async_wait<1>();                                      // tile kt has landed (tile kt + 1 may be in flight)
    __syncthreads();                                         // ... for every thread; stage (kt + 2) % 3 is free
    load_kv(kt + 2);
    if (k0 > r_first + 15) continue;                         // wholly masked for this warp
    const __nv_bfloat16(*Ks)[LDS] = stage_k(kt % 3);
    const __nv_bfloat16(*Vs)[LDS] = stage_v(kt % 3);
    float s[8][4];
    scores_16x64(s, qf, Ks, lane);
    if (k0 + AT - 1 > r_first || k0 + AT > p.S) {            // the tile crosses the diagonal or the sequence end
#pragma unroll
      for (int n = 0; n < 8; ++n) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int kj = k0 + 8 * n + 2 * (lane & 3) + j;
          if (!(kj <= qi0 && kj < p.S)) s[n][j] = -INFINITY;
          if (!(kj <= qi1 && kj < p.S)) s[n][2 + j] = -INFINITY;
        }
      }
    }
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      mx0 = fmaxf(mx0, fmaxf(s[n][0], s[n][1]));
      mx1 = fmaxf(mx1, fmaxf(s[n][2], s[n][3]));
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    // running maxima in log2 units (the raw scores times scale_log2, a positive factor)
    const float mn0 = fmaxf(m0, mx0 * p.scale_log2), mn1 = fmaxf(m1, mx1 * p.scale_log2);
    // a row that has seen no key yet keeps maximum -inf: use 0 as the reference so that nothing is NaN
    const float ref0 = mn0 == -INFINITY ? 0.f : mn0, ref1 = mn1 == -INFINITY ? 0.f : mn1;
    const float a0 = exp2f(m0 - ref0), a1 = exp2f(m1 - ref1);            // exp2f(-inf) = 0
    float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      s[n][0] = exp2f(fmaf(s[n][0], p.scale_log2, -ref0)); s[n][1] = exp2f(fmaf(s[n][1], p.scale_log2, -ref0));
      s[n][2] = exp2f(fmaf(s[n][2], p.scale_log2, -ref1)); s[n][3] = exp2f(fmaf(s[n][3], p.scale_log2, -ref1));
      sum0 += s[n][0] + s[n][1];
      sum1 += s[n][2] + s[n][3];
      o[n][0] *= a0; o[n][1] *= a0; o[n][2] *= a1; o[n][3] *= a1;
    }
    sum0 += __shfl_xor_sync(0xffffffffu, sum0, 1); sum0 += __shfl_xor_sync(0xffffffffu, sum0, 2);
    sum1 += __shfl_xor_sync(0xffffffffu, sum1, 1); sum1 += __shfl_xor_sync(0xffffffffu, sum1, 2);
    l0 = l0 * a0 + sum0; l1 = l1 * a1 + sum1;
    m0 = mn0; m1 = mn1;
    uint32_t pf[4][4];
    to_a_frags(pf, s);
    accumulate_16x64(o, pf, Vs, lane);
  }
  cp_async_wait<0>();
  const float i0 = l0 > 0.f ? 1.0f / l0 : 0.f, i1 = l1 > 0.f ? 1.0f / l1 : 0.f;
  store_16x64(p.out, p.ldo, seq0 + r_first, seq0 + p.S, h * HD, o, i0, i1, lane);
  if ((lane & 3) == 0) {
    float* lse = p.lse + ((long long)b * p.H + h) * p.S;
    if (qi0 < p.S) lse[qi0] = m0 + log2f(l0);
    if (qi1 < p.S) lse[qi1] = m1 + log2f(l1);
  }
}

// ---- backward, head_dim 64, dQ: grid (query tiles, H, B); warp w owns queries 16 w .. 16 w + 15 ------------------
// Same ring as the forward kernel: the query and dO tiles sit in the third stage until their fragments are in
// registers.  Only the last key tile crosses the diagonal.  Keys beyond the sequence end need no mask of
// their own: their K rows are zero, so whatever dS they get adds nothing to dQ.
constexpr int BWD_THREADS = 128;
constexpr int BWD64_SMEM = 3 * STAGE_ELEMS * 2 + 3 * 2 * AT * 4;      // three stages + their lse / dsum rows (dK, dV kernel)
__global__ void __launch_bounds__(BWD_THREADS, 3)
attn_dq64_kernel(const AttnParams p) {
  extern __shared__ __align__(128) uint8_t att_smem[];
  auto stage_k = [&](int s) { return reinterpret_cast<__nv_bfloat16(*)[LDS]>(att_smem) + (size_t)s * 2 * AT; };
  auto stage_v = [&](int s) { return stage_k(s) + AT; };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;
  const int h = blockIdx.y, b = blockIdx.z;
  const int g = h / (p.H / p.Hkv);
  const long long seq0 = (long long)b * p.S;
  const int q0 = qt * AT;
  const int n_kt = qt + 1;
  auto load_kv = [&](int kt) {
    if (kt < n_kt) {
      tile_async<AT, BWD_THREADS>(stage_k(kt % 3), p.k, p.ldk, seq0 + kt * AT, seq0 + p.S, g * HD);
      tile_async<AT, BWD_THREADS>(stage_v(kt % 3), p.v, p.ldk, seq0 + kt * AT, seq0 + p.S, g * HD);
    }
    cp_async_commit();
  };
  tile_async<AT, BWD_THREADS>(stage_k(2), p.q, p.ldq, seq0 + q0, seq0 + p.S, h * HD);
  tile_async<AT, BWD_THREADS>(stage_v(2), p.dout, p.ldo, seq0 + q0, seq0 + p.S, h * HD);
  cp_async_commit();
  load_kv(0);
  load_kv(1);
  cp_async_wait<2>();
  __syncthreads();
  uint32_t qf[HD / 16][4], df[HD / 16][4];
#pragma unroll
  for (int kk = 0; kk < HD / 16; ++kk) { load_a(qf[kk], stage_k(2), 16 * warp, kk, lane); load_a(df[kk], stage_v(2), 16 * warp, kk, lane); }
  const int qi0 = q0 + 16 * warp + (lane >> 2), qi1 = qi0 + 8;
  const long long ro = ((long long)b * p.H + h) * p.S;
  const float lse0 = qi0 < p.S ? p.lse[ro + qi0] : 0.f, lse1 = qi1 < p.S ? p.lse[ro + qi1] : 0.f;
  const float inv_sqrt_d = p.scale_log2 / LOG2E;
  // dS = P (dP - dsum) / sqrt(d): the subtrahend and the factor are folded into one FMA per element
  const float nd0 = qi0 < p.S ? -p.dsum[ro + qi0] * inv_sqrt_d : 0.f, nd1 = qi1 < p.S ? -p.dsum[ro + qi1] * inv_sqrt_d : 0.f;
  float dq[8][4];
#pragma unroll
  for (int n = 0; n < 8; ++n) { dq[n][0] = dq[n][1] = dq[n][2] = dq[n][3] = 0.f; }

  for (int kt = 0; kt < n_kt; ++kt) {
    const int k0 = kt * AT;
    cp_async_wait<1>();
    __syncthreads();
    load_kv(kt + 2);
    const __nv_bfloat16(*Ks)[LDS] = stage_k(kt % 3);
    const __nv_bfloat16(*Vs)[LDS] = stage_v(kt % 3);
    float s[8][4], dp[8][4];
    scores_16x64(s, qf, Ks, lane);
    scores_16x64(dp, df, Vs, lane);
    const bool diag = kt == qt;
#pragma unroll
    for (int n = 0; n < 8; ++n) {
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int kj = k0 + 8 * n + 2 * (lane & 3) + j;
        float p0 = exp2f(fmaf(s[n][j], p.scale_log2, -lse0));
        float p1 = exp2f(fmaf(s[n][2 + j], p.scale_log2, -lse1));
        if (diag) { if (kj > qi0) p0 = 0.f; if (kj > qi1) p1 = 0.f; }
        s[n][j] = p0 * fmaf(dp[n][j], inv_sqrt_d, nd0);             // dS
        s[n][2 + j] = p1 * fmaf(dp[n][2 + j], inv_sqrt_d, nd1);
      }
    }
    uint32_t sf[4][4];
    to_a_frags(sf, s);
    accumulate_16x64(dq, sf, Ks, lane);                             // dQ += dS K
  }
  cp_async_wait<0>();
  store_16x64(p.dq, p.ldq, seq0 + q0 + 16 * warp, seq0 + p.S, h * HD, dq, 1.f, 1.f, lane);
}

// ---- backward, head_dim 64, dK and dV: grid (key tiles, Hkv, B); warp w owns keys 16 w .. 16 w + 15 ---------------
// The products are formed transposed (keys on the accumulator rows): S^T = K Q^T, dP^T = V dO^T; then
// dV += P^T dO and dK += dS^T Q contract over the 64 queries of a tile.  The (head, query tile) pairs that see
// this key tile form one sequence that runs through the ring (a Q tile, a dO tile and the 64 lse / dsum values per
// stage).  Only the first query tile of a head crosses the diagonal.  Queries beyond the sequence end need no
// mask: their Q and dO rows are zero, so whatever P and dS they get adds nothing to dV or dK.
__global__ void __launch_bounds__(BWD_THREADS, 2)
attn_dkv64_kernel(const AttnParams p) {
  extern __shared__ __align__(128) uint8_t att_smem[];
  auto stage_q = [&](int s) { return reinterpret_cast<__nv_bfloat16(*)[LDS]>(att_smem) + (size_t)s * 2 * AT; };
  auto stage_d = [&](int s) { return stage_q(s) + AT; };
  float* rows_all = reinterpret_cast<float*>(att_smem + 3 * STAGE_ELEMS * 2);        // [3][2][AT]: lse, dsum
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kt = blockIdx.x;                               // the first key tiles see the most queries: they start first
  const int g = blockIdx.y, b = blockIdx.z;
  const int rep = p.H / p.Hkv;
  const long long seq0 = (long long)b * p.S;
  const int k0 = kt * AT;
  const int n_qt = (p.S + AT - 1) / AT;
  const int per_head = n_qt - kt;
  const int n_it = rep * per_head;
  auto load_qd = [&](int it) {
    if (it < n_it) {
      const int h = g * rep + it / per_head, q0 = (kt + it % per_head) * AT;
      tile_async<AT, BWD_THREADS>(stage_q(it % 3), p.q, p.ldq, seq0 + q0, seq0 + p.S, h * HD);
      tile_async<AT, BWD_THREADS>(stage_d(it % 3), p.dout, p.ldo, seq0 + q0, seq0 + p.S, h * HD);
      const long long ro = ((long long)b * p.H + h) * p.S;
      const int c = threadIdx.x & (AT - 1);
      const float* src = threadIdx.x < AT ? p.lse : p.dsum;
      const bool valid = q0 + c < p.S;
      const uint32_t d = (uint32_t)__cvta_generic_to_shared(rows_all + (it % 3) * 2 * AT + threadIdx.x);
      const int nb = valid ? 4 : 0;
      asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(d), "l"(src + ro + (valid ? q0 + c : 0)), "r"(nb) : "memory");
    }
    cp_async_commit();
  };
  tile_async<AT, BWD_THREADS>(stage_q(2), p.k, p.ldk, seq0 + k0, seq0 + p.S, g * HD);
  tile_async<AT, BWD_THREADS>(stage_d(2), p.v, p.ldk, seq0 + k0, seq0 + p.S, g * HD);
  cp_async_commit();
  load_qd(0);
  load_qd(1);
  cp_async_wait<2>();
  __syncthreads();
  uint32_t kf[HD / 16][4], vf[HD / 16][4];
#pragma unroll
  for (int kk = 0; kk < HD / 16; ++kk) { load_a(kf[kk], stage_q(2), 16 * warp, kk, lane); load_a(vf[kk], stage_d(2), 16 * warp, kk, lane); }
  const int kj0 = k0 + 16 * warp + (lane >> 2), kj1 = kj0 + 8;          // this lane's two key rows
  const float inv_sqrt_d = p.scale_log2 / LOG2E;
  float dk[8][4], dv[8][4];
#pragma unroll
  for (int n = 0; n < 8; ++n) { dk[n][0] = dk[n][1] = dk[n][2] = dk[n][3] = 0.f; dv[n][0] = dv[n][1] = dv[n][2] = dv[n][3] = 0.f; }

  for (int it = 0; it < n_it; ++it) {
    cp_async_wait<1>();
    __syncthreads();
    load_qd(it + 2);
    const __nv_bfloat16(*Qs)[LDS] = stage_q(it % 3);
    const __nv_bfloat16(*Ds)[LDS] = stage_d(it % 3);
    const float* rowv = rows_all + (it % 3) * 2 * AT;
    const int q0 = (kt + it % per_head) * AT;
    const bool diag = it % per_head == 0;
    float st[8][4], dpt[8][4];
    scores_16x64(st, kf, Qs, lane);                               // S^T[key][query]
    scores_16x64(dpt, vf, Ds, lane);                              // dP^T[key][query]
    uint32_t pf[4][4];
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      const int c = 8 * n + 2 * (lane & 3);
      const float2 lse2 = *reinterpret_cast<const float2*>(rowv + c), dsm2 = *reinterpret_cast<const float2*>(rowv + AT + c);
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int qi = q0 + c + j;
        const float lse = j ? lse2.y : lse2.x, nd = -(j ? dsm2.y : dsm2.x) * inv_sqrt_d;
        float p0 = exp2f(fmaf(st[n][j], p.scale_log2, -lse));
        float p1 = exp2f(fmaf(st[n][2 + j], p.scale_log2, -lse));
        if (diag) { if (kj0 > qi) p0 = 0.f; if (kj1 > qi) p1 = 0.f; }
        st[n][j] = p0; st[n][2 + j] = p1;
        dpt[n][j] = p0 * fmaf(dpt[n][j], inv_sqrt_d, nd);          // dS^T
        dpt[n][2 + j] = p1 * fmaf(dpt[n][2 + j], inv_sqrt_d, nd);
      }
    }
    to_a_frags(pf, st);
    accumulate_16x64(dv, pf, Ds, lane);                           // dV += P^T dO
    to_a_frags(pf, dpt);
    accumulate_16x64(dk, pf, Qs, lane);                           // dK += dS^T Q
  }
  cp_async_wait<0>();
  store_16x64(p.dv, p.ldk, seq0 + k0 + 16 * warp, seq0 + p.S, g * HD, dv, 1.f, 1.f, lane);
  store_16x64(p.dk, p.ldk, seq0 + k0 + 16 * warp, seq0 + p.S, g * HD, dk, 1.f, 1.f, lane);
}

template <int D> constexpr int fwd_smem() { return 3 * AT * (D + 8) * 2 + 4 * 16 * (AT + 4) * 4 + 4 * 16 * (AT + 8) * 2; }
template <int D> constexpr int dkv_smem() { return 4 * AT * (D + 8) * 2 + 2 * 4 * AT * 20 * 4 + 4 * AT * 24 * 2 + 2 * AT * 4; }
template <int D> constexpr int dq_smem() { return 4 * AT * (D + 8) * 2 + 2 * 4 * 16 * (AT + 4) * 4 + 4 * 16 * (AT + 8) * 2; }

template <int D>
int launch_fwd(faar_ctx* ctx, const AttnParams& p) {
  cudaError_t e = cudaFuncSetAttribute(attn_fwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, fwd_smem<D>());
  if (e != cudaSuccess) return (int)e;
  dim3 grid((p.S + AT - 1) / AT, p.H, p.B);
  if (D == HD && ctx->tune_attention_fragments != 1) {
    e = cudaFuncSetAttribute(attn_fwd64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FWD64_SMEM);
    if (e != cudaSuccess) return (int)e;
  }
  faar_prof_scope ps(ctx, FAAR_K_ATTENTION);
  if (D == HD && ctx->tune_attention_fragments == 0)
    return faar_launch_attention_fwd64_tc(ctx, p.B, p.S, p.H, p.Hkv, p.q, p.ldq, p.k, p.v, p.ldk, p.out, p.ldo, p.lse,
                                          p.scale_log2);
  if (D == HD && ctx->tune_attention_fragments == 2)
    attn_fwd64_kernel<<<dim3((p.S + FQ - 1) / FQ, p.H, p.B), FWD_THREADS, FWD64_SMEM, ctx->stream>>>(p);
  else
    attn_fwd_kernel<D><<<grid, ATT_THREADS, fwd_smem<D>(), ctx->stream>>>(p);
  return (int)cudaGetLastError();
}

template <int D>
int launch_bwd(faar_ctx* ctx, const AttnParams& p, float* dsum) {
  cudaError_t e = cudaFuncSetAttribute(attn_dkv_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, dkv_smem<D>());
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_dq_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, dq_smem<D>());
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_dkv64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, BWD64_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_dq64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, BWD64_SMEM);
  if (e != cudaSuccess) return (int)e;
  faar_prof_scope ps(ctx, FAAR_K_ATTENTION);
  long long rows = (long long)p.B * p.H * ((p.S + 256 / D - 1) / (256 / D));      // warp passes of the row-sum kernel
  long long blocks = (rows + 3) / 4;
  if (blocks > (long long)ctx->num_sms * 16) blocks = (long long)ctx->num_sms * 16;
  attn_dsum_kernel<D><<<(int)blocks, ATT_THREADS, 0, ctx->stream>>>(p, dsum);
  const int tiles = (p.S + AT - 1) / AT;
  if (D == HD && ctx->tune_attention_fragments == 0) {
    int le = faar_launch_attention_dkv64_tc(ctx, p.B, p.S, p.H, p.Hkv, p.q, p.ldq, p.k, p.v, p.ldk, p.dout, p.ldo, p.lse, dsum,
                                            p.dk, p.dv, p.scale_log2);
    if (le) return le;
    return faar_launch_attention_dq64_tc(ctx, p.B, p.S, p.H, p.Hkv, p.q, p.ldq, p.k, p.v, p.ldk, p.dout, p.ldo, p.lse, dsum,
                                         p.dq, p.scale_log2);
  }
  if (D == HD && ctx->tune_attention_fragments != 1) {
    attn_dkv64_kernel<<<dim3(tiles, p.Hkv, p.B), BWD_THREADS, BWD64_SMEM, ctx->stream>>>(p);
    attn_dq64_kernel<<<dim3(tiles, p.H, p.B), BWD_THREADS, BWD64_SMEM, ctx->stream>>>(p);
    return (int)cudaGetLastError();
  }
  attn_dkv_kernel<D><<<dim3(tiles, p.Hkv, p.B), ATT_THREADS, dkv_smem<D>(), ctx->stream>>>(p);
  attn_dq_kernel<D><<<dim3(tiles, p.H, p.B), ATT_THREADS, dq_smem<D>(), ctx->stream>>>(p);
  return (int)cudaGetLastError();
}

}  // namespace

int faar_launch_attention_fwd(faar_ctx* ctx, int B, int S, int H, int Hkv, int D, const void* q, int64_t ldq, const void* k,
                              const void* v, int64_t ldk, void* out, int64_t ldo, float* lse) {
  AttnParams p = {};
  p.q = reinterpret_cast<const __nv_bfloat16*>(q); p.k = reinterpret_cast<const __nv_bfloat16*>(k);
  p.v = reinterpret_cast<const __nv_bfloat16*>(v); p.out = reinterpret_cast<__nv_bfloat16*>(out); p.lse = lse;
  p.ldq = ldq; p.ldk = ldk; p.ldo = ldo; p.B = B; p.S = S; p.H = H; p.Hkv = Hkv;
  p.scale_log2 = LOG2E / sqrtf((float)D);
  return D == 64 ? launch_fwd<64>(ctx, p) : launch_fwd<128>(ctx, p);
}

int faar_launch_attention_bwd(faar_ctx* ctx, int B, int S, int H, int Hkv, int D, const void* q, int64_t ldq, const void* k,
                              const void* v, int64_t ldk, const void* out, const void* dout, int64_t ldo, const float* lse,
                              float* dsum, void* dq, void* dk, void* dv) {
  AttnParams p = {};
  p.q = reinterpret_cast<const __nv_bfloat16*>(q); p.k = reinterpret_cast<const __nv_bfloat16*>(k);
  p.v = reinterpret_cast<const __nv_bfloat16*>(v);
  p.out = reinterpret_cast<__nv_bfloat16*>(const_cast<void*>(out)); p.lse = const_cast<float*>(lse);
  p.dout = reinterpret_cast<const __nv_bfloat16*>(dout); p.dsum = dsum;
  p.dq = reinterpret_cast<__nv_bfloat16*>(dq); p.dk = reinterpret_cast<__nv_bfloat16*>(dk); p.dv = reinterpret_cast<__nv_bfloat16*>(dv);
  p.ldq = ldq; p.ldk = ldk; p.ldo = ldo; p.B = B; p.S = S; p.H = H; p.Hkv = Hkv;
  p.scale_log2 = LOG2E / sqrtf((float)D);
  return D == 64 ? launch_bwd<64>(ctx, p, dsum) : launch_bwd<128>(ctx, p, dsum);
}
