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

// ---- backward, step 0: dsum[b, h, t] = sum_d dO[t, h, d] * O[t, h, d]  (one warp per (token, head)) -------------
template <int D>
__global__ void __launch_bounds__(ATT_THREADS)
attn_dsum_kernel(const AttnParams p, float* dsum) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long total = (long long)p.B * p.S * p.H;
  for (long long i = (long long)blockIdx.x * (ATT_THREADS / 32) + warp; i < total; i += (long long)gridDim.x * (ATT_THREADS / 32)) {
    const int h = (int)(i % p.H);
    const long long t = i / p.H;                             // token index over all sequences
    const __nv_bfloat16* o = p.out + t * p.ldo + h * D;
    const __nv_bfloat16* d = p.dout + t * p.ldo + h * D;
    float acc = 0.f;
    for (int c = lane; c < D; c += 32) acc = fmaf(__bfloat162float(o[c]), __bfloat162float(d[c]), acc);
    acc = faar_warp_sum(acc);
    if (lane == 0) {
      const long long b = t / p.S, sidx = t - b * p.S;
      dsum[(b * p.H + h) * p.S + sidx] = acc;
    }
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

template <int D> constexpr int fwd_smem() { return 3 * AT * (D + 8) * 2 + 4 * 16 * (AT + 4) * 4 + 4 * 16 * (AT + 8) * 2; }
template <int D> constexpr int dkv_smem() { return 4 * AT * (D + 8) * 2 + 2 * 4 * AT * 20 * 4 + 4 * AT * 24 * 2 + 2 * AT * 4; }
template <int D> constexpr int dq_smem() { return 4 * AT * (D + 8) * 2 + 2 * 4 * 16 * (AT + 4) * 4 + 4 * 16 * (AT + 8) * 2; }

template <int D>
int launch_fwd(faar_ctx* ctx, const AttnParams& p) {
  cudaError_t e = cudaFuncSetAttribute(attn_fwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, fwd_smem<D>());
  if (e != cudaSuccess) return (int)e;
  dim3 grid((p.S + AT - 1) / AT, p.H, p.B);
  faar_prof_scope ps(ctx, FAAR_K_ATTENTION);
  attn_fwd_kernel<D><<<grid, ATT_THREADS, fwd_smem<D>(), ctx->stream>>>(p);
  return (int)cudaGetLastError();
}

template <int D>
int launch_bwd(faar_ctx* ctx, const AttnParams& p, float* dsum) {
  cudaError_t e = cudaFuncSetAttribute(attn_dkv_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, dkv_smem<D>());
  if (e == cudaSuccess) e = cudaFuncSetAttribute(attn_dq_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, dq_smem<D>());
  if (e != cudaSuccess) return (int)e;
  faar_prof_scope ps(ctx, FAAR_K_ATTENTION);
  long long rows = (long long)p.B * p.S * p.H;
  long long blocks = (rows + 3) / 4;
  if (blocks > (long long)ctx->num_sms * 16) blocks = (long long)ctx->num_sms * 16;
  attn_dsum_kernel<D><<<(int)blocks, ATT_THREADS, 0, ctx->stream>>>(p, dsum);
  const int tiles = (p.S + AT - 1) / AT;
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
