// Full-model alignment loss (Eq. 6, Procedure steps 18-20): KL of the temperature softmaxes of the two
// models' logits, the squared error of their last hidden states, and both gradients towards the
// quantised model's outputs -- one pass over HBM.
//
// A token's two logit rows (2 x vocab BF16, 0.5 MB at a 128 K vocabulary) do not fit one SM's shared
// memory, and softmax needs the row's maximum and sum before any probability.  So a thread-block cluster
// takes the row: CTA j of the cluster loads columns [j chunk, (j+1) chunk) of both rows into its shared
// memory while it forms their running maximum and sum of exponentials, the CTAs exchange the four
// numbers through distributed shared memory, and every CTA then walks its own chunk again from shared
// memory to form P_fp, P_q, the KL terms and the gradient.  HBM sees each logit once and the gradient once.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "faar.h"
#include "faar_internal.cuh"

namespace {

constexpr int AL_THREADS = 256;
constexpr int AL_WARPS = AL_THREADS / 32;

struct AlignParams {
  const __nv_bfloat16* Zfp; const __nv_bfloat16* Zq; long long ldz; int V;
  const __nv_bfloat16* Hfp; const __nv_bfloat16* Hq; long long ldh; int D;
  __nv_bfloat16* dZ; __nv_bfloat16* dH;
  float c;                 // log2(e) / tau: softmax(z / tau) in base 2
  float gscale;            // lambda_kl / (tau T)
  float* kl_partials;      // one per CTA
  float* mse_partials;     // one per CTA
  int chunk;               // logit columns per CTA, a multiple of 8
  int dchunk;              // hidden columns per CTA, a multiple of 8
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2f(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_size() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// the float at the same shared-memory offset in CTA `peer` of the cluster
__device__ __forceinline__ float ld_peer(const float* local, uint32_t peer) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(local);
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(peer));
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(r) : "memory");
  return v;
}

// (maximum m, sum s of 2^(y - m)) of two disjoint sets merged; an empty set is (-inf, 0)
__device__ __forceinline__ void merge(float& m, float& s, float m2, float s2) {
  const float M = fmaxf(m, m2);
  if (M == -INFINITY) { m = M; s = 0.f; return; }
  s = s * ex2f(m - M) + s2 * ex2f(m2 - M);
  m = M;
}

__device__ __forceinline__ void unpack8(const uint4& raw, float (&y)[8], float c) {
  const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    y[2 * i] = __uint_as_float(r[i] << 16) * c;
    y[2 * i + 1] = __uint_as_float(r[i] & 0xFFFF0000u) * c;
  }
}

__device__ __forceinline__ void online8(const float (&y)[8], int n_valid, float& m, float& s) {
  float m8 = -INFINITY;
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (i < n_valid) m8 = fmaxf(m8, y[i]);
  if (m8 == -INFINITY) return;
  if (m8 > m) { s *= ex2f(m - m8); m = m8; }        // ex2f(-inf) = 0 on the first group
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (i < n_valid) s += ex2f(y[i] - m);
}

__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}

__global__ void __launch_bounds__(AL_THREADS)
align_loss_kernel(const AlignParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  uint4* const zf = reinterpret_cast<uint4*>(smem_raw);            // this CTA's chunk of the Z_fp row, raw BF16
  uint4* const zq = zf + p.chunk / 8;
  __shared__ float wred[4][AL_WARPS];
  __shared__ float stats[4];                                       // (m_fp, s_fp, m_q, s_q) of this CTA's chunk
  __shared__ float row[2];                                         // log2-sum-exp of the whole row: fp, q
  const uint32_t cs = cluster_size(), rank = cluster_rank();
  const int t = blockIdx.x / cs;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col0 = (int)rank * p.chunk;
  const int ncols = max(0, min(p.chunk, p.V - col0));              // valid logit columns of this CTA
  const int ngroups = (ncols + 7) / 8;
  const uint4* gf = reinterpret_cast<const uint4*>(p.Zfp + (long long)t * p.ldz + col0);
  const uint4* gq = reinterpret_cast<const uint4*>(p.Zq + (long long)t * p.ldz + col0);

  // ---- pass 1: HBM -> shared memory, running (max, sum) per thread
  float mf = -INFINITY, sf = 0.f, mq = -INFINITY, sq = 0.f;
  for (int g = threadIdx.x; g < ngroups; g += AL_THREADS) {
    const uint4 a = gf[g], b = gq[g];                              // rows are padded to 8 columns (ldz >= ceil8(V))
    zf[g] = a;
    zq[g] = b;
    const int nv = min(8, ncols - 8 * g);
    float y[8];
    unpack8(a, y, p.c);
    online8(y, nv, mf, sf);
    unpack8(b, y, p.c);
    online8(y, nv, mq, sq);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    merge(mf, sf, __shfl_xor_sync(0xffffffffu, mf, o), __shfl_xor_sync(0xffffffffu, sf, o));
    merge(mq, sq, __shfl_xor_sync(0xffffffffu, mq, o), __shfl_xor_sync(0xffffffffu, sq, o));
  }
  if (lane == 0) { wred[0][warp] = mf; wred[1][warp] = sf; wred[2][warp] = mq; wred[3][warp] = sq; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = wred[0][0], b = wred[1][0], c = wred[2][0], d = wred[3][0];
    for (int w = 1; w < AL_WARPS; ++w) { merge(a, b, wred[0][w], wred[1][w]); merge(c, d, wred[2][w], wred[3][w]); }
    stats[0] = a; stats[1] = b; stats[2] = c; stats[3] = d;
  }
  cluster_barrier();                                               // every CTA's stats are written
  if (threadIdx.x == 0) {
    float a = -INFINITY, b = 0.f, c = -INFINITY, d = 0.f;
    for (uint32_t r = 0; r < cs; ++r) {                            // the same order in every CTA
      merge(a, b, ld_peer(&stats[0], r), ld_peer(&stats[1], r));
      merge(c, d, ld_peer(&stats[2], r), ld_peer(&stats[3], r));
    }
    row[0] = a + lg2f(b);
    row[1] = c + lg2f(d);
  }
  __syncthreads();
  const float lse_f = row[0], lse_q = row[1];

  // ---- pass 2: probabilities, KL terms and the gradient from shared memory
  float kl = 0.f;
  __nv_bfloat16* const gd = p.dZ ? p.dZ + (long long)t * p.ldz + col0 : nullptr;
  for (int g = threadIdx.x; g < ngroups; g += AL_THREADS) {
    const int nv = min(8, ncols - 8 * g);
    float yf[8], yq[8], gr[8];
    unpack8(zf[g], yf, p.c);
    unpack8(zq[g], yq, p.c);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float lf = yf[i] - lse_f, lq = yq[i] - lse_q;          // log2 of the probabilities
      const float pf = ex2f(lf), pq = ex2f(lq);
      if (i < nv) kl = fmaf(pf, lf - lq, kl);
      gr[i] = p.gscale * (pq - pf);
    }
    if (gd) {
      if (nv == 8) {
        *reinterpret_cast<uint4*>(gd + 8 * g) = make_uint4(pack2(gr[0], gr[1]), pack2(gr[2], gr[3]), pack2(gr[4], gr[5]),
                                                            pack2(gr[6], gr[7]));
      } else {
        for (int i = 0; i < nv; ++i) gd[8 * g + i] = __float2bfloat16_rn(gr[i]);
      }
    }
  }

  // ---- last hidden states: this CTA's slice of the token's row
  float mse = 0.f;
  {
    const int d0 = (int)rank * p.dchunk;
    const int nd = max(0, min(p.dchunk, p.D - d0));
    const __nv_bfloat16* hf = p.Hfp + (long long)t * p.ldh + d0;
    const __nv_bfloat16* hq = p.Hq + (long long)t * p.ldh + d0;
    __nv_bfloat16* dh = p.dH ? p.dH + (long long)t * p.ldh + d0 : nullptr;
    for (int g = threadIdx.x; 8 * g < nd; g += AL_THREADS) {
      const int nv = min(8, nd - 8 * g);
      float a[8], b[8], d[8];
      unpack8(reinterpret_cast<const uint4*>(hf)[g], a, 1.0f);     // rows are padded to 8 columns (ldh >= ceil8(D))
      unpack8(reinterpret_cast<const uint4*>(hq)[g], b, 1.0f);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        d[i] = b[i] - a[i];
        if (i < nv) mse = fmaf(d[i], d[i], mse);
        d[i] *= 2.0f;
      }
      if (dh) {
        if (nv == 8) {
          *reinterpret_cast<uint4*>(dh + 8 * g) = make_uint4(pack2(d[0], d[1]), pack2(d[2], d[3]), pack2(d[4], d[5]),
                                                              pack2(d[6], d[7]));
        } else {
          for (int i = 0; i < nv; ++i) dh[8 * g + i] = __float2bfloat16_rn(d[i]);
        }
      }
    }
  }

  kl = faar_warp_sum(kl);
  mse = faar_warp_sum(mse);
  __syncthreads();                                                 // wred is reused
  if (lane == 0) { wred[0][warp] = kl; wred[1][warp] = mse; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = 0.f, b = 0.f;
    for (int w = 0; w < AL_WARPS; ++w) { a += wred[0][w]; b += wred[1][w]; }
    p.kl_partials[blockIdx.x] = a * 0.6931471805599453f;           // log2 -> natural log
    p.mse_partials[blockIdx.x] = b;
  }
  cluster_barrier();                                               // no CTA leaves while a peer may still read its stats
}

}  // namespace

// Cluster size for a vocabulary: the smallest power of two up to 8 whose per-CTA share of the two rows
// fits in 72 KB (three CTAs per SM, so that one CTA's loads overlap another's arithmetic), else the
// smallest that fits in 200 KB; 0 if none does.
int faar_align_cluster_size(int vocab, int* chunk_out) {
  int pick = 0;
  for (int pass = 0; pass < 2 && !pick; ++pass)
    for (int cs = 1; cs <= 8; cs *= 2) {
      const int chunk = ((vocab + cs - 1) / cs + 7) / 8 * 8;
      if ((size_t)chunk * 4 <= (pass == 0 ? 72u * 1024u : 200u * 1024u)) { pick = cs; *chunk_out = chunk; break; }
    }
  return pick;
}

int faar_launch_align_loss(faar_ctx* ctx, int T, int vocab, int hidden, const void* Z_fp, const void* Z_q, int64_t ldz,
                           const void* H_fp, const void* H_q, int64_t ldh, float tau, float lambda_kl, void* dZ_q,
                           void* dH_q, float* kl_partials, float* mse_partials, int* n_partials) {
  AlignParams p;
  int chunk = 0;
  const int cs = faar_align_cluster_size(vocab, &chunk);
  if (cs == 0) return (int)cudaErrorInvalidValue;
  p.Zfp = reinterpret_cast<const __nv_bfloat16*>(Z_fp); p.Zq = reinterpret_cast<const __nv_bfloat16*>(Z_q);
  p.ldz = ldz; p.V = vocab;
  p.Hfp = reinterpret_cast<const __nv_bfloat16*>(H_fp); p.Hq = reinterpret_cast<const __nv_bfloat16*>(H_q);
  p.ldh = ldh; p.D = hidden;
  p.dZ = reinterpret_cast<__nv_bfloat16*>(dZ_q); p.dH = reinterpret_cast<__nv_bfloat16*>(dH_q);
  p.c = (float)(1.4426950408889634 / (double)tau);
  p.gscale = (float)((double)lambda_kl / ((double)tau * (double)T));
  p.kl_partials = kl_partials; p.mse_partials = mse_partials;
  p.chunk = chunk;
  p.dchunk = ((hidden + cs - 1) / cs + 7) / 8 * 8;
  const size_t smem = (size_t)chunk * 4;
  cudaError_t ce = cudaFuncSetAttribute(align_loss_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (ce != cudaSuccess) return (int)ce;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3((unsigned)T * (unsigned)cs, 1, 1);
  cfg.blockDim = dim3(AL_THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = ctx->stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  *n_partials = T * cs;
  faar_prof_scope ps(ctx, FAAR_K_ALIGN_LOSS);
  ce = cudaLaunchKernelEx(&cfg, align_loss_kernel, p);
  if (ce != cudaSuccess) return (int)ce;
  return (int)cudaGetLastError();
}
