// Full-model alignment loss (Eq. 6, Procedure steps 18-20): KL of the temperature softmaxes of the two
// models' logits, the squared error of their last hidden states, and both gradients towards the
// quantised model's outputs.
//
// Softmax needs a row's maximum and sum before any probability, and a token's two logit rows (2 x vocab
// BF16, 0.5 MB at a 128 K vocabulary) do not fit one SM's shared memory.  One persistent CTA per SM takes
// a token at a time and reads its rows twice: the first pass (from HBM) keeps a running maximum and sum
// of exponentials per thread, the second (the same 0.5 MB again, which L2 still holds: one row pair per
// SM is 76 MB over the chip) forms P_fp, P_q, the KL terms and the gradient.  HBM sees each logit once and
// the gradient once; the four exponentials per vocabulary entry cost about as much time on the
// special-function units as the traffic does on HBM, and both passes mix the two.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "faar.h"
#include "faar_internal.cuh"

namespace {

constexpr int AL_THREADS = 1024;
constexpr int AL_WARPS = AL_THREADS / 32;

struct AlignParams {
  const __nv_bfloat16* Zfp; const __nv_bfloat16* Zq; long long ldz; int V;
  const __nv_bfloat16* Hfp; const __nv_bfloat16* Hq; long long ldh; int D;
  __nv_bfloat16* dZ; __nv_bfloat16* dH;
  float c;                 // log2(e) / tau: softmax(z / tau) in base 2
  float gscale;            // lambda_kl / (tau T)
  float* kl_partials;      // one per CTA
  float* mse_partials;     // one per CTA
  int T;                   // tokens; CTA k takes tokens k, k + gridDim.x, ...
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
__device__ __forceinline__ uint64_t l2_stream_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_keep_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint4 ldg128_policy(const uint4* ptr, uint64_t pol) {
  uint4 v;
  asm volatile("ld.global.L2::cache_hint.v4.b32 {%0,%1,%2,%3}, [%4], %5;" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(ptr), "l"(pol));
  return v;
}
// the gradient is written once and not read here: it should not push the rows out of L2
__device__ __forceinline__ void stg128_policy(void* ptr, uint4 v, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1,%2,%3,%4}, %5;" ::"l"(ptr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w),
               "l"(pol)
               : "memory");
}

// (maximum m, sum s of 2^(y - m)) of two disjoint sets merged; an empty set is (-inf, 0)
__device__ __forceinline__ void merge(float& m, float& s, float m2, float s2) {
  const float M = fmaxf(m, m2);
  if (M == -INFINITY) { m = M; s = 0.f; return; }
  s = s * ex2f(m - M) + s2 * ex2f(m2 - M);
  m = M;
}

__device__ __forceinline__ void unpack8(const uint4& raw, float (&y)[8]) {      // eight BF16 -> FP32
  const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    y[2 * i] = __uint_as_float(r[i] << 16);
    y[2 * i + 1] = __uint_as_float(r[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t w) { return *reinterpret_cast<__nv_bfloat162*>(&w); }
// elements n..7 of a group of eight BF16 replaced by -1e30 (BF16 0xF149)
__device__ __forceinline__ uint4 mask_tail(uint4 v, int n) {
  uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (2 * i >= n) w[i] = 0xF149F149u;
    else if (2 * i + 1 >= n) w[i] = (w[i] & 0xFFFFu) | 0xF1490000u;
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}

__global__ void __launch_bounds__(AL_THREADS, 1)
align_loss_kernel(const AlignParams p) {
  __shared__ float wred[4][AL_WARPS];
  __shared__ float row[2];                                         // log2-sum-exp of the token's row: fp, q
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int ngroups = (p.V + 7) / 8;                               // 16-byte groups of a row (rows are padded: ldz >= ceil8(V))
  const int tail = p.V & 7;                                        // valid columns of a partial last group, 0 = none
  const uint64_t stream = l2_stream_policy(), keep = l2_keep_policy();   // first pass: keep the rows in L2; second: done with them
  float kl = 0.f, mse = 0.f;                                       // this thread's share over all of the CTA's tokens
  for (int t = blockIdx.x; t < p.T; t += gridDim.x) {
    const uint4* gf = reinterpret_cast<const uint4*>(p.Zfp + (long long)t * p.ldz);
    const uint4* gq = reinterpret_cast<const uint4*>(p.Zq + (long long)t * p.ldz);

    // ---- pass 1 (from HBM): running maximum and sum of 2^(c z - max) per thread.  Columns beyond the
    // vocabulary in the last group count as -1e30 (their exponentials are 0).
    float mf = -INFINITY, sf = 0.f, mq = -INFINITY, sq = 0.f;
    auto online = [&](uint4 v, float& m, float& s) {
      const __nv_bfloat162 x = __hmax2(__hmax2(as_bf162(v.x), as_bf162(v.y)), __hmax2(as_bf162(v.z), as_bf162(v.w)));
      const float m8 = fmaxf(__low2float(x), __high2float(x)) * p.c;          // tau > 0: scaling keeps the order
      if (m8 > m) { s *= ex2f(m - m8); m = m8; }                                // 2^-inf = 0 on the first group
      float z[8];
      unpack8(v, z);
#pragma unroll
      for (int i = 0; i < 8; ++i) s += ex2f(fmaf(z[i], p.c, -m));
    };
    {
      int g = threadIdx.x;
      for (; g + AL_THREADS < ngroups; g += 2 * AL_THREADS) {      // two groups per tensor in flight; only the second can be the row's last
        const uint4 a0 = ldg128_policy(gf + g, keep), b0 = ldg128_policy(gq + g, keep);
        const uint4 a1 = ldg128_policy(gf + g + AL_THREADS, keep), b1 = ldg128_policy(gq + g + AL_THREADS, keep);
        online(a0, mf, sf);
        online(b0, mq, sq);
        if (tail && g + AL_THREADS == ngroups - 1) {
          online(mask_tail(a1, tail), mf, sf);
          online(mask_tail(b1, tail), mq, sq);
        } else {
          online(a1, mf, sf);
          online(b1, mq, sq);
        }
      }
      if (g < ngroups) {
        uint4 a = ldg128_policy(gf + g, keep), b = ldg128_policy(gq + g, keep);
        if (tail && g == ngroups - 1) { a = mask_tail(a, tail); b = mask_tail(b, tail); }
        online(a, mf, sf);
        online(b, mq, sq);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      merge(mf, sf, __shfl_xor_sync(0xffffffffu, mf, o), __shfl_xor_sync(0xffffffffu, sf, o));
      merge(mq, sq, __shfl_xor_sync(0xffffffffu, mq, o), __shfl_xor_sync(0xffffffffu, sq, o));
    }
    __syncthreads();                                               // the previous token's readers of wred / row are done
    if (lane == 0) { wred[0][warp] = mf; wred[1][warp] = sf; wred[2][warp] = mq; wred[3][warp] = sq; }
    __syncthreads();
    if (threadIdx.x == 0) {
      float a = wred[0][0], b = wred[1][0], c = wred[2][0], d = wred[3][0];
      for (int w = 1; w < AL_WARPS; ++w) { merge(a, b, wred[0][w], wred[1][w]); merge(c, d, wred[2][w], wred[3][w]); }
      row[0] = a + lg2f(b);
      row[1] = c + lg2f(d);
    }
    __syncthreads();
    const float lse_f = row[0], lse_q = row[1];

    // ---- pass 2 (the same rows again, now from L2: one row pair per SM is in flight, far less than L2 holds):
    // log2 P = c z - lse, so log2 P_fp - log2 P_q = c (z_fp - z_q) - (lse_fp - lse_q)
    const float dlse = lse_f - lse_q;
    __nv_bfloat16* const gd = p.dZ ? p.dZ + (long long)t * p.ldz : nullptr;
    for (int g = threadIdx.x; g < ngroups; g += AL_THREADS) {
      uint4 va = ldg128_policy(gf + g, stream), vb = ldg128_policy(gq + g, stream);
      const bool last_partial = tail && g == ngroups - 1;
      if (last_partial) { va = mask_tail(va, tail); vb = mask_tail(vb, tail); }
      float a[8], b[8], gr[8];
      unpack8(va, a);
      unpack8(vb, b);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float pf = ex2f(fmaf(a[i], p.c, -lse_f)), pq = ex2f(fmaf(b[i], p.c, -lse_q));
        kl = fmaf(pf, fmaf(a[i] - b[i], p.c, -dlse), kl);
        gr[i] = p.gscale * (pq - pf);
      }
      if (gd) {
        if (!last_partial) {
          stg128_policy(gd + 8 * g, make_uint4(pack2(gr[0], gr[1]), pack2(gr[2], gr[3]), pack2(gr[4], gr[5]), pack2(gr[6], gr[7])),
                        stream);
        } else {
          for (int i = 0; i < tail; ++i) gd[8 * g + i] = __float2bfloat16_rn(gr[i]);
        }
      }
    }

    // ---- last hidden states
    {
      const __nv_bfloat16* hf = p.Hfp + (long long)t * p.ldh;
      const __nv_bfloat16* hq = p.Hq + (long long)t * p.ldh;
      __nv_bfloat16* dh = p.dH ? p.dH + (long long)t * p.ldh : nullptr;
      for (int g = threadIdx.x; 8 * g < p.D; g += AL_THREADS) {
        const int nv = min(8, p.D - 8 * g);
        float a[8], b[8], d[8];
        unpack8(reinterpret_cast<const uint4*>(hf)[g], a);         // rows are padded to 8 columns (ldh >= ceil8(D))
        unpack8(reinterpret_cast<const uint4*>(hq)[g], b);
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
}

}  // namespace

int faar_launch_align_loss(faar_ctx* ctx, int T, int vocab, int hidden, const void* Z_fp, const void* Z_q, int64_t ldz,
                           const void* H_fp, const void* H_q, int64_t ldh, float tau, float lambda_kl, void* dZ_q,
                           void* dH_q, float* kl_partials, float* mse_partials, int* n_partials) {
  AlignParams p;
  p.Zfp = reinterpret_cast<const __nv_bfloat16*>(Z_fp); p.Zq = reinterpret_cast<const __nv_bfloat16*>(Z_q);
  p.ldz = ldz; p.V = vocab;
  p.Hfp = reinterpret_cast<const __nv_bfloat16*>(H_fp); p.Hq = reinterpret_cast<const __nv_bfloat16*>(H_q);
  p.ldh = ldh; p.D = hidden;
  p.dZ = reinterpret_cast<__nv_bfloat16*>(dZ_q); p.dH = reinterpret_cast<__nv_bfloat16*>(dH_q);
  p.c = (float)(1.4426950408889634 / (double)tau);
  p.gscale = (float)((double)lambda_kl / ((double)tau * (double)T));
  p.kl_partials = kl_partials; p.mse_partials = mse_partials;
  p.T = T;
  // one persistent CTA per SM, each looping over its tokens: one row pair per SM in flight keeps the second
  // pass inside L2
  const int grid = T < ctx->num_sms ? T : ctx->num_sms;
  *n_partials = grid;
  faar_prof_scope ps(ctx, FAAR_K_ALIGN_LOSS);
  align_loss_kernel<<<grid, AL_THREADS, 0, ctx->stream>>>(p);
  return (int)cudaGetLastError();
}
