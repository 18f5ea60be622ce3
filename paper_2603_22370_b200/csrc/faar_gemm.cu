// Tensor-core kernels of the FAAR layer step for sm_100a.
//
// One persistent, warp-specialised kernel computes C[M,N] = A[M,Kc] * B[N,Kc]^T
// for BF16 operands that both have the contraction dimension contiguous:
//   warp 0      : TMA producer  (cp.async.bulk.tensor, 128-byte swizzle, 4-6 stage ring)
//   warp 1      : MMA issuer    (tcgen05.mma kind::f16, 128 x BN x 16, FP32 accumulators in TMEM)
//   warps 2..9  : epilogue      (tcgen05.ld, two accumulator buffers so the epilogue of one
//                                tile overlaps the main loop of the next)
// The three epilogues are the operations of the layer step:
//   REF : Y_fp = X W^T                                   (Procedure step 8)
//   FWD : r = Y_q - Y_ref, sum r^2, dY = 2c r -> dY^T     (steps 9-10, Eq. 5 first term)
//   BWD : G = dY^T X -> dV -> optimiser update + clip     (step 13, Eq. 5, with Eq. 2/3 chain rule)
// In all of them the accumulator row (TMEM lane) is the output feature o.
//
// Every wait on an mbarrier is bounded: after about two seconds the waiting
// thread records a code in the status word, raises a CTA-wide abort flag and
// every role leaves its loop; the CTA then frees its tensor memory and exits.
#include <cuda.h>

#include "faar_internal.cuh"

namespace {

constexpr int BM = 128;
constexpr int BK = 64;                 // 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int NUM_EPI_WARPS = 8;
constexpr int NUM_THREADS = 32 * (2 + NUM_EPI_WARPS);
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;

template <int BN> struct TileCfg {
  static constexpr int STAGES = BN == 256 ? 4 : 6;
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TMEM_COLS = 2 * BN;                     // two accumulator buffers
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// ---- PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(done) : "r"(bar), "r"(parity) : "memory");
  return done;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

struct AbortCtl {
  volatile int* flag;     // shared memory
  uint32_t* status;       // global status word
};

// Returns false if the wait was abandoned (time limit, or another thread raised the flag).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const AbortCtl& ac, uint32_t code) {
  unsigned long long t0 = global_ns();
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 0xFF) == 0) {
      if (*ac.flag) return false;
      if (global_ns() - t0 > WAIT_LIMIT_NS) {
        atomicCAS(ac.status, 0u, code);
        *ac.flag = 1;
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const AbortCtl& ac, uint32_t code) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, ac, code);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: rows of 64 bf16 (128 B) with 128-byte swizzle, contraction
// dimension contiguous; groups of 8 rows are 1024 B apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);        // start address
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                          // descriptor version for sm_100
  d |= (uint64_t)2 << 61;                          // 128-byte swizzle
  return d;
}
// Instruction descriptor: D = F32, A = B = BF16, both K-major, M = 128, N = BN.
template <int BN> __device__ __forceinline__ constexpr uint32_t make_idesc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

struct KParams {
  int M, N, Kc;
  uint32_t* status;
  // REF / FWD
  void* Yout; int yout_dtype; long long ldy;
  const void* Yref; int yref_dtype;
  __nv_bfloat16* dYt; long long ld_dyt;
  float mse2c;
  float* partials;
  // BWD
  float* V; const uint8_t* code; const uint8_t* scales; const float* s_global;
  float* adam_m; float* adam_u; float* dV;
  float beta, lam_over_n, lr, b1, b2, eps, inv_bc1, inv_bc2; int opt;
};

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}

// ---- epilogues: one call handles 16 accumulator columns of one row ---------------------------
// REF: write acc to Y[t, o].
__device__ __forceinline__ void epi_ref(const KParams& p, int o, int t0, const uint32_t (&acc)[16]) {
  if (o >= p.M) return;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    int t = t0 + j;
    if (t < p.N) {
      float a = __uint_as_float(acc[j]);
      if (p.yout_dtype == FAAR_BF16)
        reinterpret_cast<__nv_bfloat16*>(p.Yout)[(long long)t * p.ldy + o] = __float2bfloat16_rn(a);
      else
        reinterpret_cast<float*>(p.Yout)[(long long)t * p.ldy + o] = a;
    }
  }
}

// FWD: residual, sum of squares, dY^T.
__device__ __forceinline__ float epi_fwd(const KParams& p, int o, int t0, const uint32_t (&acc)[16]) {
  if (o >= p.M) return 0.f;
  float yr[16];
  if (p.yref_dtype == FAAR_BF16) {
    const __nv_bfloat16* y = reinterpret_cast<const __nv_bfloat16*>(p.Yref);
#pragma unroll
    for (int j = 0; j < 16; ++j) yr[j] = (t0 + j < p.N) ? __bfloat162float(y[(long long)(t0 + j) * p.ldy + o]) : 0.f;
  } else {
    const float* y = reinterpret_cast<const float*>(p.Yref);
#pragma unroll
    for (int j = 0; j < 16; ++j) yr[j] = (t0 + j < p.N) ? y[(long long)(t0 + j) * p.ldy + o] : 0.f;
  }
  float ss = 0.f;
  float dy[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    float a = __uint_as_float(acc[j]);
    float r = (t0 + j < p.N) ? a - yr[j] : 0.f;
    ss = fmaf(r, r, ss);
    dy[j] = p.mse2c * r;
  }
  __nv_bfloat16* drow = p.dYt + (long long)o * p.ld_dyt + t0;
  if (t0 + 16 <= p.N) {
    uint4* d4 = reinterpret_cast<uint4*>(drow);
    d4[0] = make_uint4(pack_bf16x2(dy[0], dy[1]), pack_bf16x2(dy[2], dy[3]), pack_bf16x2(dy[4], dy[5]), pack_bf16x2(dy[6], dy[7]));
    d4[1] = make_uint4(pack_bf16x2(dy[8], dy[9]), pack_bf16x2(dy[10], dy[11]), pack_bf16x2(dy[12], dy[13]), pack_bf16x2(dy[14], dy[15]));
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (t0 + j < p.N) drow[j] = __float2bfloat16_rn(dy[j]);
  }
  if (p.Yout) {
    __nv_bfloat16* yq = reinterpret_cast<__nv_bfloat16*>(p.Yout);
#pragma unroll
    for (int j = 0; j < 16; ++j)
      if (t0 + j < p.N) yq[(long long)(t0 + j) * p.ldy + o] = __float2bfloat16_rn(__uint_as_float(acc[j]));
  }
  return ss;
}

// BWD: acc = G[o, k0..k0+15] (one scale block).  Returns the Round Loss contribution of the
// pre-update v's.
__device__ __forceinline__ float epi_bwd(const KParams& p, int o, int k0, const uint32_t (&acc)[16], float s_global) {
  if (o >= p.M || k0 >= p.N) return 0.f;
  const long long e = (long long)o * p.N + k0;
  float v[16];
  {
    const float4* vp = reinterpret_cast<const float4*>(p.V + e);
#pragma unroll
    for (int q = 0; q < 4; ++q) { float4 t = vp[q]; v[4*q] = t.x; v[4*q+1] = t.y; v[4*q+2] = t.z; v[4*q+3] = t.w; }
  }
  const uint2 cw2 = *reinterpret_cast<const uint2*>(p.code + e / 2);
  const float s = __fmul_rn(faar_e4m3_to_float(p.scales[e / 16]), s_global);
  const float sb = s * p.beta;
  float g[16];
  float rl = 0.f;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    uint32_t nib = ((j < 8 ? cw2.x : cw2.y) >> (4 * (j & 7))) & 0xF;
    int k = nib & 7;
    float z = fmaf(p.beta, v[j], -0.5f * p.beta);
    float ex = __expf(-fabsf(z));
    float hs = __fdividef(1.0f, 1.0f + ex);
    float dh = ex * hs * hs;                        // h (1 - h)
    float chain = sb * faar_width(k) * dh;
    chain = (nib & 8) ? -chain : chain;
    g[j] = fmaf(__uint_as_float(acc[j]), chain, p.lam_over_n * fmaf(-8.f, v[j], 4.f));
    float t = fmaf(2.f, v[j], -1.f);
    rl += fmaf(-t, t, 1.f);
  }
  if (p.dV) {
    float4* dp = reinterpret_cast<float4*>(p.dV + e);
#pragma unroll
    for (int q = 0; q < 4; ++q) dp[q] = make_float4(g[4*q], g[4*q+1], g[4*q+2], g[4*q+3]);
  }
  float vn[16];
  if (p.opt == 1) {
    float4* mp = reinterpret_cast<float4*>(p.adam_m + e);
    float4* up = reinterpret_cast<float4*>(p.adam_u + e);
    float m[16], u[16];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float4 t = mp[q]; m[4*q] = t.x; m[4*q+1] = t.y; m[4*q+2] = t.z; m[4*q+3] = t.w;
      float4 w = up[q]; u[4*q] = w.x; u[4*q+1] = w.y; u[4*q+2] = w.z; u[4*q+3] = w.w;
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      m[j] = fmaf(p.b1, m[j], (1.f - p.b1) * g[j]);
      u[j] = fmaf(p.b2, u[j], (1.f - p.b2) * g[j] * g[j]);
      float mh = m[j] * p.inv_bc1;
      float uh = u[j] * p.inv_bc2;
      vn[j] = v[j] - p.lr * mh / (sqrtf(uh) + p.eps);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      mp[q] = make_float4(m[4*q], m[4*q+1], m[4*q+2], m[4*q+3]);
      up[q] = make_float4(u[4*q], u[4*q+1], u[4*q+2], u[4*q+3]);
    }
  } else {
#pragma unroll
    for (int j = 0; j < 16; ++j) vn[j] = fmaf(-p.lr, g[j], v[j]);
  }
  float4* vp = reinterpret_cast<float4*>(p.V + e);
#pragma unroll
  for (int q = 0; q < 4; ++q)
    vp[q] = make_float4(fminf(fmaxf(vn[4*q], 0.f), 1.f), fminf(fmaxf(vn[4*q+1], 0.f), 1.f),
                        fminf(fmaxf(vn[4*q+2], 0.f), 1.f), fminf(fmaxf(vn[4*q+3], 0.f), 1.f));
  return rl;
}

// ---- the kernel ------------------------------------------------------------------------------
template <int MODE, int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
faar_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const KParams p) {
  using Cfg = TileCfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  uint8_t* ctl = smem + Cfg::STAGES * Cfg::STAGE_BYTES;
  const uint32_t ctl_u32 = base + Cfg::STAGES * Cfg::STAGE_BYTES;
  // control block: full[S], empty[S], tmem_full[2], tmem_empty[2], tmem base, abort flag
  auto full_bar = [&](int s) { return ctl_u32 + 8u * s; };
  auto empty_bar = [&](int s) { return ctl_u32 + 8u * (Cfg::STAGES + s); };
  auto tfull_bar = [&](int a) { return ctl_u32 + 8u * (2 * Cfg::STAGES + a); };
  auto tempty_bar = [&](int a) { return ctl_u32 + 8u * (2 * Cfg::STAGES + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctl + 8 * (2 * Cfg::STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + 8 * (2 * Cfg::STAGES + 4) + 4);
  const AbortCtl ac{abort_flag, p.status};

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (p.M + BM - 1) / BM, n_tiles = (p.N + BN - 1) / BN;
  const int total_tiles = m_tiles * n_tiles;
  const int k_blocks = (p.Kc + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), NUM_EPI_WARPS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % m_tiles) * BM, n0 = (tile / m_tiles) * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, ac, 0x100u | stage);
          if (!ok) break;
          const uint32_t sa = base + stage * Cfg::STAGE_BYTES, sb = sa + Cfg::A_BYTES;
          mbar_expect_tx(full_bar(stage), Cfg::STAGE_BYTES);
          tma_load_2d(sa, &tmA, kb * BK, m0, full_bar(stage));
          tma_load_2d(sb, &tmB, kb * BK, n0, full_bar(stage));
          if (++stage == Cfg::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // give copies already in flight a bounded chance to land before the CTA exits
        for (int s = 0; s < Cfg::STAGES; ++s) {
          unsigned long long t0 = global_ns();
          const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
          while (!mbar_try_wait(full_bar(s), par) && global_ns() - t0 < 50000000ull) {}
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc<BN>();
      int stage = 0; uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1;
        ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, ac, 0x200u | acc);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          ok = mbar_wait(full_bar(stage), phase, ac, 0x300u | stage);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = base + stage * Cfg::STAGE_BYTES, sb = sa + Cfg::A_BYTES;
          const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sb);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing 16 bf16 = 32 bytes inside the swizzled row: +2 in the 16-byte address field
            tc_mma_bf16(tmem_d, da + 2u * k, db + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit(empty_bar(stage));
          if (++stage == Cfg::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(tfull_bar(acc));
      }
    }
  } else {
    // ---------------- epilogue ----------------
    const int ew = warp - 2;
    const int quarter = warp & 3;                    // TMEM lanes this warp may read
    const int col_begin = (ew >> 2) * (BN / 2);
    float warp_acc = 0.f;
    float s_global = 0.f;
    if (MODE == FAAR_GEMM_BWD) s_global = *p.s_global;
    int it = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1;
      bool ok = mbar_wait(tfull_bar(acc), acc_phase, ac, 0x400u | acc);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int m0 = (tile % m_tiles) * BM, n0 = (tile / m_tiles) * BN;
      const int o = m0 + quarter * 32 + lane;
      const uint32_t trow = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
#pragma unroll 1
      for (int c = col_begin; c < col_begin + BN / 2; c += 16) {
        if (n0 + c >= p.N) break;                    // warp-uniform
        uint32_t r[16];
        tmem_ld16(trow + (uint32_t)c, r);
        tmem_ld_wait();
        if (MODE == FAAR_GEMM_REF) epi_ref(p, o, n0 + c, r);
        else if (MODE == FAAR_GEMM_FWD) warp_acc += epi_fwd(p, o, n0 + c, r);
        else warp_acc += epi_bwd(p, o, n0 + c, r, s_global);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
    }
    if (MODE != FAAR_GEMM_REF) {
      warp_acc = faar_warp_sum(warp_acc);
      if (lane == 0) p.partials[blockIdx.x * NUM_EPI_WARPS + ew] = warp_acc;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
  }
}

// ---- host side ----------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// rows x cols bf16 matrix, cols contiguous, row stride ld elements; box = box_rows x 64.
int make_map(faar_ctx* ctx, CUtensorMap* map, const void* ptr, int rows, int cols, int64_t ld, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : (int)cudaErrorInvalidValue;
}

template <int MODE, int BN>
int launch(faar_ctx* ctx, const faar_gemm_args* a, const KParams& kp, int grid) {
  using Cfg = TileCfg<BN>;
  CUtensorMap tmA, tmB;
  int e = make_map(ctx, &tmA, a->A, a->M, a->Kc, a->lda, BM);
  if (e) return e;
  e = make_map(ctx, &tmB, a->B, a->N, a->Kc, a->ldb, BN);
  if (e) return e;
  auto kern = faar_gemm_kernel<MODE, BN>;
  cudaError_t ce = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
  if (ce != cudaSuccess) return (int)ce;
  faar_prof_scope ps(ctx, MODE == FAAR_GEMM_REF ? FAAR_K_GEMM_REF : (MODE == FAAR_GEMM_FWD ? FAAR_K_GEMM_FWD : FAAR_K_GEMM_BWD));
  kern<<<grid, NUM_THREADS, Cfg::SMEM_BYTES, ctx->stream>>>(tmA, tmB, kp);
  return (int)cudaGetLastError();
}

int pick_bn(const faar_ctx* ctx, int M, int N) {
  // the wide tile unless it leaves most SMs idle
  long long tiles256 = (long long)((M + BM - 1) / BM) * ((N + 255) / 256);
  return tiles256 >= ctx->num_sms ? 256 : 128;
}

}  // namespace

int faar_gemm_max_partials(const faar_ctx* ctx, int, int) { return ctx->num_sms * NUM_EPI_WARPS; }

int faar_launch_gemm(faar_ctx* ctx, const faar_gemm_args* a, int* n_partials_out) {
  KParams kp;
  kp.M = a->M; kp.N = a->N; kp.Kc = a->Kc; kp.status = a->status;
  kp.Yout = a->Yout; kp.yout_dtype = a->yout_dtype; kp.ldy = a->ldy;
  kp.Yref = a->Yref; kp.yref_dtype = a->yref_dtype;
  kp.dYt = a->dYt; kp.ld_dyt = a->ld_dyt; kp.mse2c = a->mse2c; kp.partials = a->partials;
  kp.V = a->V; kp.code = a->code; kp.scales = a->scales; kp.s_global = a->s_global;
  kp.adam_m = a->adam_m; kp.adam_u = a->adam_u; kp.dV = a->dV;
  kp.beta = a->beta; kp.lam_over_n = a->lam_over_n; kp.lr = a->lr; kp.b1 = a->b1; kp.b2 = a->b2; kp.eps = a->eps;
  kp.inv_bc1 = a->inv_bc1; kp.inv_bc2 = a->inv_bc2; kp.opt = a->opt;

  const int bn = pick_bn(ctx, a->M, a->N);
  const long long tiles = (long long)((a->M + BM - 1) / BM) * ((a->N + bn - 1) / bn);
  const int grid = (int)(tiles < ctx->num_sms ? tiles : ctx->num_sms);
  if (n_partials_out) *n_partials_out = grid * NUM_EPI_WARPS;
  switch (a->mode * 2 + (bn == 256 ? 1 : 0)) {
    case FAAR_GEMM_REF * 2 + 0: return launch<FAAR_GEMM_REF, 128>(ctx, a, kp, grid);
    case FAAR_GEMM_REF * 2 + 1: return launch<FAAR_GEMM_REF, 256>(ctx, a, kp, grid);
    case FAAR_GEMM_FWD * 2 + 0: return launch<FAAR_GEMM_FWD, 128>(ctx, a, kp, grid);
    case FAAR_GEMM_FWD * 2 + 1: return launch<FAAR_GEMM_FWD, 256>(ctx, a, kp, grid);
    case FAAR_GEMM_BWD * 2 + 0: return launch<FAAR_GEMM_BWD, 128>(ctx, a, kp, grid);
    case FAAR_GEMM_BWD * 2 + 1: return launch<FAAR_GEMM_BWD, 256>(ctx, a, kp, grid);
  }
  return (int)cudaErrorInvalidValue;
}
