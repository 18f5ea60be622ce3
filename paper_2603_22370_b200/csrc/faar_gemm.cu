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
constexpr int EPI_WARP_BYTES = 32 * 32 * 4;   // one 32 x 32 FP32 accumulator block per epilogue warp

template <int BN> struct TileCfg {
  static constexpr int STAGES = BN == 256 ? 4 : 6;
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TMEM_COLS = 2 * BN;                     // two accumulator buffers
  static constexpr int EPI_BYTES = NUM_EPI_WARPS * EPI_WARP_BYTES;   // BWD: per-warp transposition buffers
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
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
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ float4 lds128(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
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

// BWD.  A warp's 32 x 32 block of G (row = output feature o, column = input feature k) has been
// staged in shared memory, row r at stg + 128 r, its eight 16-byte units XOR-swizzled by (r & 7).
// Here lane (a, b) = (lane / 8, lane % 8) handles, in pass q, row 4q + a and columns 4b..4b+3, so
// that eight lanes cover 128 contiguous bytes of a row of V / m / u and every global access is a
// full line.  Returns the Round Loss contribution of the pre-update v's.
__device__ __forceinline__ float sqrt_approx(float x) {       // sqrt(0) = 0, about 1 ulp
  float y;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float width_of(uint32_t k) {       // interval widths .5 .5 .5 .5 1 1 2
  return __uint_as_float((126u + ((0x2500u >> (2u * k)) & 3u)) << 23);
}

template <int OPT>
__device__ __forceinline__ float epi_bwd_block(const KParams& p, uint32_t stg, int lane, int o_first, int k_first,
                                               float s_global) {
  const int a = lane >> 3, b = lane & 7;
  const int kcol = k_first + 4 * b;
  const bool col_ok = kcol < p.N;
  const float hb = -0.5f * p.beta;
  const float c1 = 1.f - p.b1, c2 = 1.f - p.b2;
  float rl = 0.f;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    float4 v[4], m[4], u[4];
    uint32_t cw[4], sb[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int o = o_first + 16 * half + 4 * q + a;
      if (col_ok && o < p.M) {
        const long long e = (long long)o * p.N + kcol;
        v[q] = *reinterpret_cast<const float4*>(p.V + e);
        cw[q] = *reinterpret_cast<const uint16_t*>(p.code + (e >> 1));
        sb[q] = p.scales[e >> 4];
        if (OPT == 1) {
          m[q] = *reinterpret_cast<const float4*>(p.adam_m + e);
          u[q] = *reinterpret_cast<const float4*>(p.adam_u + e);
        }
      }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int row = 16 * half + 4 * q + a;
      const int o = o_first + row;
      if (col_ok && o < p.M) {
        const long long e = (long long)o * p.N + kcol;
        const float4 g4 = lds128(stg + (uint32_t)row * 128u + (uint32_t)((b ^ (row & 7)) << 4));
        const float G[4] = {g4.x, g4.y, g4.z, g4.w};
        const float vv[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
        const float sbeta = __fmul_rn(faar_e4m3_to_float(sb[q]), s_global) * p.beta;
        float g[4], vn[4], mn[4], un[4];
        float mm[4], uu[4];
        if (OPT == 1) {
          mm[0] = m[q].x; mm[1] = m[q].y; mm[2] = m[q].z; mm[3] = m[q].w;
          uu[0] = u[q].x; uu[1] = u[q].y; uu[2] = u[q].z; uu[3] = u[q].w;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t nib = (cw[q] >> (4 * i)) & 0xFu;
          const float z = fmaf(p.beta, vv[i], hb);
          const float ex = __expf(-fabsf(z));
          const float hs = __fdividef(1.0f, 1.0f + ex);
          const float dh = ex * hs * hs;                                     // h (1 - h)
          float chain = sbeta * width_of(nib & 7u) * dh;
          chain = __uint_as_float(__float_as_uint(chain) ^ ((nib & 8u) << 28));   // sign of w
          g[i] = fmaf(G[i], chain, p.lam_over_n * fmaf(-8.f, vv[i], 4.f));
          const float t = fmaf(2.f, vv[i], -1.f);
          rl += fmaf(-t, t, 1.f);
          if (OPT == 1) {
            mn[i] = fmaf(p.b1, mm[i], c1 * g[i]);
            un[i] = fmaf(p.b2, uu[i], c2 * g[i] * g[i]);
            const float den = sqrt_approx(un[i] * p.inv_bc2) + p.eps;
            vn[i] = fmaf(-p.lr * p.inv_bc1, __fdividef(mn[i], den), vv[i]);
          } else {
            vn[i] = fmaf(-p.lr, g[i], vv[i]);
          }
          vn[i] = fminf(fmaxf(vn[i], 0.f), 1.f);
        }
        if (p.dV) *reinterpret_cast<float4*>(p.dV + e) = make_float4(g[0], g[1], g[2], g[3]);
        if (OPT == 1) {
          *reinterpret_cast<float4*>(p.adam_m + e) = make_float4(mn[0], mn[1], mn[2], mn[3]);
          *reinterpret_cast<float4*>(p.adam_u + e) = make_float4(un[0], un[1], un[2], un[3]);
        }
        *reinterpret_cast<float4*>(p.V + e) = make_float4(vn[0], vn[1], vn[2], vn[3]);
      }
    }
  }
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
  const uint32_t epi_u32 = base + Cfg::STAGES * Cfg::STAGE_BYTES;
  uint8_t* ctl = smem + Cfg::STAGES * Cfg::STAGE_BYTES + Cfg::EPI_BYTES;
  const uint32_t ctl_u32 = epi_u32 + Cfg::EPI_BYTES;
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
      if constexpr (MODE == FAAR_GEMM_BWD) {
        const uint32_t stg = epi_u32 + (uint32_t)ew * EPI_WARP_BYTES;
#pragma unroll 1
        for (int c = col_begin; c < col_begin + BN / 2; c += 32) {
          if (n0 + c >= p.N) break;                    // warp-uniform
          uint32_t r[32];
          tmem_ld32(trow + (uint32_t)c, r);
          tmem_ld_wait();
#pragma unroll
          for (int u = 0; u < 8; ++u)
            sts128(stg + (uint32_t)lane * 128u + (uint32_t)((u ^ (lane & 7)) << 4), r[4 * u], r[4 * u + 1], r[4 * u + 2],
                   r[4 * u + 3]);
          __syncwarp();
          warp_acc += p.opt == 1 ? epi_bwd_block<1>(p, stg, lane, m0 + quarter * 32, n0 + c, s_global)
                                 : epi_bwd_block<0>(p, stg, lane, m0 + quarter * 32, n0 + c, s_global);
          __syncwarp();                                // the block is consumed before the next one lands
        }
      } else {
#pragma unroll 1
        for (int c = col_begin; c < col_begin + BN / 2; c += 16) {
          if (n0 + c >= p.N) break;                    // warp-uniform
          uint32_t r[16];
          tmem_ld16(trow + (uint32_t)c, r);
          tmem_ld_wait();
          if (MODE == FAAR_GEMM_REF) epi_ref(p, o, n0 + c, r);
          else warp_acc += epi_fwd(p, o, n0 + c, r);
        }
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
