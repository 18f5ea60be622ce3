// NVFP4 x NVFP4 GEMM on the block-scaled tensor-core path of sm_100a: consumes what the library's own
// hardening (faar_harden_pack + faar_swizzle_scales) and activation quantiser (faar_act_fakequant +
// faar_swizzle_scales) produce -- packed E2M1 codes, E4M3 block scales in the 128 x 4 tiled order, FP32 tensor
// scales -- and returns C = alpha * A B^T in BF16 ("Hardening and Inference": the final weights are
// deployable on NVFP4 hardware as they are).
//
//   C[M,N] = (sA sB) * sum_k  A[m,k] B[n,k]        A: [M, K/2] bytes, B: [N, K/2] bytes, two codes per byte
//
// One CTA computes a 128 x 128 tile (tcgen05.mma kind::mxf4nvf4, block size 16, M = 128, N = 128, K = 64 per
// instruction; FP32 accumulators in tensor memory, two buffers so that a tile's epilogue overlaps the next
// tile's main loop).  A stage of the operand ring holds 256 elements of the contraction: 128 rows x 128
// bytes of A and of B (TMA, 128-byte swizzle: a row of 256 codes is exactly one swizzle row) plus their scale
// tiles, 4 x 512 bytes each, which are contiguous in the tiled layout and arrive by bulk copy.  The MMA
// thread moves a stage's scale tiles into tensor memory (tcgen05.cp, 32 lanes x 128 bits replicated to the
// four lane quarters: the layout the block-scaled MMA reads) and issues the four MMAs; tensor-core
// instructions of one thread execute in order, so the scale columns are reused by every stage.
//   warp 0: producer     warp 1: tensor memory + MMA issue     warps 2-5: epilogue (one lane quarter each)
// Every barrier wait is bounded (status word, orderly exit), as in the BF16 kernels.
#include <cuda.h>

#include "faar_internal.cuh"

namespace {

constexpr int TM = 128, TN = 128;            // output tile
constexpr int KS = 256;                      // contraction elements per stage = 128 bytes per row
constexpr int KI = 64;                       // contraction elements per MMA
constexpr int ROW_BYTES = KS / 2;            // 128
constexpr int A_BYTES = TM * ROW_BYTES;      // 16 KB
constexpr int B_BYTES = TN * ROW_BYTES;      // 16 KB
constexpr int SF_TILE = 512;                 // scales of 128 rows x 64 contraction elements
constexpr int SF_BYTES = (KS / KI) * SF_TILE;              // per operand and stage: 2 KB
constexpr int STAGE = A_BYTES + B_BYTES + 2 * SF_BYTES;    // 36 KB
constexpr int STAGES = 5;
constexpr int THREADS = 32 * 6;
constexpr int TMEM_COLS = 512;               // 2 x 128 accumulator columns + 16 + 16 scale columns
constexpr int COL_SFA = 2 * TN, COL_SFB = 2 * TN + 16;
constexpr int CTL = 256;
constexpr int SMEM = STAGES * STAGE + CTL + 1024;
constexpr unsigned long long LIMIT_NS = 2000000000ull;

struct P4 {
  int M, N, K;
  const uint8_t* sfa; const uint8_t* sfb;    // tiled scales: [row tile][k tile][512]
  int k_tiles;                               // 64-element tiles along the contraction (scale layout: padded)
  const float* sa; const float* sb;
  __nv_bfloat16* C; long long ldc;
  uint32_t* status;
};

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint32_t b, uint32_t n) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(b), "r"(n)); }
__device__ __forceinline__ void bar_arrive(uint32_t b) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(b) : "memory"); }
__device__ __forceinline__ void bar_expect(uint32_t b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t bar_try(uint32_t b, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(b), "r"(parity) : "memory");
  return ok;
}
__device__ __forceinline__ unsigned long long now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
struct Abort { volatile int* flag; uint32_t* status; };
__device__ __noinline__ bool bar_wait_slow(uint32_t b, uint32_t parity, const Abort& ab, uint32_t code) {
  const unsigned long long t0 = now_ns();
  for (uint32_t spin = 1;; ++spin) {
    if (bar_try(b, parity)) return true;
    if ((spin & 0xFF) == 0) {
      if (*ab.flag) return false;
      if (now_ns() - t0 > LIMIT_NS) { atomicCAS(ab.status, 0u, code); *ab.flag = 1; return false; }
    }
  }
}
__device__ __forceinline__ bool bar_wait(uint32_t b, uint32_t parity, const Abort& ab, uint32_t code) {
  return bar_try(b, parity) ? true : bar_wait_slow(b, parity, ab, code);
}
__device__ __forceinline__ void tma_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// plain bulk copy global -> shared; both addresses 16-byte aligned, size a multiple of 16
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Operand descriptor: rows of 128 bytes, 128-byte swizzle, contraction contiguous, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t desc_sw128(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// Scale-tile descriptor for tcgen05.cp: 32 rows of 16 bytes, no swizzle, 8-row groups 128 B apart.
__device__ __forceinline__ uint64_t desc_sf(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)(128 >> 4) << 32) | ((uint64_t)1 << 46);
}
// Instruction descriptor of kind::mxf4nvf4: A = B = E2M1 (code 1), both K-major, E4M3 scales, N >> 3, M >> 4, K = 64.
__device__ __forceinline__ uint32_t idesc_fp4() {
  return (1u << 7) | (1u << 10) | ((uint32_t)(TN >> 3) << 17) | (0u << 23) | ((uint32_t)(TM >> 4) << 24);
}
__device__ __forceinline__ void cp_sf(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void mma_fp4(uint32_t d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t sfa, uint32_t sfb,
                                        uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
      ::"r"(d), "l"(da), "l"(db), "r"(idesc), "r"(sfa), "r"(sfb), "r"(acc) : "memory");
}
__device__ __forceinline__ void ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__global__ void __launch_bounds__(THREADS, 1)
nvfp4_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const P4 p) {
  extern __shared__ uint8_t raw[];
  const uint32_t base = (s32(raw) + 1023u) & ~1023u;
  uint8_t* smem = raw + (base - s32(raw));
  const uint32_t ctl = base + STAGES * STAGE;
  uint8_t* ctl_p = smem + STAGES * STAGE;
  auto full = [&](int s) { return ctl + 8u * s; };
  auto empty = [&](int s) { return ctl + 8u * (STAGES + s); };
  auto tfull = [&](int a) { return ctl + 8u * (2 * STAGES + a); };
  auto tempty = [&](int a) { return ctl + 8u * (2 * STAGES + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctl_p + 8 * (2 * STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl_p + 8 * (2 * STAGES + 4) + 4);
  const Abort ab{abort_flag, p.status};
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const int m_tiles = (p.M + TM - 1) / TM, n_tiles = (p.N + TN - 1) / TN;
  const int tiles = m_tiles * n_tiles;
  const int k_stages = (p.k_tiles + 3) / 4;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { bar_init(full(s), 1); bar_init(empty(s), 1); }
    for (int a = 0; a < 2; ++a) { bar_init(tfull(a), 1); bar_init(tempty(a), 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(const_cast<uint32_t*>(tmem_slot))),
                 "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; bool ok = true;
      for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x) {
        const int mt = t % m_tiles, nt = t / m_tiles;
        for (int ks = 0; ks < k_stages; ++ks) {
          ok = bar_wait(empty(stage), phase ^ 1u, ab, 0x900u | stage);
          if (!ok) break;
          const int n_kt = min(4, p.k_tiles - 4 * ks);                 // scale tiles of this stage
          const uint32_t sa = base + stage * STAGE, sb = sa + A_BYTES, sfa = sb + B_BYTES, sfb = sfa + SF_BYTES;
          bar_expect(full(stage), (uint32_t)(A_BYTES + B_BYTES + 2 * n_kt * SF_TILE));
          tma_2d(sa, &tmA, ks * ROW_BYTES, mt * TM, full(stage));
          tma_2d(sb, &tmB, ks * ROW_BYTES, nt * TN, full(stage));
          bulk_g2s(sfa, p.sfa + ((size_t)mt * p.k_tiles + 4 * ks) * SF_TILE, (uint32_t)(n_kt * SF_TILE), full(stage));
          bulk_g2s(sfb, p.sfb + ((size_t)nt * p.k_tiles + 4 * ks) * SF_TILE, (uint32_t)(n_kt * SF_TILE), full(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) { const unsigned long long t0 = now_ns(); while (now_ns() - t0 < 2000000ull) {} }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; int it = 0; bool ok = true;
      const uint32_t idesc = idesc_fp4();
      for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++it) {
        const int acc = it & 1;
        ok = bar_wait(tempty(acc), (uint32_t)((it >> 1) & 1) ^ 1u, ab, 0xA00u | acc);
        if (!ok) break;
        fence_after();
        const uint32_t d = tmem + (uint32_t)(acc * TN);
        for (int ks = 0; ks < k_stages; ++ks) {
          ok = bar_wait(full(stage), phase, ab, 0xB00u | stage);
          if (!ok) break;
          fence_after();
          const int n_kt = min(4, p.k_tiles - 4 * ks);
          const uint32_t sa = base + stage * STAGE, sb = sa + A_BYTES, sfa = sb + B_BYTES, sfb = sfa + SF_BYTES;
          for (int j = 0; j < n_kt; ++j) {
            cp_sf(tmem + (uint32_t)(COL_SFA + 4 * j), desc_sf(sfa + j * SF_TILE));
            cp_sf(tmem + (uint32_t)(COL_SFB + 4 * j), desc_sf(sfb + j * SF_TILE));
          }
          const uint64_t da = desc_sw128(sa), db = desc_sw128(sb);
          for (int j = 0; j < n_kt; ++j)            // 64 codes = 32 bytes further inside the swizzled row: +2
            mma_fp4(d, da + 2u * j, db + 2u * j, idesc, tmem + (uint32_t)(COL_SFA + 4 * j), tmem + (uint32_t)(COL_SFB + 4 * j),
                    (ks | j) != 0 ? 1u : 0u);
          commit(empty(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) commit(tfull(acc));
      }
    }
  } else {
    const int quarter = warp & 3;
    const float alpha = *p.sa * *p.sb;
    int it = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
      const int acc = it & 1;
      bool ok = bar_wait(tfull(acc), (uint32_t)((it >> 1) & 1), ab, 0xC00u | acc);
      if (!__all_sync(0xffffffffu, ok)) break;
      fence_after();
      const int mt = t % m_tiles, nt = t / m_tiles;
      const int row = mt * TM + quarter * 32 + lane;
      const uint32_t trow = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * TN);
#pragma unroll 1
      for (int c = 0; c < TN; c += 16) {
        const int col = nt * TN + c;
        if (col >= p.N) break;
        uint32_t r[16];
        ld16(trow + (uint32_t)c, r);
        if (row < p.M) {
          __nv_bfloat16* out = p.C + (long long)row * p.ldc + col;
          if (col + 16 <= p.N && ((reinterpret_cast<uintptr_t>(out) & 15) == 0)) {
            uint32_t o[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(r[2 * i]) * alpha, __uint_as_float(r[2 * i + 1]) * alpha);
              o[i] = *reinterpret_cast<uint32_t*>(&v);
            }
            reinterpret_cast<uint4*>(out)[0] = make_uint4(o[0], o[1], o[2], o[3]);
            reinterpret_cast<uint4*>(out)[1] = make_uint4(o[4], o[5], o[6], o[7]);
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i)
              if (col + i < p.N) out[i] = __float2bfloat16_rn(__uint_as_float(r[i]) * alpha);
          }
        }
      }
      fence_before();
      __syncwarp();
      if (lane == 0) bar_arrive(tempty(acc));
    }
  }
  __syncwarp();
  fence_before();
  __syncthreads();
  if (warp == 1) {
    fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// rows x (K/2) bytes, bytes of a row contiguous; box = 128 bytes x 128 rows.
int byte_map(faar_ctx* ctx, CUtensorMap* map, const void* ptr, int rows, int K) {
  cuuint64_t dims[2] = {(cuuint64_t)(K / 2), (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)(K / 2)};
  cuuint32_t box[2] = {(cuuint32_t)ROW_BYTES, (cuuint32_t)TM};
  cuuint32_t es[2] = {1, 1};
  CUresult r = reinterpret_cast<EncodeFn>(ctx->encode_tiled)(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims,
                                                             strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : (int)cudaErrorInvalidValue;
}

}  // namespace

int faar_launch_nvfp4_gemm(faar_ctx* ctx, int M, int N, int K, const uint8_t* A, const uint8_t* sfa, const float* sa,
                           const uint8_t* B, const uint8_t* sfb, const float* sb, void* C, int64_t ldc, uint32_t* status) {
  static_assert(TM == TN, "one box shape serves both operands");
  static_assert(SMEM <= 227 * 1024, "shared memory budget");
  CUtensorMap tmA, tmB;
  int e = byte_map(ctx, &tmA, A, M, K);
  if (e) return e;
  e = byte_map(ctx, &tmB, B, N, K);
  if (e) return e;
  cudaError_t ce = cudaFuncSetAttribute(nvfp4_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (ce != cudaSuccess) return (int)ce;
  P4 p;
  p.M = M; p.N = N; p.K = K; p.sfa = sfa; p.sfb = sfb; p.k_tiles = (K + KI - 1) / KI;
  p.sa = sa; p.sb = sb; p.C = reinterpret_cast<__nv_bfloat16*>(C); p.ldc = ldc; p.status = status;
  const long long tiles = (long long)((M + TM - 1) / TM) * ((N + TN - 1) / TN);
  const int grid = (int)(tiles < ctx->num_sms ? tiles : ctx->num_sms);
  faar_prof_scope ps(ctx, FAAR_K_NVFP4_GEMM);
  nvfp4_gemm_kernel<<<grid, THREADS, SMEM, ctx->stream>>>(tmA, tmB, p);
  return (int)cudaGetLastError();
}
