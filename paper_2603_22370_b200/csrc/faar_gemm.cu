// Tensor-core kernels of the FAAR layer step for sm_100a.
//
// One persistent, warp-specialised kernel computes C[M,N] = A[M,Kc] * B[N,Kc]^T for BF16 operands that
// both have the contraction dimension contiguous.  It runs as clusters of two CTAs that share one
// 256 x bn output tile (tcgen05 cta_group::2): CTA r of the pair loads rows [128 r, 128 r + 128) of the
// A tile and rows [bn/2 r, bn/2 (r+1)) of the B tile into its own shared memory, the leader CTA (r = 0)
// issues the 256 x bn x 16 MMAs for both, and each CTA ends up with its 128 accumulator rows x bn
// columns (FP32) in its own tensor memory.  Halving the B tile per CTA halves the shared-memory
// traffic per flop, which is what bounds a single-CTA 128 x 256 tile.
//   warp 0      : TMA producer  (cp.async.bulk.tensor, 128-byte swizzle, multi-stage ring; both CTAs,
//                                both crediting the leader's "full" barrier)
//   warp 1      : MMA issuer    (leader CTA only; tcgen05.mma kind::f16, tcgen05.commit to the
//                                "empty" / "accumulator full" barriers of both CTAs)
//   warps 2..   : epilogue      (tcgen05.ld; two accumulator buffers, so the epilogue of one tile
//                                overlaps the main loop of the next)
// The three epilogues are the operations of the layer step:
//   REF : Y_fp = X W^T                                   (Procedure step 8)
//   FWD : r = Y_q - Y_ref, sum r^2, dY = 2c r -> dY^T     (steps 9-10, Eq. 5 first term)
//   BWD : G = dY^T X -> dV -> optimiser update + clip     (step 13, Eq. 5, with Eq. 2/3 chain rule)
// In all of them the accumulator row (TMEM lane) is the output feature o.
//
// Every wait on an mbarrier is bounded: after about two seconds the waiting thread records a code in
// the status word, raises a CTA-wide abort flag and every role leaves its loop; both CTAs then meet at
// the closing cluster barrier, free their tensor memory and exit.
#include <cuda.h>

#include "faar_internal.cuh"

namespace {

constexpr int BM = 128;                // accumulator rows per CTA; the CTA pair covers 256
constexpr int BK = 64;                 // 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;
constexpr int PW = 64;                         // BWD epilogue: columns of a staged panel of G
constexpr int PANEL_BYTES = 32 * PW * 4;       // one 32-row x PW-column FP32 panel per TMEM lane quarter
constexpr int SMEM_LIMIT = 227 * 1024;
constexpr int CTL_BYTES = 512;
constexpr int MAX_EPI_WARPS = 16;

// The tile width bn (accumulator columns, a multiple of 16 up to 256) is a launch parameter chosen by
// the host (pick_bn).  Shared memory and tensor memory are laid out for the widest tile.
constexpr int BN_MAX = 256;
// WIDE: the pair's tile is 256 x 512, the whole of tensor memory as ONE accumulator (two column halves of 256,
// each fed by its own MMA from the same A stage).  A stage then holds this CTA's 128 rows of both B halves.
// Per flop the tile pulls a quarter less operand data through the SM than a 256 x 256 tile, which is what
// bounds these kernels; the price is that the epilogue of a tile no longer overlaps the next tile's main loop
// (the two halves drain one after the other while the issuer waits).
constexpr int WIDE_BN = 2 * BN_MAX;
template <int MODE, bool WIDE = false> struct Cfg {
  static constexpr int EPI_WARPS = MODE == FAAR_GEMM_BWD ? 16 : 8;
  static constexpr int THREADS = 32 * (2 + EPI_WARPS);
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int BH_BYTES = (BN_MAX / 2) * BK * 2;       // this CTA's 128 rows of one 256-column B tile
  static constexpr int B_BYTES = WIDE ? 2 * BH_BYTES : BH_BYTES;   // slot size
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int EPI_BYTES = MODE == FAAR_GEMM_BWD ? 4 * PANEL_BYTES : 0;
  static constexpr int FIT = (SMEM_LIMIT - 1024 - CTL_BYTES - EPI_BYTES) / STAGE_BYTES;
  static constexpr int STAGES = FIT > 8 ? 8 : FIT;
  static constexpr int TMEM_COLS = 2 * BN_MAX;                 // two accumulator buffers
  static constexpr int COL_GROUPS = EPI_WARPS / 4;             // warps sharing one TMEM lane quarter
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 /*alignment slack*/ + CTL_BYTES;
};

// ---- PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address, in CTA `rank` of the cluster, of the object that sits at shared::cta address `addr` here
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// arrive on a barrier given by its shared::cluster address (this CTA's or the peer's)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
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
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

struct AbortCtl {
  volatile int* flag;     // shared memory
  uint32_t* status;       // global status word
  unsigned long long limit_ns = WAIT_LIMIT_NS;
};

// Returns false if the wait was abandoned (time limit, or another thread raised the flag).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const AbortCtl& ac, uint32_t code) {
  unsigned long long t0 = global_ns();
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 0xFF) == 0) {
      if (*ac.flag) return false;
      if (global_ns() - t0 > ac.limit_ns) {
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

// 2-D tiled TMA load into this CTA's shared memory; the byte count is credited to `bar`, which may be
// a barrier of either CTA of the pair (shared::cluster address).  No multicast.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar,
                                            uint64_t l2_policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar), "l"(l2_policy) : "memory");
}
// L2 eviction policies: GEMM operands are re-read by many CTAs and should stay; the per-weight
// optimiser state streams through once per step and should be the first to go.
__device__ __forceinline__ uint64_t l2_policy_keep() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_stream() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ float4 ldg128_stream(const float* ptr, uint64_t pol) {
  float4 v;
  asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.f32 {%0,%1,%2,%3}, [%4], %5;"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr), "l"(pol));
  return v;
}
__device__ __forceinline__ void stg128_stream(float* ptr, float a, float b, float c, float d, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1,%2,%3,%4}, %5;" ::"l"(ptr), "f"(a), "f"(b), "f"(c), "f"(d), "l"(pol)
               : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// When all MMAs issued so far have completed, arrive on the barrier at offset `bar` in both CTAs.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
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
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ float4 lds128(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}

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
// The same for an operand stored with its M (or N) index contiguous and the contraction index as the row
// ("MN-major"): 64 elements (128 B) of one contraction index form a row, 8 consecutive contraction indices a
// 1024-byte swizzle atom; atoms follow each other along the contraction (stride byte offset, 1024 B: a TMA box
// of 64 x 64 elements lands exactly so) and along M / N (leading byte offset: the next 64-element box, 8192 B on).
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)(8192 >> 4) << 16;                // leading byte offset: next 64 M / N elements
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset: next 8 contraction indices
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
constexpr int MN_BOX = 64;                         // M / N elements per MN-major TMA box
constexpr int MN_BOX_BYTES = MN_BOX * BK * 2;      // 8192
constexpr uint32_t MN_KSTEP = (UMMA_K * 128) >> 4; // 16 contraction indices on: 2048 B in the address field
// Instruction descriptor: D = F32, A = B = BF16, M = 256 (the CTA pair), N = bn; bits 15 / 16 say that A / B is
// MN-major instead of K-major.
__device__ __forceinline__ uint32_t make_idesc(int bn, int a_mn = 0, int b_mn = 0) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
         ((uint32_t)(bn >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
}

struct KParams {
  int M, N, Kc;
  int bn;                 // tile width
  int n_full_cols;        // tile columns of full width; the columns after them are bn/2 wide (tail split)
  int a_mn, b_mn;         // operand stored with M (N) contiguous, [Kc, M] / [Kc, N], instead of [M, Kc] / [N, Kc]
  uint32_t* status;
  long long ext_yout, ext_dyt, ext_state, ext_wsoft;   // bytes of Yout, dYt, each of V / m / u / dV, wsoft_next (debug checks)
  // REF / FWD
  void* Yout; int yout_dtype; long long ldy;
  const void* Yref; int yref_dtype;
  int yref_t;             // Y_ref / Y_out stored transposed: [O, ldy] with ldy >= T rounded up to 16
  __nv_bfloat16* dYt; long long ld_dyt;
  float mse2c;
  float act_scale;        // FWD: Y_q = act_scale * acc; BWD: G = act_scale * acc
  float* partials;
  // BWD: M = O, N = K
  float* V; const uint8_t* code; const uint8_t* scales; const float* s_global;
  float* adam_m; float* adam_u; float* dV;
  float beta, lam_over_n, lr, b1, b2, eps, inv_bc1, inv_bc2; int opt;
  // BWD, optional: the next step's BF16 forward operand, from the updated v (null = not wanted)
  __nv_bfloat16* wsoft_next; float beta_next;
  // BWD, optional: the CTA that finishes last also forms the step's two loss values
  uint32_t* fin_counter;            // workspace word, zero between launches
  const float* fin_mse_partials; int fin_n_mse; float fin_scale_mse;
  float fin_scale_round; float* fin_out2;   // {L_MSE, L_round}; null = no final sums here
};

// Tile t of the launch: the first n_full_cols tile columns are bn wide, the remaining columns bn/2
// (half-width tiles fill the last, partly empty wave of the CTA pairs and halve the epilogue that
// nothing overlaps).  Tiles are numbered row block fastest, all full-width tiles first.
struct TileCoord { int m0, n0, w; };
__device__ __forceinline__ TileCoord tile_coord(const KParams& p, int t, int m_tiles) {
  const int full_tiles = m_tiles * p.n_full_cols;
  TileCoord c;
  if (t < full_tiles) {
    c.m0 = (t % m_tiles) * (2 * BM);
    c.n0 = (t / m_tiles) * p.bn;
    c.w = p.bn;
  } else {
    const int u = t - full_tiles;
    c.m0 = (u % m_tiles) * (2 * BM);
    c.n0 = p.n_full_cols * p.bn + (u / m_tiles) * (p.bn / 2);
    c.w = p.bn / 2;
  }
  return c;
}
__device__ __forceinline__ int tile_count(const KParams& p, int m_tiles) {
  const int rest = p.N - p.n_full_cols * p.bn;                    // columns covered by half-width tiles
  const int half_cols = rest > 0 ? (rest + p.bn / 2 - 1) / (p.bn / 2) : 0;
  return m_tiles * (p.n_full_cols + half_cols);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}

// Debug build (-DFAAR_DEBUG): every epilogue store is checked against the extent of the tensor it writes; a
// store that would leave it is skipped and recorded in the status word (0xD00 | tensor id), which
// faar_check_status reports.  No trap, no assert: the kernel runs on.  In the normal build the check is gone.
#ifdef FAAR_DEBUG
__device__ __forceinline__ bool dbg_in_range(const KParams& p, const void* ptr, long long bytes, const void* base,
                                             long long extent, uint32_t id) {
  const long long off = reinterpret_cast<const char*>(ptr) - reinterpret_cast<const char*>(base);
  if (off >= 0 && off + bytes <= extent) return true;
  atomicCAS(p.status, 0u, 0xD00u | id);
  return false;
}
#define FAAR_DBG_OK(p, ptr, bytes, base, extent, id) dbg_in_range(p, ptr, bytes, base, extent, id)
#else
#define FAAR_DBG_OK(p, ptr, bytes, base, extent, id) true
#endif

// ---- epilogues: one call handles 16 accumulator columns of one row ---------------------------
// REF: write acc to Y[t, o].
__device__ __forceinline__ void epi_ref(const KParams& p, int o, int t0, const uint32_t (&acc)[16]) {
  if (o >= p.M) return;
  if (p.yref_t) {                                    // row o of the transposed target: 16 contiguous values
    // (the row is padded to a multiple of 16, so a full vector store stays inside it)
    if (p.yout_dtype == FAAR_BF16) {
      uint4* d4 = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.Yout) + (long long)o * p.ldy + t0);
      float a[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) a[j] = (t0 + j < p.N) ? __uint_as_float(acc[j]) : 0.f;
      if (!FAAR_DBG_OK(p, d4, 32, p.Yout, p.ext_yout, 1u)) return;
      d4[0] = make_uint4(pack_bf16x2(a[0], a[1]), pack_bf16x2(a[2], a[3]), pack_bf16x2(a[4], a[5]), pack_bf16x2(a[6], a[7]));
      d4[1] = make_uint4(pack_bf16x2(a[8], a[9]), pack_bf16x2(a[10], a[11]), pack_bf16x2(a[12], a[13]), pack_bf16x2(a[14], a[15]));
    } else {
      float4* d4 = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.Yout) + (long long)o * p.ldy + t0);
      if (!FAAR_DBG_OK(p, d4, 64, p.Yout, p.ext_yout, 1u)) return;
#pragma unroll
      for (int q = 0; q < 4; ++q)
        d4[q] = make_float4((t0 + 4 * q < p.N) ? __uint_as_float(acc[4 * q]) : 0.f,
                            (t0 + 4 * q + 1 < p.N) ? __uint_as_float(acc[4 * q + 1]) : 0.f,
                            (t0 + 4 * q + 2 < p.N) ? __uint_as_float(acc[4 * q + 2]) : 0.f,
                            (t0 + 4 * q + 3 < p.N) ? __uint_as_float(acc[4 * q + 3]) : 0.f);
    }
    return;
  }
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    int t = t0 + j;
    if (t < p.N) {
      float a = __uint_as_float(acc[j]);
      if (p.yout_dtype == FAAR_BF16) {
        __nv_bfloat16* q = reinterpret_cast<__nv_bfloat16*>(p.Yout) + (long long)t * p.ldy + o;
        if (FAAR_DBG_OK(p, q, 2, p.Yout, p.ext_yout, 1u)) *q = __float2bfloat16_rn(a);
      } else {
        float* q = reinterpret_cast<float*>(p.Yout) + (long long)t * p.ldy + o;
        if (FAAR_DBG_OK(p, q, 4, p.Yout, p.ext_yout, 1u)) *q = a;
      }
    }
  }
}

// FWD: residual, sum of squares, dY^T.
// Y_ref[t0..t0+15, o] for this lane's output feature o.
__device__ __forceinline__ void load_yref(const KParams& p, int o, int t0, float (&yr)[16]) {
  if (o >= p.M) return;
  if (p.yref_t) {
    if (p.yref_dtype == FAAR_BF16) {
      const uint4* y4 = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.Yref) + (long long)o * p.ldy + t0);
      const uint4 a = y4[0], b = y4[1];
      const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        yr[2 * i] = __uint_as_float(w[i] << 16);
        yr[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
      }
    } else {
      const float4* y4 = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.Yref) + (long long)o * p.ldy + t0);
#pragma unroll
      for (int q = 0; q < 4; ++q) { const float4 v = y4[q]; yr[4 * q] = v.x; yr[4 * q + 1] = v.y; yr[4 * q + 2] = v.z; yr[4 * q + 3] = v.w; }
    }
    return;
  }
  if (p.yref_dtype == FAAR_BF16) {
    const __nv_bfloat16* y = reinterpret_cast<const __nv_bfloat16*>(p.Yref);
#pragma unroll
    for (int j = 0; j < 16; ++j) yr[j] = (t0 + j < p.N) ? __bfloat162float(y[(long long)(t0 + j) * p.ldy + o]) : 0.f;
  } else {
    const float* y = reinterpret_cast<const float*>(p.Yref);
#pragma unroll
    for (int j = 0; j < 16; ++j) yr[j] = (t0 + j < p.N) ? y[(long long)(t0 + j) * p.ldy + o] : 0.f;
  }
}

__device__ __forceinline__ float epi_fwd(const KParams& p, int o, int t0, const uint32_t (&acc)[16], const float (&yr)[16]) {
  if (o >= p.M) return 0.f;
  float ss = 0.f;
  float dy[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    float a = __uint_as_float(acc[j]) * p.act_scale;
    float r = (t0 + j < p.N) ? a - yr[j] : 0.f;
    ss = fmaf(r, r, ss);
    dy[j] = p.mse2c * r;
  }
  __nv_bfloat16* drow = p.dYt + (long long)o * p.ld_dyt + t0;
  if (!FAAR_DBG_OK(p, drow, 2 * (t0 + 16 <= p.N ? 16 : p.N - t0), p.dYt, p.ext_dyt, 2u)) return ss;
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
      if (t0 + j < p.N) {
        __nv_bfloat16* q = yq + (p.yref_t ? (long long)o * p.ldy + t0 + j : (long long)(t0 + j) * p.ldy + o);
        if (FAAR_DBG_OK(p, q, 2, p.Yout, p.ext_yout, 1u)) *q = __float2bfloat16_rn(__uint_as_float(acc[j]) * p.act_scale);
      }
  }
  return ss;
}

// ---- BWD epilogue ----------------------------------------------------------------------------
__device__ __forceinline__ float sqrt_approx(float x) {       // sqrt(0) = 0, about 1 ulp
  float y;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The four epilogue warps that share a TMEM lane quarter stage a 32-row x PW-column panel of G in
// shared memory (row r at panel + 4 PW r, its 16-byte units XOR-swizzled by (r & 7)); then warp `sub`
// of the quarter takes rows 8 sub .. 8 sub + 7, LPR = PW / 4 lanes per row and lane l the columns
// 4 (l % LPR)..+3, so that one warp instruction moves 512 bytes of V / m / u as 32 / LPR row pieces of
// 4 PW contiguous bytes each: whole lines as 16-byte vectors.  (A panel of 128 columns gives one 512-byte
// piece per instruction but leaves room for five TMA stages only; the sixth stage is worth more.)
// The per-weight state of RPG such instructions is requested together before any of it is computed
// (one measured fastest: the sixteen warps of a CTA already keep 24 KB of state loads in flight).
// FULL: the panel lies wholly inside the matrix (no bounds tests).
// o_first: output feature of panel row 0; k_first: input feature of panel column 0; k_end: first
// input feature beyond the tile (or the matrix).
// Returns the Round Loss contribution of the pre-update v's.
constexpr int RPG = 1;
constexpr int LPR = PW / 4;                     // lanes per panel row
constexpr int RPI = 32 / LPR;                   // rows per warp instruction
constexpr int ITS = 8 / RPI;                    // instructions per warp and panel
template <int OPT, bool FULL>
__device__ __forceinline__ float epi_bwd_rows(const KParams& p, uint32_t panel, int lane, int sub, int o_first,
                                              int k_first, int k_end, float s_global) {
  const int cu = lane % LPR;                                       // 16-byte unit of the row
  const int kcol = k_first + 4 * cu;
  const bool col_ok = FULL || kcol < k_end;
  const int r0 = 8 * sub + lane / LPR;                             // this lane's row in the first instruction
  const long long e0 = (long long)(o_first + r0) * p.N + kcol;     // row r0 element of this lane
  float* const Vp = p.V + e0;
  float* const Mp = p.adam_m + e0;
  float* const Up = p.adam_u + e0;
  const uint8_t* const Cp = p.code + (e0 >> 1);
  const uint8_t* const Sp = p.scales + (e0 >> 4);
  const float bl = p.beta * 1.44269504088896341f;                 // beta log2(e): e^x as 2^(x log2 e)
  const float hbl = -0.5f * bl;
  const float c1 = 1.f - p.b1, c2 = 1.f - p.b2;
  const float step_size = p.lr * p.inv_bc1;
  const float rbc2 = sqrtf(p.inv_bc2);                            // sqrt(u / bc2) = sqrt(u) sqrt(1 / bc2)
  const float lam4 = -4.f * p.lam_over_n;                         // (lambda / N) (4 - 8 v) = lam4 (2 v - 1)
  float nbl_next, hbl_next;                                       // OPT & 2: constants of the next step's Eq. 3
  faar_operand_consts(p.beta_next, &nbl_next, &hbl_next);
  const uint64_t stream = l2_policy_stream();
  const uint64_t vkeep = l2_policy_keep();       // the updated V is the next kernel's input (soft weights)
  float tt = 0.f, n_el = 0.f;                                     // sum of (2 v - 1)^2, elements seen
#pragma unroll
  for (int grp = 0; grp < ITS / RPG; ++grp) {
    float4 v[RPG], m[RPG], u[RPG];
    uint32_t cw[RPG], sb[RPG];
    bool ok[RPG];
#pragma unroll
    for (int q = 0; q < RPG; ++q) {
      const int i = RPI * (RPG * grp + q);                              // row r0 + i
      ok[q] = FULL || (col_ok && o_first + r0 + i < p.M);
      if (ok[q]) {
        const int off = i * p.N;
        v[q] = ldg128_stream(Vp + off, stream);
        cw[q] = *reinterpret_cast<const uint16_t*>(Cp + (off >> 1));
        sb[q] = Sp[off >> 4];
        if (OPT & 1) {
          m[q] = ldg128_stream(Mp + off, stream);
          u[q] = ldg128_stream(Up + off, stream);
        }
      }
    }
#pragma unroll
    for (int q = 0; q < RPG; ++q) {
      if (ok[q]) {
        const int i = RPI * (RPG * grp + q);
        const int row = r0 + i;
        const int off = i * p.N;
        const float4 g4 = lds128(panel + (uint32_t)row * (4u * PW) + (uint32_t)((cu ^ (row & 7)) << 4));
        const float G[4] = {g4.x, g4.y, g4.z, g4.w};
        const float vv[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
        // s beta / 2 (the narrowest interval is 0.5 wide); act_scale: G = act_scale * acc
        const float sc = __fmul_rn(faar_e4m3_to_float(sb[q]), s_global);
        const float sbh = sc * (0.5f * p.beta * p.act_scale);
        // byte j: log2 of (interval width / 0.5) of element j, looked up by its interval index k (0 0 0 0 1 1 2)
        const uint32_t ksel = cw[q] & 0x7777u;
        const uint32_t wlog = __byte_perm(0u, 0x00020101u, ksel);
        // OPT & 2: bytes 3 and 2 of the lower node's float (0 .5 1 1.5 2 3 4) by the same look-up
        uint32_t lo_hi = 0u, lo_lo = 0u;
        if (OPT & 2) {
          lo_hi = __byte_perm(0x3F3F3F00u, 0x00404040u, ksel);
          lo_lo = __byte_perm(0xC0800000u, 0x00804000u, ksel);
        }
        float wn[4];
        float g[4], vn[4], mn[4], un[4];
        float mm[4], uu[4];
        if (OPT & 1) {
          mm[0] = m[q].x; mm[1] = m[q].y; mm[2] = m[q].z; mm[3] = m[q].w;
          uu[0] = u[q].x; uu[1] = u[q].y; uu[2] = u[q].z; uu[3] = u[q].w;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float ex = ex2_approx(-fabsf(fmaf(bl, vv[j], hbl)));         // e^-|beta (v - 0.5)|
          const float hs = rcp_approx(1.0f + ex);
          const float dh = ex * hs * hs;                                     // h (1 - h)
          // dh times the width factor by an add to its exponent field (a dh flushed to 0 becomes ~1e-38), then
          // the sign of w from bit 3 of the nibble
          const uint32_t wexp = (j < 3 ? wlog << (23 - 8 * j) : wlog >> 1) & 0x01800000u;
          const uint32_t sgn = (cw[q] << (28 - 4 * j)) & 0x80000000u;
          float chain = sbh * __uint_as_float(__float_as_uint(dh) + wexp);
          chain = __uint_as_float(__float_as_uint(chain) ^ sgn);
          const float t = fmaf(2.f, vv[j], -1.f);
          g[j] = fmaf(G[j], chain, lam4 * t);
          tt = fmaf(t, t, tt);
          if (OPT & 1) {
            mn[j] = fmaf(p.b1, mm[j], c1 * g[j]);
            un[j] = fmaf(p.b2, uu[j], c2 * g[j] * g[j]);
            const float den = fmaf(sqrt_approx(un[j]), rbc2, p.eps);
            vn[j] = __saturatef(fmaf(-step_size, mn[j] * rcp_approx(den), vv[j]));   // clip to [0, 1]
          } else {
            vn[j] = __saturatef(fmaf(-p.lr, g[j], vv[j]));
          }
          if (OPT & 2) {
            // Eq. 2 / Eq. 3 at the updated v with the next step's beta: (lo + h width) s with the sign of w, in
            // the soft-weights kernel's operations, so that the BF16 operand is the same bit for bit
            const float lo = __uint_as_float(__byte_perm(lo_hi, lo_lo, (uint32_t)((j << 12) | ((4 + j) << 8))) & 0xFFFF0000u);
            const float wd = __uint_as_float(0x3F000000u + wexp);
            const float mag = faar_operand_weight(faar_sigmoid_operand(nbl_next, hbl_next, vn[j]), lo, wd, sc);
            wn[j] = __uint_as_float(__float_as_uint(mag) ^ sgn);
          }
        }
        // one check covers the five stores below: they share the element offset e0 + off
        if (!FAAR_DBG_OK(p, Vp + off, 16, p.V, p.ext_state, 3u)) continue;
        if ((OPT & 2) && !FAAR_DBG_OK(p, p.wsoft_next + e0 + off, 8, p.wsoft_next, p.ext_wsoft, 4u)) continue;
        if (OPT & 2)
          *reinterpret_cast<uint2*>(p.wsoft_next + e0 + off) = make_uint2(pack_bf16x2(wn[0], wn[1]), pack_bf16x2(wn[2], wn[3]));
        if (p.dV) stg128_stream(p.dV + e0 + off, g[0], g[1], g[2], g[3], stream);
        if (OPT & 1) {
          stg128_stream(Mp + off, mn[0], mn[1], mn[2], mn[3], stream);
          stg128_stream(Up + off, un[0], un[1], un[2], un[3], stream);
        }
        stg128_stream(Vp + off, vn[0], vn[1], vn[2], vn[3], vkeep);
        n_el += 4.f;
      }
    }
  }
  return n_el - tt;                                               // sum of 1 - (2 v - 1)^2
}

// ---- the kernel ------------------------------------------------------------------------------
// Launched as clusters of two CTAs along x: CTAs 2c and 2c+1 form pair c.
// MN: bit 0 = the A operand, bit 1 = the B operand is stored with its M / N index contiguous (KParams.a_mn / b_mn);
// a compile-time choice, so that the K-major kernels carry no trace of the other layout in their issue loops.
template <int MODE, int OPT, bool WIDE, int MN>
__global__ void __launch_bounds__(Cfg<MODE, WIDE>::THREADS, 1)
faar_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmBh, const KParams p) {
  using C = Cfg<MODE, WIDE>;
  constexpr bool A_MN = (MN & 1) != 0, B_MN = (MN & 2) != 0;
  const int BN = p.bn;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;       // the same offset in both CTAs of the pair
  uint8_t* smem = smem_raw + (base - raw);
  const uint32_t epi_u32 = base + C::STAGES * C::STAGE_BYTES;
  uint8_t* ctl = smem + C::STAGES * C::STAGE_BYTES + C::EPI_BYTES;
  const uint32_t ctl_u32 = epi_u32 + C::EPI_BYTES;
  // control block: full[S], empty[S], tmem_full[2], tmem_empty[2], tmem base, abort flag
  auto full_bar = [&](int s) { return ctl_u32 + 8u * s; };
  auto empty_bar = [&](int s) { return ctl_u32 + 8u * (C::STAGES + s); };
  auto tfull_bar = [&](int a) { return ctl_u32 + 8u * (2 * C::STAGES + a); };
  auto tempty_bar = [&](int a) { return ctl_u32 + 8u * (2 * C::STAGES + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctl + 8 * (2 * C::STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + 8 * (2 * C::STAGES + 4) + 4);
  const AbortCtl ac{abort_flag, p.status};

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();             // 0 = leader of the pair
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int m_tiles = (p.M + 2 * BM - 1) / (2 * BM);
  // WIDE: tiles of 512 columns, numbered row block fastest; no tail split
  const int total_tiles = WIDE ? m_tiles * ((p.N + WIDE_BN - 1) / WIDE_BN) : tile_count(p, m_tiles);
  const int k_blocks = (p.Kc + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    // accumulator-empty barriers are used in the leader only: every epilogue warp of both CTAs arrives there
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * C::EPI_WARPS); }
    for (int q = 0; q < 8; ++q) mbar_init(ctl_u32 + 256u + 8u * q, 4);   // panel staged / panel consumed, per lane quarter
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  cluster_sync_all();                                  // barriers of both CTAs are initialised
  tc_fence_after();
  faar_pdl_sync();                                     // set-up done; now wait for the previous kernel's data
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer (both CTAs) ----------------
    if (lane == 0) {
      const uint64_t keep = l2_policy_keep();
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      auto coords = [&](int tile) {
        TileCoord tc;
        if (WIDE) { tc.m0 = (tile % m_tiles) * (2 * BM); tc.n0 = (tile / m_tiles) * WIDE_BN; tc.w = BN_MAX; }
        else tc = tile_coord(p, tile, m_tiles);
        return tc;
      };
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
        const TileCoord tc = coords(tile);
        const int m0 = tc.m0 + (int)rank * BM;
        const int n0 = tc.n0 + (int)rank * (tc.w / 2);
        const CUtensorMap* mapB = tc.w == BN ? &tmB : &tmBh;      // box of w/2 rows
        for (int kb = 0; kb < k_blocks; ++kb) {
          ok = mbar_wait(empty_bar(stage), phase ^ 1u, ac, 0x100u | stage);
          if (!ok) break;
          const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
          // the leader's barrier collects the bytes of both CTAs' copies
          if (rank == 0)
            mbar_expect_tx(full_bar(stage), WIDE ? 2u * (uint32_t)(C::A_BYTES + C::B_BYTES)
                                                 : 2u * (uint32_t)(C::A_BYTES + (tc.w / 2) * BK * 2));
          const uint32_t leader_full = map_to_cta(full_bar(stage), 0);
          if (A_MN) {                                          // two boxes of 64 rows of A, each [64 k][64 m]
            tma_load_2d(sa, &tmA, m0, kb * BK, leader_full, keep);
            tma_load_2d(sa + MN_BOX_BYTES, &tmA, m0 + MN_BOX, kb * BK, leader_full, keep);
          } else {
            tma_load_2d(sa, &tmA, kb * BK, m0, leader_full, keep);
          }
          if (B_MN) {                                          // w/2 = 128 or 64 rows of B: two boxes or one
            tma_load_2d(sb, &tmB, n0, kb * BK, leader_full, keep);
            if (tc.w / 2 > MN_BOX) tma_load_2d(sb + MN_BOX_BYTES, &tmB, n0 + MN_BOX, kb * BK, leader_full, keep);
          } else {
            tma_load_2d(sb, mapB, kb * BK, n0, leader_full, keep);
          }
          // second column half (rows beyond the matrix arrive as zeros)
          if (WIDE) tma_load_2d(sb + C::BH_BYTES, &tmB, kb * BK, n0 + BN_MAX, leader_full, keep);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // give copies already in flight a bounded chance to land before the CTA exits
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 2000000ull) {}
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (leader CTA only) ----------------
    if (lane == 0 && rank == 0) {
      int stage = 0; uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs, ++it) {
        // WIDE: the two column halves take the place of the two accumulator buffers; both must be drained
        const int acc = WIDE ? 0 : it & 1;
        const uint32_t acc_phase = WIDE ? it & 1 : (it >> 1) & 1;
        ok = mbar_wait(tempty_bar(acc), acc_phase ^ 1u, ac, 0x200u | acc);
        if (ok && WIDE) ok = mbar_wait(tempty_bar(1), acc_phase ^ 1u, ac, 0x201u);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * BN_MAX;
        const uint32_t idesc = make_idesc(WIDE ? BN_MAX : tile_coord(p, tile, m_tiles).w, A_MN ? 1 : 0, B_MN ? 1 : 0);
        for (int kb = 0; kb < k_blocks; ++kb) {
          ok = mbar_wait(full_bar(stage), phase, ac, 0x300u | stage);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
          const uint64_t da = A_MN ? make_smem_desc_mn(sa) : make_smem_desc(sa);
          const uint64_t db = B_MN ? make_smem_desc_mn(sb) : make_smem_desc(sb);
          constexpr uint32_t ka = A_MN ? MN_KSTEP : 2u, kbs = B_MN ? MN_KSTEP : 2u;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing 16 bf16 = 32 bytes inside the swizzled row: +2 in the 16-byte address field
            // (MN-major: 16 rows of 128 bytes further on)
            tc_mma_bf16(tmem_d, da + ka * k, db + kbs * k, idesc, (kb | k) != 0 ? 1u : 0u);
            if (WIDE)
              tc_mma_bf16(tmem_d + BN_MAX, da + 2u * k, make_smem_desc(sb + C::BH_BYTES) + 2u * k, idesc,
                          (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit_pair(empty_bar(stage));            // frees this stage in both CTAs
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) {
          tc_commit_pair(tfull_bar(acc));              // accumulator ready in both CTAs
          if (WIDE) tc_commit_pair(tfull_bar(1));
        }
      }
    }
  } else {
    // ---------------- epilogue (both CTAs) ----------------
    const int ew = warp - 2;
    const int quarter = warp & 3;                      // TMEM lanes this warp may read
    // REF / FWD: the warps that share a lane quarter split the tile's columns in 16-column chunks
    const int cg = ew >> 2;                            // which of the warps sharing this lane quarter
    float warp_acc = 0.f;
    float s_global = 0.f;
    if (MODE == FAAR_GEMM_BWD) s_global = *p.s_global;
    uint32_t pn = 0;                                   // panels this quarter has staged so far
    bool dead = false;
    // One pass per accumulator buffer that fills: a tile, or (WIDE) a 256-column half of a tile.
    for (int vt = 0;; ++vt) {
      const int it = WIDE ? vt >> 1 : vt;
      const int tile = pair + it * n_pairs;
      if (tile >= total_tiles) break;
      const int acc = WIDE ? vt & 1 : it & 1;
      const uint32_t acc_phase = WIDE ? it & 1 : (it >> 1) & 1;
      bool ok = mbar_wait(tfull_bar(acc), acc_phase, ac, 0x400u | acc);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      TileCoord tc;
      if (WIDE) { tc.m0 = (tile % m_tiles) * (2 * BM); tc.n0 = (tile / m_tiles) * WIDE_BN + acc * BN_MAX; tc.w = BN_MAX; }
      else tc = tile_coord(p, tile, m_tiles);
      const int m0 = tc.m0 + (int)rank * BM, n0 = tc.n0, TW = tc.w;
      const int cols_per_warp = ((TW / C::COL_GROUPS + 15) / 16) * 16;
      const int col_begin = cg * cols_per_warp;
      const int col_end = min(col_begin + cols_per_warp, TW);
      const int o = m0 + quarter * 32 + lane;
      const uint32_t trow = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN_MAX);
      if constexpr (MODE == FAAR_GEMM_BWD) {
        // PW-column panels, staged by the four warps of this lane quarter together (see epi_bwd_rows)
        const int sub = ew >> 2;
        const uint32_t panel = epi_u32 + (uint32_t)quarter * PANEL_BYTES;
        const uint32_t pfull = ctl_u32 + 256u + 16u * quarter, pdone = pfull + 8u;
        const int o_first = m0 + quarter * 32;
        bool released = false;
#pragma unroll 1
        for (int pc = 0; pc < TW; pc += PW) {
          if (n0 + pc >= p.N || o_first >= p.M) break;   // the same decision in all four warps
          // the quarter's previous panel has been consumed by all four warps
          bool okp = mbar_wait(pdone, (pn & 1u) ^ 1u, ac, 0x500u | quarter);
          if (!__all_sync(0xffffffffu, okp)) { dead = true; break; }
          static_assert(PW == 64, "each of the four warps stages PW / 4 = 16 accumulator columns");
          const int c = pc + 16 * sub;
          if (c < TW && n0 + c < p.N) {
            uint32_t r[16];
            tmem_ld16(trow + (uint32_t)c, r);
            tmem_ld_wait();
#pragma unroll
            for (int u = 0; u < 4; ++u)
              sts128(panel + (uint32_t)lane * (4u * PW) + (uint32_t)(((4 * sub + u) ^ (lane & 7)) << 4), r[4 * u],
                     r[4 * u + 1], r[4 * u + 2], r[4 * u + 3]);
          }
          if (pc + PW >= TW || n0 + pc + PW >= p.N) {    // this warp's last read of the accumulator
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
            released = true;
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(pfull);
          okp = mbar_wait(pfull, pn & 1u, ac, 0x600u | quarter);
          if (!__all_sync(0xffffffffu, okp)) { dead = true; break; }
          const int k_end = min(p.N, n0 + TW);           // columns of this tile that exist
          if (o_first + 32 <= p.M && n0 + pc + PW <= k_end)
            warp_acc += epi_bwd_rows<OPT, true>(p, panel, lane, sub, o_first, n0 + pc, k_end, s_global);
          else
            warp_acc += epi_bwd_rows<OPT, false>(p, panel, lane, sub, o_first, n0 + pc, k_end, s_global);
          __syncwarp();
          if (lane == 0) mbar_arrive(pdone);
          ++pn;
        }
        if (dead) break;
        if (!released) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
        }
        continue;
      } else {
        if (MODE == FAAR_GEMM_FWD && p.yref_t && p.yref_dtype == FAAR_BF16) {
          // transposed BF16 target: this lane's 64 values of four chunks are requested together
          // (eight 16-byte loads in flight), so a tile costs two load latencies instead of one per chunk
#pragma unroll 1
          for (int cb = col_begin; cb < col_end; cb += 64) {
            if (n0 + cb >= p.N) break;                   // warp-uniform
            uint4 yraw[8];
            if (o < p.M) {
              const uint4* y4 = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.Yref) +
                                                               (long long)o * p.ldy + n0 + cb);
#pragma unroll
              for (int q = 0; q < 4; ++q)
                if (cb + 16 * q < col_end && n0 + cb + 16 * q < p.N) { yraw[2 * q] = y4[2 * q]; yraw[2 * q + 1] = y4[2 * q + 1]; }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int c = cb + 16 * q;
              if (c < col_end && n0 + c < p.N) {         // warp-uniform
                uint32_t r[16];
                tmem_ld16(trow + (uint32_t)c, r);
                tmem_ld_wait();
                const uint32_t w[8] = {yraw[2 * q].x, yraw[2 * q].y, yraw[2 * q].z, yraw[2 * q].w,
                                       yraw[2 * q + 1].x, yraw[2 * q + 1].y, yraw[2 * q + 1].z, yraw[2 * q + 1].w};
                float yr[16];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  yr[2 * i] = __uint_as_float(w[i] << 16);
                  yr[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
                }
                warp_acc += epi_fwd(p, o, n0 + c, r, yr);
              }
            }
          }
        } else {
#pragma unroll 1
          for (int c = col_begin; c < col_end; c += 16) {
            if (n0 + c >= p.N) break;                    // warp-uniform
            uint32_t r[16];
            tmem_ld16(trow + (uint32_t)c, r);
            tmem_ld_wait();
            if (MODE == FAAR_GEMM_REF) {
              epi_ref(p, o, n0 + c, r);
            } else {
              float yr[16];
              load_yref(p, o, n0 + c, yr);
              warp_acc += epi_fwd(p, o, n0 + c, r, yr);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
    }
    if (MODE != FAAR_GEMM_REF) {
      warp_acc = faar_warp_sum(warp_acc);
      if (lane == 0) p.partials[blockIdx.x * C::EPI_WARPS + ew] = warp_acc;
    }
  }

  __syncwarp();
  // Neither CTA may leave while the other can still read its shared memory, write its tensor memory
  // or arrive on its barriers.
  tc_fence_before();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }

  if constexpr (MODE == FAAR_GEMM_BWD) {
    // Final loss sums by whichever CTA finishes last: always the same partials in the same order
    // (strided double accumulation, then a tree), so the result does not depend on which CTA it is.
    if (p.fin_out2 != nullptr) {
      double* sh = reinterpret_cast<double*>(smem);          // the operand ring is idle by now
      volatile int* last_flag = reinterpret_cast<volatile int*>(smem + 256 * sizeof(double));
      if (threadIdx.x == 0) {
        __threadfence();                                     // this CTA's partials, ordered by the barrier above
        int last = 0;
        // after a wait that gave up the partials are incomplete: no final sums (the caller re-initialises
        // the workspace, which also clears this counter)
        if (*reinterpret_cast<volatile uint32_t*>(p.status) == 0u) {
          const uint32_t prev = atomicAdd(p.fin_counter, 1u);
          last = prev == gridDim.x - 1;
          if (last) *p.fin_counter = 0u;                     // ready for the next launch
        }
        __threadfence();
        *last_flag = last;
      }
      __syncthreads();
      if (*last_flag) {
        const int n_round = (int)gridDim.x * C::EPI_WARPS;
        for (int which = 0; which < 2; ++which) {
          const float* src = which ? p.partials : p.fin_mse_partials;
          const int n = which ? n_round : p.fin_n_mse;
          double acc = 0.0;
          if (threadIdx.x < 256)
            for (int i = threadIdx.x; i < n; i += 256) acc += (double)__ldcg(src + i);
          __syncthreads();
          if (threadIdx.x < 256) sh[threadIdx.x] = acc;
          __syncthreads();
          for (int st = 128; st > 0; st >>= 1) {
            if (threadIdx.x < st) sh[threadIdx.x] += sh[threadIdx.x + st];
            __syncthreads();
          }
          if (threadIdx.x == 0) p.fin_out2[which] = (float)(sh[0] * (double)(which ? p.fin_scale_round : p.fin_scale_mse));
        }
      }
    }
  }
}

// A wait that nothing will ever satisfy, with a short limit: exercises the give-up path of the bounded
// waits (status word, flag, orderly exit) without any other kernel machinery.
__global__ void __launch_bounds__(64, 1) wait_selftest_kernel(uint32_t* status, unsigned long long limit_ns) {
  __shared__ alignas(8) unsigned long long bar;
  __shared__ int flag;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  AbortCtl ac{&flag, status, limit_ns};
  if (threadIdx.x == 0) (void)mbar_wait(b, 0u, ac, 0x700u);       // nobody arrives: gives up after limit_ns
  __syncthreads();
  if (threadIdx.x == 32) (void)mbar_wait(b, 0u, ac, 0x701u);      // sees the raised flag and leaves at once
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

// An operand stored [kc_rows, mn_cols] (M or N contiguous, row stride ld elements): boxes of 64 x 64.
int make_map_mn(faar_ctx* ctx, CUtensorMap* map, const void* ptr, int kc_rows, int mn_cols, int64_t ld) {
  cuuint64_t dims[2] = {(cuuint64_t)mn_cols, (cuuint64_t)kc_rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)MN_BOX, (cuuint32_t)BK};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : (int)cudaErrorInvalidValue;
}

// Tile width for an M x N output.  A tile's time is set by the operand bytes it pulls through the SM (A rows
// are not shared between tiles), not by its columns, so 256-wide tiles win wherever they were measured
// against narrower ones that fill more CTA pairs (down_proj-, gate-, q- and k_proj-shaped layers), with one
// exception: the dW GEMM of a small layer, whose per-weight epilogue is heavy, gains from spreading 128-wide
// tiles over twice as many pairs while fewer than half of the pairs would have a 256-wide tile.  A tile is
// never wider than the output rounded up to 32 columns.
int pick_bn_k_major(const faar_ctx* ctx, int mode, int M, int N, int pairs);
int pick_bn(const faar_ctx* ctx, int mode, int M, int N, int pairs, bool b_mn) {
  const int bn = pick_bn_k_major(ctx, mode, M, N, pairs);
  // an N-contiguous B comes in boxes of 64 columns per CTA: widths 128 and 256 only
  return b_mn && bn % 128 != 0 ? (N <= 128 ? 128 : BN_MAX) : bn;
}
int pick_bn_k_major(const faar_ctx* ctx, int mode, int M, int N, int pairs) {
  if (ctx->tune_bn >= 128 && ctx->tune_bn <= BN_MAX && ctx->tune_bn % 16 == 0) return ctx->tune_bn;
  const long long m_tiles = (M + 2 * BM - 1) / (2 * BM);
  int bn = BN_MAX;
  if (N < BN_MAX) bn = N <= 128 ? 128 : (N + 31) / 32 * 32;
  if (mode == FAAR_GEMM_BWD && 2 * m_tiles * ((N + BN_MAX - 1) / BN_MAX) < pairs) bn = 128;
  return bn;
}

// How many trailing tile columns to cut into half-width tiles.  Tiles go to CTA pairs round-robin, all
// full-width tiles first.  A half tile costs 0.75 of a full one (its A rows are loaded all the same), and
// the epilogue of a pair's last tile is not overlapped by anything (0.4 of that tile's cost).  Returns the
// number of full-width columns that minimises the busiest pair's time (ties: fewer half tiles).
int pick_full_cols(const faar_ctx* ctx, int M, int N, int bn, int pairs) {
  const int m_tiles = (M + 2 * BM - 1) / (2 * BM);
  const int n_cols = (N + bn - 1) / bn;
  if (bn % 32 != 0) return n_cols;
  if (ctx->tune_tail >= 0) return ctx->tune_tail < n_cols ? n_cols - ctx->tune_tail : 0;
  double best = -1.0;
  int best_full = n_cols;
  for (int split = 0; split <= n_cols && split <= 16; ++split) {
    const int full_cols = n_cols - split;
    const long long full_tiles = (long long)m_tiles * full_cols;
    const int rest = N - full_cols * bn;
    const long long half_tiles = rest > 0 ? (long long)m_tiles * ((rest + bn / 2 - 1) / (bn / 2)) : 0;
    const long long total = full_tiles + half_tiles;
    double worst = 0.0;
    for (int p = 0; p < pairs && p < total; ++p) {
      double load = 0.0, last = 0.0;
      for (long long t = p; t < total; t += pairs) { last = t < full_tiles ? 1.0 : 0.75; load += last; }
      load += 0.4 * last;
      if (load > worst) worst = load;
    }
    if (best < 0.0 || worst < best - 1e-9) { best = worst; best_full = full_cols; }
  }
  return best_full;
}

// Whether a launch takes 256 x 512 tiles (see Cfg): only on request (ctx->tune_wide == 1) and where the shape
// allows.  Measured: on a down_proj-shaped layer (2048 x 8192, 4096 tokens) in a short job at full clocks the
// forward GEMM gains 1-4 % (64 tiles in one wave instead of 128 in two unequal ones), but in the long,
// power-capped jobs of whole decoder blocks the same launch and the q / o projections lose 6-10 %; the dW GEMM
// loses 29 % (its long epilogue is no longer hidden) and the plain product loses whenever it needs more than
// one wave.  No rule was found that wins consistently, so the default never takes them.
bool pick_wide(const faar_ctx* ctx, int N, int bn) {
  return ctx->tune_wide == 1 && bn == BN_MAX && N > BN_MAX;
}

template <int MODE, int OPT, bool WIDE, int MN>
int launch_variant(faar_ctx* ctx, const faar_gemm_args* a, KParams& kp, int* n_partials_out, int bn, int max_pairs,
                   const cudaLaunchConfig_t& base_cfg) {
  using C = Cfg<MODE, WIDE>;
  static_assert(C::STAGES >= 3, "ring too short");
  static_assert(C::SMEM_BYTES <= SMEM_LIMIT, "shared memory budget");
  static_assert(C::EPI_WARPS <= MAX_EPI_WARPS, "partials budget");
  auto kern = faar_gemm_kernel<MODE, OPT, WIDE, MN>;
  cudaError_t ce = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
  if (ce != cudaSuccess) return (int)ce;
  cudaLaunchConfig_t cfg = base_cfg;
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  kp.bn = bn;
  kp.n_full_cols = WIDE ? 0 : pick_full_cols(ctx, a->M, a->N, bn, max_pairs);
  if (a->b_mn && bn != BN_MAX) kp.n_full_cols = (a->N + bn - 1) / bn;      // half tiles of a 128-wide tile would be 32 columns per CTA
  CUtensorMap tmA, tmB, tmBh;
  kp.a_mn = a->a_mn; kp.b_mn = a->b_mn;
  int e = a->a_mn ? make_map_mn(ctx, &tmA, a->A, a->Kc, a->M, a->lda) : make_map(ctx, &tmA, a->A, a->M, a->Kc, a->lda, BM);
  if (e) return e;
  if (a->b_mn) {
    e = make_map_mn(ctx, &tmB, a->B, a->Kc, a->N, a->ldb);    // one map serves full and half-width tiles
    tmBh = tmB;
  } else {
    e = make_map(ctx, &tmB, a->B, a->N, a->Kc, a->ldb, bn / 2);
    if (e) return e;
    e = make_map(ctx, &tmBh, a->B, a->N, a->Kc, a->ldb, bn % 32 == 0 ? bn / 4 : bn / 2);   // half-width tiles
  }
  if (e) return e;
  const long long m_tiles = (a->M + 2 * BM - 1) / (2 * BM);
  const int rest_cols = a->N - kp.n_full_cols * bn;
  const long long tiles = WIDE ? m_tiles * ((a->N + WIDE_BN - 1) / WIDE_BN)
                               : m_tiles * (kp.n_full_cols + (rest_cols > 0 ? (rest_cols + bn / 2 - 1) / (bn / 2) : 0));
  const int pairs = (int)(tiles < max_pairs ? tiles : max_pairs);
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  if (n_partials_out) *n_partials_out = 2 * pairs * C::EPI_WARPS;
  ctx->last_gemm_bn = WIDE ? WIDE_BN : bn;
  ctx->last_gemm_pairs = pairs;
  ctx->last_gemm_split = WIDE ? 0 : (a->N + bn - 1) / bn - kp.n_full_cols;
  faar_prof_scope ps(ctx, MODE == FAAR_GEMM_REF ? FAAR_K_GEMM_REF : (MODE == FAAR_GEMM_FWD ? FAAR_K_GEMM_FWD : FAAR_K_GEMM_BWD));
  ce = cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmBh, kp);
  if (ce != cudaSuccess) return (int)ce;
  return (int)cudaGetLastError();
}

template <int MODE, int OPT = 0>
int launch(faar_ctx* ctx, const faar_gemm_args* a, KParams& kp, int* n_partials_out) {
  using C = Cfg<MODE>;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.blockDim = dim3(C::THREADS, 1, 1);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = ctx->stream;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  // how many CTA pairs the device can hold at once (a GPC with an odd SM count strands one SM); asked once
  // per context and kernel mode, with the context's device current (every variant takes one CTA per SM)
  int& max_pairs = ctx->gemm_max_pairs[MODE == FAAR_GEMM_BWD ? 2 + OPT : MODE];
  if (max_pairs == 0) {
    auto kern = faar_gemm_kernel<MODE, OPT, false, 0>;
    cudaError_t ce = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
    if (ce != cudaSuccess) return (int)ce;
    cfg.gridDim = dim3(2 * (ctx->num_sms / 2), 1, 1);
    int n = 0;
    ce = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
    if (ce != cudaSuccess || n <= 0) { (void)cudaGetLastError(); n = ctx->num_sms / 2; }
    if (n > ctx->num_sms / 2) n = ctx->num_sms / 2;
    max_pairs = n;
  }
  const int bn = pick_bn(ctx, MODE, a->M, a->N, max_pairs, a->b_mn != 0);
  const int mn = (a->a_mn ? 1 : 0) | (a->b_mn ? 2 : 0);
  // which operand layouts a mode is ever launched with: the plain product with A untransposed (input gradient),
  // the dW product with B or with both untransposed
  if constexpr (MODE == FAAR_GEMM_REF) {
    if (mn == 1) return launch_variant<MODE, OPT, false, 1>(ctx, a, kp, n_partials_out, bn, max_pairs, cfg);
  }
  if constexpr (MODE == FAAR_GEMM_BWD) {
    if (mn == 2) return launch_variant<MODE, OPT, false, 2>(ctx, a, kp, n_partials_out, bn, max_pairs, cfg);
    if (mn == 3) return launch_variant<MODE, OPT, false, 3>(ctx, a, kp, n_partials_out, bn, max_pairs, cfg);
  }
  if (mn != 0) return (int)cudaErrorInvalidValue;
  if (pick_wide(ctx, a->N, bn)) return launch_variant<MODE, OPT, true, 0>(ctx, a, kp, n_partials_out, bn, max_pairs, cfg);
  return launch_variant<MODE, OPT, false, 0>(ctx, a, kp, n_partials_out, bn, max_pairs, cfg);
}

}  // namespace

int faar_launch_wait_selftest(faar_ctx* ctx, uint32_t* status, unsigned long long limit_ns) {
  wait_selftest_kernel<<<1, 64, 0, ctx->stream>>>(status, limit_ns);
  return (int)cudaGetLastError();
}

int faar_gemm_max_partials(const faar_ctx* ctx, int, int) { return ctx->num_sms * MAX_EPI_WARPS; }

int faar_launch_gemm(faar_ctx* ctx, const faar_gemm_args* a, int* n_partials_out) {
  KParams kp;
  kp.M = a->M; kp.N = a->N; kp.Kc = a->Kc; kp.bn = BN_MAX; kp.n_full_cols = 0; kp.status = a->status;
  {
    const long long ysz = a->yout_dtype == FAAR_BF16 ? 2 : 4;
    // Y is [N(T), ldy] or, transposed, [M(O), ldy]; the last row ends after its last valid (or padded) column
    kp.ext_yout = a->Yout ? (a->yref_t ? ((long long)(a->M - 1) * a->ldy + (a->N + 15) / 16 * 16)
                                       : ((long long)(a->N - 1) * a->ldy + a->M)) * ysz : 0;
    kp.ext_dyt = a->dYt ? ((long long)(a->M - 1) * a->ld_dyt + a->N) * 2 : 0;
    kp.ext_state = (long long)a->M * a->N * 4;
    kp.ext_wsoft = (long long)a->M * a->N * 2;
  }
  kp.Yout = a->Yout; kp.yout_dtype = a->yout_dtype; kp.ldy = a->ldy;
  kp.Yref = a->Yref; kp.yref_dtype = a->yref_dtype; kp.yref_t = a->yref_t;
  kp.dYt = a->dYt; kp.ld_dyt = a->ld_dyt; kp.mse2c = a->mse2c; kp.act_scale = a->act_scale; kp.partials = a->partials;
  kp.V = a->V; kp.code = a->code; kp.scales = a->scales; kp.s_global = a->s_global;
  kp.adam_m = a->adam_m; kp.adam_u = a->adam_u; kp.dV = a->dV;
  kp.beta = a->beta; kp.lam_over_n = a->lam_over_n; kp.lr = a->lr; kp.b1 = a->b1; kp.b2 = a->b2; kp.eps = a->eps;
  kp.inv_bc1 = a->inv_bc1; kp.inv_bc2 = a->inv_bc2; kp.opt = a->opt;
  kp.wsoft_next = a->wsoft_next; kp.beta_next = a->beta_next;
  kp.fin_counter = a->fin_counter; kp.fin_mse_partials = a->fin_mse_partials; kp.fin_n_mse = a->fin_n_mse;
  kp.fin_scale_mse = a->fin_scale_mse; kp.fin_scale_round = a->fin_scale_round; kp.fin_out2 = a->fin_out2;
  // the BWD epilogue forms row offsets of up to 7 rows in 32-bit element counts (the entry points refuse
  // such a K with FAAR_ERR_SHAPE before they get here)
  if (a->mode == FAAR_GEMM_BWD && (long long)a->N * 8 > 0x7FFFFFFFll) return (int)cudaErrorInvalidValue;

  switch (a->mode) {
    case FAAR_GEMM_REF: return launch<FAAR_GEMM_REF>(ctx, a, kp, n_partials_out);
    case FAAR_GEMM_FWD: return launch<FAAR_GEMM_FWD>(ctx, a, kp, n_partials_out);
    case FAAR_GEMM_BWD:
      // OPT bit 0: Adam; bit 1: also write the next step's forward operand
      if (a->wsoft_next)
        return a->opt == 1 ? launch<FAAR_GEMM_BWD, 3>(ctx, a, kp, n_partials_out)
                           : launch<FAAR_GEMM_BWD, 2>(ctx, a, kp, n_partials_out);
      return a->opt == 1 ? launch<FAAR_GEMM_BWD, 1>(ctx, a, kp, n_partials_out)
                         : launch<FAAR_GEMM_BWD, 0>(ctx, a, kp, n_partials_out);
  }
  return (int)cudaErrorInvalidValue;
}
