// Causal attention for head_dim 64 on the tcgen05 tensor cores (sm_100a): the forward kernel first, then the two
// backward kernels (dQ; dK and dV), which are built the same way and described where they start.
//
// Forward.  One CTA takes 128 queries of one head and sweeps the keys in tiles of 64 (one sweep):
//   S   = Q K_j^T       tcgen05.mma  M = 128, N = 64, K = 64   -> 64 FP32 columns of tensor memory
//   P_j = 2^(c S - m)   four warps, one query row per thread (its tensor-memory lane): no shuffles; the row
//                       goes back to tensor memory as BF16 pairs, 32 columns (tcgen05.st)
//   O  += P_j V_j       tcgen05.mma  M = 128, N = 64, K = 64   accumulating in 64 more columns over the whole sweep;
//                       P_j is the A operand, read from tensor memory; V_j is read from shared memory as it lies
//                       in memory (keys as rows: a B operand with its N index contiguous)
//   m is the row's reference, not its running maximum: it moves to a tile's maximum only when that exceeds it by
//   more than 2^8 (probabilities stay below 2^8, the final division by their sum and lse = m + log2(sum) are
//   exact either way); only then is O rescaled, in tensor memory, between two P V products.
// Q, K_j, V_j arrive by TMA (two stages for K and V).  A fifth warp's lane 0 issues every copy and every MMA; the
// scores have two buffers in tensor memory, so S of tile j + 1 is formed while the warps work on tile j, and two
// CTAs per SM overlap what remains serial (softmax -> P V).
// Rows of a query tile beyond the sequence end compute on whatever rows follow in memory (or zeros past the
// tensor) and are not stored; keys beyond the end are masked.
// Every barrier wait is bounded; a wait that gives up records a code in a status word of this module (read by
// faar_attention_status), raises the CTA's abort flag and all roles leave.
#include <cuda.h>

#include <type_traits>

#include "faar_internal.cuh"

namespace {

constexpr int QT = 128, KT = 64, HD = 64;
constexpr int Q_BYTES = QT * HD * 2, KV_BYTES = KT * HD * 2;
constexpr int OFF_K = Q_BYTES, OFF_V = OFF_K + 2 * KV_BYTES, OFF_CTL = OFF_V + 2 * KV_BYTES;
constexpr int CTL = 256;
constexpr int SMEM = OFF_CTL + CTL + 1024;
constexpr int THREADS = 160;
constexpr int TMEM_COLS = 256;                     // S of even / odd tiles: columns 0..63 / 64..127, O: 128..191, P: 192..223 / 224..255
constexpr float FWD_SLACK = 8.0f;                  // log2 of how far a tile's maximum may exceed the row's reference
constexpr unsigned long long LIMIT_NS = 2000000000ull;

__device__ uint32_t g_attn_status;                 // 0 = no wait has given up since the last read-and-clear

struct TcParams {
  __nv_bfloat16* out; float* lse;
  long long ldo;
  int B, S, H, Hkv;
  float scale_log2;
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
__device__ __noinline__ bool bar_wait_slow(uint32_t b, uint32_t parity, volatile int* abort_flag, uint32_t code) {
  const unsigned long long t0 = now_ns();
  for (uint32_t spin = 1;; ++spin) {
    if (bar_try(b, parity)) return true;
    if ((spin & 0xFF) == 0) {
      if (*abort_flag) return false;
      if (now_ns() - t0 > LIMIT_NS) { atomicCAS(&g_attn_status, 0u, code); *abort_flag = 1; return false; }
    }
  }
}
__device__ __forceinline__ bool bar_wait(uint32_t b, uint32_t parity, volatile int* abort_flag, uint32_t code) {
  return bar_try(b, parity) ? true : bar_wait_slow(b, parity, abort_flag, code);
}
__device__ __forceinline__ void tma_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Operand with the contraction index contiguous: rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t desc_k_major(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// Operand with its N index contiguous (64 of them = one 128-byte row per contraction index): groups of 8
// contraction indices 1024 B apart; a single 64-wide group along N, so the leading offset is not used.
__device__ __forceinline__ uint64_t desc_n_major(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)(8192 >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// D = F32, A = B = BF16, M = 128, N = 64; bit 16: B has its N index contiguous.
__device__ __forceinline__ uint32_t idesc(int b_n_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_n_major << 16) | ((uint32_t)(KT >> 3) << 17) | ((uint32_t)(QT >> 4) << 24);
}
__device__ __forceinline__ void mma(uint32_t d, uint64_t da, uint64_t db, uint32_t id, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(d), "l"(da), "l"(db), "r"(id), "r"(acc) : "memory");
}
// 32 consecutive FP32 columns of this thread's tensor-memory lane
__device__ __forceinline__ void ld32(uint32_t taddr, float (&r)[32]) {
  uint32_t u[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,"
      "%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]), "=r"(u[9]),
        "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]), "=r"(u[17]), "=r"(u[18]),
        "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]),
        "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) r[i] = __uint_as_float(u[i]);
}
// Two such loads in flight together (one wait for both)
__device__ __forceinline__ void ld32x2(uint32_t ta, uint32_t tb, float (&a)[32], float (&b)[32]) {
  uint32_t u[32], v[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%64];\n\t"
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%65];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]), "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31]),
        "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(ta), "r"(tb) : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) { a[i] = __uint_as_float(u[i]); b[i] = __uint_as_float(v[i]); }
}
// 32 consecutive 32-bit columns of this thread's tensor-memory lane, written (BF16 pairs of an A operand)
__device__ __forceinline__ void st32(uint32_t taddr, const uint32_t (&u)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,"
      "%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]), "r"(u[8]), "r"(u[9]),
        "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15]), "r"(u[16]), "r"(u[17]), "r"(u[18]), "r"(u[19]),
        "r"(u[20]), "r"(u[21]), "r"(u[22]), "r"(u[23]), "r"(u[24]), "r"(u[25]), "r"(u[26]), "r"(u[27]), "r"(u[28]), "r"(u[29]),
        "r"(u[30]), "r"(u[31])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void st16(uint32_t taddr, const uint32_t (&u)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]), "r"(u[8]), "r"(u[9]),
        "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15])
      : "memory");
}
__device__ __forceinline__ void wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D (+)= A B with A read from tensor memory (128 lanes = rows, two BF16 contraction elements per 32-bit column,
// the lower index in the lower half) and B from shared memory
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a_tmem, uint64_t db, uint32_t id, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
               ::"r"(d), "r"(a_tmem), "l"(db), "r"(id), "r"(acc) : "memory");
}
// 2^x on the special-function unit, one instruction (relative error about 2^-22; -inf gives 0; results below the
// normal range are flushed to zero, which is what a probability that small should be)
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// max of three in one instruction
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(THREADS, 2)
attn_fwd64_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV, const TcParams p) {
  extern __shared__ uint8_t raw[];
  const uint32_t base = (s32(raw) + 1023u) & ~1023u;
  uint8_t* smem = raw + (base - s32(raw));
  const uint32_t ctl = base + OFF_CTL;
  const uint32_t bar_q = ctl, bar_p = ctl + 72, bar_o = ctl + 80;
  auto kfull = [&](int s) { return ctl + 8u + 8u * s; };
  auto vfull = [&](int s) { return ctl + 24u + 8u * s; };
  auto bar_s = [&](int s) { return ctl + 40u + 8u * s; };         // scores of a tile in buffer s are complete
  auto bar_sfree = [&](int s) { return ctl + 56u + 8u * s; };     // ... have been read by all 128 rows
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + OFF_CTL + 96);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_CTL + 100);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // one-dimensional grid, query tile slowest and descending: CTAs start in order of decreasing work
  const int hb = p.H * p.B;
  const int qt = (int)(gridDim.x / hb) - 1 - (int)(blockIdx.x / hb);
  const int h = (blockIdx.x % hb) % p.H, b = (blockIdx.x % hb) / p.H;
  const int g = h / (p.H / p.Hkv);
  const long long seq0 = (long long)b * p.S;
  const int q0 = qt * QT;
  const int last_q = min(q0 + QT, p.S) - 1;
  const int n_kt = last_q / KT + 1;                          // key tiles that some query of this tile sees

  if (threadIdx.x == 0) {
    bar_init(bar_q, 1);
    for (int s = 0; s < 2; ++s) { bar_init(kfull(s), 1); bar_init(vfull(s), 1); }
    for (int s = 0; s < 2; ++s) { bar_init(bar_s(s), 1); bar_init(bar_sfree(s), 128); }
    bar_init(bar_o, 1); bar_init(bar_p, 128);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(const_cast<uint32_t*>(tmem_slot))),
                 "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t sQ = base;
  auto sK = [&](int s) { return base + OFF_K + (uint32_t)s * KV_BYTES; };
  auto sV = [&](int s) { return base + OFF_V + (uint32_t)s * KV_BYTES; };

  if (warp == 4) {
    // ---------------- copies and MMAs: one thread ----------------
    if (lane == 0) {
      auto load_k = [&](int j) { bar_expect(kfull(j & 1), KV_BYTES); tma_2d(sK(j & 1), &tmK, g * HD, (int)(seq0 + (long long)j * KT), kfull(j & 1)); };
      auto load_v = [&](int j) { bar_expect(vfull(j & 1), KV_BYTES); tma_2d(sV(j & 1), &tmV, g * HD, (int)(seq0 + (long long)j * KT), vfull(j & 1)); };
      bar_expect(bar_q, Q_BYTES);
      tma_2d(sQ, &tmQ, h * HD, (int)(seq0 + q0), bar_q);
      load_k(0); load_v(0);
      if (n_kt > 1) { load_k(1); load_v(1); }
      bool ok = bar_wait(bar_q, 0u, abort_flag, 0xA01u);
      const uint32_t id_s = idesc(0), id_pv = idesc(1);
      // S of tile j into score buffer j & 1.  The scores of tile j + 1 are issued before this thread waits for the
      // probabilities of tile j, so the tensor cores form them while the four warps work on tile j.
      auto issue_s = [&](int j) {
        const uint64_t da = desc_k_major(sQ), db = desc_k_major(sK(j & 1));
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) mma(tmem + 64u * (uint32_t)(j & 1), da + 2u * k, db + 2u * k, id_s, k != 0 ? 1u : 0u);
        commit(bar_s(j & 1));
      };
      if (ok) ok = bar_wait(kfull(0), 0u, abort_flag, 0xA10u);
      if (ok) { fence_after(); issue_s(0); }
      for (int j = 0; j < n_kt && ok; ++j) {
        const int st = j & 1;
        const uint32_t ph = (uint32_t)((j >> 1) & 1);
        if (j + 1 < n_kt) {
          ok = bar_wait(kfull((j + 1) & 1), (uint32_t)(((j + 1) >> 1) & 1), abort_flag, 0xA10u | ((j + 1) & 1));
          // its score buffer last held tile j - 1
          if (ok && j >= 1) ok = bar_wait(bar_sfree((j + 1) & 1), (uint32_t)(((j - 1) >> 1) & 1), abort_flag, 0xA20u);
          if (!ok) break;
          fence_after();
          issue_s(j + 1);
        }
        // P_j written (into P buffer j & 1): S_j has been read, so its K stage is free
        ok = bar_wait(bar_p, (uint32_t)(j & 1), abort_flag, 0xA30u);
        if (!ok) break;
        if (j + 2 < n_kt) load_k(j + 2);
        ok = bar_wait(vfull(st), ph, abort_flag, 0xA40u | st);
        // P V_{j-1} complete: its V stage is free
        if (ok && j > 0) ok = bar_wait(bar_o, (uint32_t)((j - 1) & 1), abort_flag, 0xA50u);
        if (!ok) break;
        if (j >= 1 && j + 1 < n_kt) load_v(j + 1);
        fence_after();
        {
          const uint64_t db = desc_n_major(sV(st));
          const uint32_t ta = tmem + 192u + 32u * (uint32_t)st;      // P_j: 16 contraction steps = 8 columns
#pragma unroll
          for (int k = 0; k < KT / 16; ++k) mma_ts(tmem + 128u, ta + 8u * k, db + 128u * k, id_pv, (j | k) != 0 ? 1u : 0u);
        }
        commit(bar_o);
      }
      if (!ok) { const unsigned long long t0 = now_ns(); while (now_ns() - t0 < 2000000ull) {} }   // copies in flight
    }
  } else {
    // ---------------- softmax: thread = query row = tensor-memory lane ----------------
    const int row = 32 * warp + lane;
    const int qi = q0 + row;
    const uint32_t t_lane = tmem + ((uint32_t)(32 * warp) << 16), t_o = t_lane + 128u;
    float m = -INFINITY, l = 0.f;                             // the reference the row's probabilities are relative to; their sum
    bool ok = true;
    for (int j = 0; j < n_kt; ++j) {
      const int k0 = j * KT;
      const uint32_t t_s = t_lane + 64u * (uint32_t)(j & 1);
      ok = bar_wait(bar_s(j & 1), (uint32_t)((j >> 1) & 1), abort_flag, 0xB10u);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      fence_after();
      float s[KT];
      {
        float t[32], t2[32];
        ld32x2(t_s, t_s + 32u, t, t2);
#pragma unroll
        for (int i = 0; i < 32; ++i) { s[i] = t[i]; s[32 + i] = t2[i]; }
      }
      fence_before();
      bar_arrive(bar_sfree(j & 1));
      if (k0 + KT - 1 > q0 || k0 + KT > p.S) {                // the tile crosses some row's diagonal, or the sequence end
#pragma unroll
        for (int i = 0; i < KT; ++i)
          if (!(k0 + i <= qi && k0 + i < p.S)) s[i] = -INFINITY;
      }
      float mx4[4] = {s[0], s[1], s[2], s[3]};                   // four independent chains, two scores per instruction
#pragma unroll
      for (int i = 4; i < KT; i += 8) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (i + 2 * c + 1 < KT) mx4[c] = max3(mx4[c], s[i + 2 * c], s[i + 2 * c + 1]);
      }
      const float m_tile = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
      // The output accumulates in tensor memory over the whole sweep.  The row's reference moves only when a tile's
      // maximum exceeds it by more than 2^FWD_SLACK: until then the probabilities (at most 2^FWD_SLACK) and their sum
      // stay relative to the old one, which the final division and lse = m + log2(l) undo exactly, and the
      // accumulated output needs no rescaling.
      const float m_new = m_tile > m + FWD_SLACK ? m_tile : m;
      const float ref = m_new == -INFINITY ? 0.f : m_new;     // a row beyond the sequence may have seen no key
      const float alpha = ex2(m - ref);                       // 1 while the reference stays
      const bool moved = m_new != m && j > 0;
      bool prev_done = j == 0;                                // P V_{j-1} known to be complete
      if (__any_sync(0xffffffffu, moved)) {                   // O = O * 2^(m_old - m_new), between P V_{j-1} and P V_j
        ok = bar_wait(bar_o, (uint32_t)((j - 1) & 1), abort_flag, 0xB20u);
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
        prev_done = true;
        fence_after();
        const float a = moved ? alpha : 1.0f;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          float t[32];
          uint32_t u[32];
          ld32(t_o + 32u * half, t);
#pragma unroll
          for (int i = 0; i < 32; ++i) u[i] = __float_as_uint(t[i] * a);
          st32(t_o + 32u * half, u);
        }
      }
      // exponent arguments and sums two at a time (packed FP32 multiply-add and add: the same roundings)
      const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nr2 = make_float2(-ref, -ref);
      float2 sum2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      uint32_t pk[KT / 2];
#pragma unroll
      for (int w = 0; w < KT / 2; ++w) {
        const float2 x = __ffma2_rn(make_float2(s[2 * w], s[2 * w + 1]), sc2, nr2);
        const float2 e = make_float2(ex2(x.x), ex2(x.y));
        sum2[w & 1] = __fadd2_rn(sum2[w & 1], e);
        pk[w] = pack2(e.x, e.y);
      }
      st32(t_lane + 192u + 32u * (uint32_t)(j & 1), pk);             // this row of P_j, an A operand in tensor memory
      fence_before();
      bar_arrive(bar_p);
      l = l * alpha + ((sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y));
      m = m_new;
      // every completion of bar_o is observed in order (it has had this tile's softmax to happen): P buffer j & 1 is
      // then free for tile j + 2, and the parity of a later wait cannot be mistaken
      if (!prev_done) {
        ok = bar_wait(bar_o, (uint32_t)((j - 1) & 1), abort_flag, 0xB21u);
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      }
    }
    if (ok) {
      ok = bar_wait(bar_o, (uint32_t)((n_kt - 1) & 1), abort_flag, 0xB30u);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      fence_after();
      const float inv = l > 0.f ? 1.0f / l : 0.f;
      uint4* dst = reinterpret_cast<uint4*>(p.out + (seq0 + qi) * p.ldo + h * HD);
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        float t[32];
        ld32(t_o + 32u * half, t);
        if (qi < p.S) {
#pragma unroll
          for (int c = 0; c < 4; ++c)
            dst[4 * half + c] = make_uint4(pack2(t[8 * c] * inv, t[8 * c + 1] * inv), pack2(t[8 * c + 2] * inv, t[8 * c + 3] * inv),
                                           pack2(t[8 * c + 4] * inv, t[8 * c + 5] * inv), pack2(t[8 * c + 6] * inv, t[8 * c + 7] * inv));
        }
      }
      if (qi < p.S) p.lse[((long long)b * p.H + h) * p.S + qi] = m + log2f(l);
    }
  }
  __syncwarp();
  fence_before();
  __syncthreads();
  if (warp == 4) {
    fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

// ---- backward, dQ: one CTA per 128 queries of a head, sweeping the key tiles up to the diagonal ---------------
//   S_j = Q K_j^T, dP_j = dO V_j^T     two MMAs into 64 + 64 columns of tensor memory
//   dS_j = P_j (dP_j - delta) / sqrt(d), P_j = 2^(c S_j - lse)     one query row per thread, written as BF16
//                                                                   pairs into 32 columns of tensor memory, the
//                                                                   third product's A operand
//   dQ += dS_j K_j                       third MMA, accumulating in 64 more columns over the whole sweep (K_j read
//                                        as it lies in memory: keys as contraction rows, d contiguous)
// The dQ product of tile j - 1 is issued after the score products of tile j, so it runs while the rows work on
// tile j; K / V tiles come through three TMA stages.  Only the final dQ leaves tensor memory.
constexpr int DQ_OFF_DO = Q_BYTES, DQ_OFF_KV = 2 * Q_BYTES, DQ_STAGE = 2 * KV_BYTES, DQ_STAGES = 3;
constexpr int DQ_OFF_CTL = DQ_OFF_KV + DQ_STAGES * DQ_STAGE;
constexpr int DQ_SMEM = DQ_OFF_CTL + CTL + 1024;
// The backward kernels have no reduction along a row, so two threads share a row (32 of the 64 columns each:
// warps w and w + 4 read the same tensor-memory lanes): eight row warps, the ninth issues copies and MMAs.
constexpr int BWD_THREADS = 288, ROW_THREADS = 256;

struct TcBwdParams {
  const float* lse; const float* dsum;
  __nv_bfloat16* dq; __nv_bfloat16* dk; __nv_bfloat16* dv;
  long long ldq, ldk;
  int B, S, H, Hkv;
  float scale_log2, inv_sqrt_d;
};

__global__ void __launch_bounds__(BWD_THREADS, 2)
attn_dq64_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmDO,
                    const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const TcBwdParams p) {
  extern __shared__ uint8_t raw[];
  const uint32_t base = (s32(raw) + 1023u) & ~1023u;
  uint8_t* smem = raw + (base - s32(raw));
  const uint32_t ctl = base + DQ_OFF_CTL;
  const uint32_t bar_qd = ctl, bar_s = ctl + 40, bar_sfree = ctl + 48, bar_ds = ctl + 56, bar_done = ctl + 64;
  auto kvfull = [&](int s) { return ctl + 8u + 8u * s; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + DQ_OFF_CTL + 96);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + DQ_OFF_CTL + 100);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // one-dimensional grid, query tile slowest and descending: CTAs start in order of decreasing work
  const int hb = p.H * p.B;
  const int qt = (int)(gridDim.x / hb) - 1 - (int)(blockIdx.x / hb);
  const int h = (blockIdx.x % hb) % p.H, b = (blockIdx.x % hb) / p.H;
  const int g = h / (p.H / p.Hkv);
  const long long seq0 = (long long)b * p.S;
  const int q0 = qt * QT;
  const int last_q = min(q0 + QT, p.S) - 1;
  const int n_kt = last_q / KT + 1;

  if (threadIdx.x == 0) {
    bar_init(bar_qd, 1);
    for (int s = 0; s < DQ_STAGES; ++s) bar_init(kvfull(s), 1);
    bar_init(bar_s, 1); bar_init(bar_done, 1);
    bar_init(bar_sfree, ROW_THREADS); bar_init(bar_ds, ROW_THREADS);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(const_cast<uint32_t*>(tmem_slot))),
                 "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;                         // S: columns 0..63, dP: 64..127, dQ: 128..191, dS (BF16 pairs): 192..223
  const uint32_t sQ = base, sDO = base + DQ_OFF_DO;
  auto sK = [&](int s) { return base + DQ_OFF_KV + (uint32_t)s * DQ_STAGE; };
  auto sV = [&](int s) { return sK(s) + KV_BYTES; };

  if (warp == 8) {
    if (lane == 0) {
      auto load_kv = [&](int j) {
        const int st = j % DQ_STAGES;
        bar_expect(kvfull(st), 2 * KV_BYTES);
        tma_2d(sK(st), &tmK, g * HD, (int)(seq0 + (long long)j * KT), kvfull(st));
        tma_2d(sV(st), &tmV, g * HD, (int)(seq0 + (long long)j * KT), kvfull(st));
      };
      bar_expect(bar_qd, 2 * Q_BYTES);
      tma_2d(sQ, &tmQ, h * HD, (int)(seq0 + q0), bar_qd);
      tma_2d(sDO, &tmDO, h * HD, (int)(seq0 + q0), bar_qd);
      load_kv(0);
      if (n_kt > 1) load_kv(1);
      bool ok = bar_wait(bar_qd, 0u, abort_flag, 0xC01u);
      const uint32_t id_k = idesc(0), id_n = idesc(1);
      auto issue_dq = [&](int j) {                            // dQ += dS_j K_j
        const uint64_t db = desc_n_major(sK(j % DQ_STAGES));
#pragma unroll
        for (int k = 0; k < KT / 16; ++k) mma_ts(tmem + 128u, tmem + 192u + 8u * k, db + 128u * k, id_n, (j | k) != 0 ? 1u : 0u);
        commit(bar_done);
      };
      for (int j = 0; j < n_kt && ok; ++j) {
        const int st = j % DQ_STAGES;
        if (j >= 1 && j + 1 < n_kt) {                         // stage of tile j + 1 last held tile j - 2
          if (j >= 2) ok = bar_wait(bar_done, (uint32_t)((j - 2) & 1), abort_flag, 0xC10u);
          if (!ok) break;
          load_kv(j + 1);
        }
        ok = bar_wait(kvfull(st), (uint32_t)((j / DQ_STAGES) & 1), abort_flag, 0xC20u | st);
        if (ok && j > 0) ok = bar_wait(bar_sfree, (uint32_t)((j - 1) & 1), abort_flag, 0xC30u);
        if (!ok) break;
        fence_after();
        {
          const uint64_t dq_ = desc_k_major(sQ), dk_ = desc_k_major(sK(st)), dd = desc_k_major(sDO), dv_ = desc_k_major(sV(st));
#pragma unroll
          for (int k = 0; k < HD / 16; ++k) mma(tmem, dq_ + 2u * k, dk_ + 2u * k, id_k, k != 0 ? 1u : 0u);
#pragma unroll
          for (int k = 0; k < HD / 16; ++k) mma(tmem + 64u, dd + 2u * k, dv_ + 2u * k, id_k, k != 0 ? 1u : 0u);
        }
        commit(bar_s);
        if (j > 0) {
          ok = bar_wait(bar_ds, (uint32_t)((j - 1) & 1), abort_flag, 0xC40u);
          if (!ok) break;
          fence_after();
          issue_dq(j - 1);
        }
      }
      if (ok) ok = bar_wait(bar_ds, (uint32_t)((n_kt - 1) & 1), abort_flag, 0xC50u);
      if (ok) { fence_after(); issue_dq(n_kt - 1); }
      if (!ok) { const unsigned long long t0 = now_ns(); while (now_ns() - t0 < 2000000ull) {} }
    }
  } else {
    const int row = 32 * (warp & 3) + lane, half = warp >> 2;    // this thread: columns 32 half .. 32 half + 31 of its row
    const int qi = q0 + row;
    const uint32_t t_lane = tmem + ((uint32_t)(32 * (warp & 3)) << 16);
    const long long ro = ((long long)b * p.H + h) * p.S;
    const float lse = qi < p.S ? p.lse[ro + qi] : 0.f;
    const float nd = qi < p.S ? -p.dsum[ro + qi] * p.inv_sqrt_d : 0.f;
    bool ok = true;
    for (int j = 0; j < n_kt; ++j) {
      const int k0 = j * KT;
      ok = bar_wait(bar_s, (uint32_t)(j & 1), abort_flag, 0xD10u);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      fence_after();
      float s[32];
      auto tile = [&](auto diag_tag) {                        // P (dP - delta) / sqrt(d); the mask only where needed
        constexpr bool DIAG = decltype(diag_tag)::value;
        float t[32], d[32];
        ld32x2(t_lane + 32u * half, t_lane + 64u + 32u * half, t, d);
        const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nl2 = make_float2(-lse, -lse);
        const float2 is2 = make_float2(p.inv_sqrt_d, p.inv_sqrt_d), nd2 = make_float2(nd, nd);
#pragma unroll
        for (int i = 0; i < 32; i += 2) {                        // two elements per multiply-add
          const float2 x = __ffma2_rn(make_float2(t[i], t[i + 1]), sc2, nl2);
          float2 pr = make_float2(ex2(x.x), ex2(x.y));
          if (DIAG) {                                            // above the diagonal (and beyond the sequence end)
            if (k0 + 32 * half + i > qi) pr.x = 0.f;
            if (k0 + 32 * half + i + 1 > qi) pr.y = 0.f;
          }
          const float2 r = __fmul2_rn(pr, __ffma2_rn(make_float2(d[i], d[i + 1]), is2, nd2));
          s[i] = r.x; s[i + 1] = r.y;
        }
      };
      if (k0 + KT - 1 > q0) tile(std::true_type{}); else tile(std::false_type{});   // some key of the tile above some row
      fence_before();
      bar_arrive(bar_sfree);
      if (j > 0) {                                            // the dS buffer is free once dQ of tile j - 1 has run
        ok = bar_wait(bar_done, (uint32_t)((j - 1) & 1), abort_flag, 0xD20u);
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      }
      uint32_t pk[16];
#pragma unroll
      for (int w = 0; w < 16; ++w) pk[w] = pack2(s[2 * w], s[2 * w + 1]);
      st16(t_lane + 192u + 16u * half, pk);                   // this thread's half of the row of dS_j: an A operand
      wait_st();
      fence_before();
      bar_arrive(bar_ds);
    }
    if (ok) {
      ok = bar_wait(bar_done, (uint32_t)((n_kt - 1) & 1), abort_flag, 0xD30u);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      fence_after();
      uint4* dst = reinterpret_cast<uint4*>(p.dq + (seq0 + qi) * p.ldq + h * HD);
      {
        float t[32];
        ld32(t_lane + 128u + 32u * half, t);
        if (qi < p.S) {
#pragma unroll
          for (int c = 0; c < 4; ++c)
            dst[4 * half + c] = make_uint4(pack2(t[8 * c], t[8 * c + 1]), pack2(t[8 * c + 2], t[8 * c + 3]),
                                           pack2(t[8 * c + 4], t[8 * c + 5]), pack2(t[8 * c + 6], t[8 * c + 7]));
        }
      }
    }
  }
  __syncwarp();
  fence_before();
  __syncthreads();
  if (warp == 8) {
    fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

// ---- backward, dK and dV: one CTA per 128 keys of a key / value head ------------------------------------------
// The keys are the rows (tensor-memory lanes); the CTA sweeps the (head, 64-query tile) pairs that see them:
//   S^T = K Q_i^T, dP^T = V dO_i^T          two MMAs into 64 + 64 columns of tensor memory
//   P^T = 2^(c S^T - lse_q), dS^T = P^T (dP^T - delta_q) / sqrt(d)    one key row per thread; both written as BF16
//                                            pairs over the columns the thread has just read (its half of S^T, of
//                                            dP^T), from where they are the A operands of the accumulating products
//   dV += P^T dO_i, dK += dS^T Q_i           two MMAs that accumulate in 64 + 64 columns over the whole sweep
//                                            (dO_i and Q_i read as they lie in memory: queries as contraction rows)
// 256 columns of tensor memory and under 100 KB of shared memory: two CTAs per SM, which overlap each other's serial
// chain (score products -> rows -> accumulating products -> next item's score products, which overwrite P^T / dS^T
// and so wait for the accumulating products).  Q / dO tiles come through four TMA stages (requested three items
// ahead), lse and delta of a tile's 64 queries are staged in shared memory by the row threads themselves.  Queries
// beyond the sequence end are masked (their rows hold the next sequence's data).
constexpr int KV_OFF_V = Q_BYTES, KV_OFF_QD = 2 * Q_BYTES, KV_STAGE = 2 * KV_BYTES, KV_STAGES = 4;
constexpr int KV_OFF_ROWV = KV_OFF_QD + KV_STAGES * KV_STAGE, KV_OFF_CTL = KV_OFF_ROWV + 2 * 2 * KT * 4;
constexpr int KV_SMEM = KV_OFF_CTL + CTL + 1024;
static_assert(2 * KV_SMEM <= 227 * 1024, "two CTAs per SM");
// S^T: columns 0..63, dP^T: 64..127, dV: 128..191, dK: 192..255.  The thread of row half h reads columns 32 h .. 32 h + 31
// of S^T (dP^T) and writes its 32 values of P^T (dS^T) as 16 BF16 pairs to columns 32 h .. 32 h + 15 of the same buffer.
constexpr int KV_TMEM = 256;

__global__ void __launch_bounds__(BWD_THREADS, 2)
attn_dkv64_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmDO,
                     const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const TcBwdParams p) {
  extern __shared__ uint8_t raw[];
  const uint32_t base = (s32(raw) + 1023u) & ~1023u;
  uint8_t* smem = raw + (base - s32(raw));
  const uint32_t ctl = base + KV_OFF_CTL;
  const uint32_t bar_kv = ctl;
  auto qfull = [&](int s) { return ctl + 8u + 8u * s; };          // 4
  auto bar_s = [&](int s) { return ctl + 40u + 8u * s; };         // 2 (items alternate): the score products of an item are complete
  auto bar_pds = [&](int s) { return ctl + 72u + 8u * s; };       // 2: P^T / dS^T of an item written by all rows
  auto bar_done = [&](int s) { return ctl + 88u + 8u * s; };      // 2: the accumulating MMAs of an item have run
  auto bar_rv = [&](int s) { return ctl + 112u + 8u * s; };       // 2: lse / delta of an item staged, previous use read by all
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + KV_OFF_CTL + 128);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + KV_OFF_CTL + 132);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // one-dimensional grid, key tile slowest: CTAs start in order of decreasing work (the first key tiles see the
  // most queries), so the short ones fill the end of the launch
  const int groups = p.Hkv * p.B;
  const int kt = blockIdx.x / groups, g = (blockIdx.x % groups) % p.Hkv, b = (blockIdx.x % groups) / p.Hkv;
  const int rep = p.H / p.Hkv;
  const long long seq0 = (long long)b * p.S;
  const int k0 = kt * QT;
  const int n_qt = (p.S + KT - 1) / KT;
  const int qt0 = k0 / KT;                                         // first query tile that sees a key of this tile
  const int per_head = n_qt - qt0;
  const int n_it = rep * per_head;

  if (threadIdx.x == 0) {
    bar_init(bar_kv, 1);
    for (int s = 0; s < KV_STAGES; ++s) bar_init(qfull(s), 1);
    for (int s = 0; s < 2; ++s) {
      bar_init(bar_s(s), 1); bar_init(bar_done(s), 1); bar_init(bar_pds(s), ROW_THREADS); bar_init(bar_rv(s), ROW_THREADS);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(const_cast<uint32_t*>(tmem_slot))),
                 "r"((uint32_t)KV_TMEM) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t sKt = base, sVt = base + KV_OFF_V;
  auto sQ = [&](int s) { return base + KV_OFF_QD + (uint32_t)s * KV_STAGE; };
  auto sDO = [&](int s) { return sQ(s) + KV_BYTES; };
  auto head_of = [&](int i) { return g * rep + i / per_head; };
  auto q0_of = [&](int i) { return (qt0 + i % per_head) * KT; };

  if (warp == 8) {
    if (lane == 0) {
      auto load_item = [&](int i) {
        const int st = i % KV_STAGES;
        bar_expect(qfull(st), 2 * KV_BYTES);
        tma_2d(sQ(st), &tmQ, head_of(i) * HD, (int)(seq0 + q0_of(i)), qfull(st));
        tma_2d(sDO(st), &tmDO, head_of(i) * HD, (int)(seq0 + q0_of(i)), qfull(st));
      };
      bar_expect(bar_kv, 2 * Q_BYTES);
      tma_2d(sKt, &tmK, g * HD, (int)(seq0 + k0), bar_kv);
      tma_2d(sVt, &tmV, g * HD, (int)(seq0 + k0), bar_kv);
      load_item(0);
      if (n_it > 1) load_item(1);
      if (n_it > 2) load_item(2);
      bool ok = bar_wait(bar_kv, 0u, abort_flag, 0xE01u);
      const uint32_t id_k = idesc(0), id_n = idesc(1);
      auto issue_s = [&](int i) {                              // S^T and dP^T of item i
        const int st = i % KV_STAGES;
        const uint64_t dk_ = desc_k_major(sKt), dq_ = desc_k_major(sQ(st)), dv_ = desc_k_major(sVt), dd = desc_k_major(sDO(st));
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) mma(tmem, dk_ + 2u * k, dq_ + 2u * k, id_k, k != 0 ? 1u : 0u);
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) mma(tmem + 64u, dv_ + 2u * k, dd + 2u * k, id_k, k != 0 ? 1u : 0u);
        commit(bar_s(i & 1));
      };
      if (ok) ok = bar_wait(qfull(0), 0u, abort_flag, 0xE10u);
      if (ok) { fence_after(); issue_s(0); }
      for (int i = 0; i < n_it && ok; ++i) {
        if (i + 3 < n_it) {                                    // its stage last held item i - 1: wait for that item's
          if (i >= 1) ok = bar_wait(bar_done((i - 1) & 1), (uint32_t)(((i - 1) >> 1) & 1), abort_flag, 0xE40u);   // MMAs
          if (!ok) break;
          load_item(i + 3);
        }
        ok = bar_wait(bar_pds(i & 1), (uint32_t)((i >> 1) & 1), abort_flag, 0xE30u);
        if (!ok) break;
        fence_after();
        {
          // A operands from tensor memory: contraction steps 0, 1 (queries 0..31) in columns 0..15 of the buffer,
          // steps 2, 3 (queries 32..63) in columns 32..47
          const int st = i % KV_STAGES;
          const uint64_t dd = desc_n_major(sDO(st)), dq_ = desc_n_major(sQ(st));
#pragma unroll
          for (int k = 0; k < KT / 16; ++k)
            mma_ts(tmem + 128u, tmem + (uint32_t)(32 * (k >> 1) + 8 * (k & 1)), dd + 128u * k, id_n, (i | k) != 0 ? 1u : 0u);
#pragma unroll
          for (int k = 0; k < KT / 16; ++k)
            mma_ts(tmem + 192u, tmem + 64u + (uint32_t)(32 * (k >> 1) + 8 * (k & 1)), dq_ + 128u * k, id_n, (i | k) != 0 ? 1u : 0u);
        }
        commit(bar_done(i & 1));
        if (i + 1 < n_it) {
          // the next item's score products overwrite P^T / dS^T: after the accumulating products have read them
          ok = bar_wait(qfull((i + 1) % KV_STAGES), (uint32_t)(((i + 1) / KV_STAGES) & 1), abort_flag, 0xE10u);
          if (ok) ok = bar_wait(bar_done(i & 1), (uint32_t)((i >> 1) & 1), abort_flag, 0xE20u);
          if (!ok) break;
          fence_after();
          issue_s(i + 1);
        }
      }
      if (!ok) { const unsigned long long t0 = now_ns(); while (now_ns() - t0 < 2000000ull) {} }
    }
  } else {
    const int row = 32 * (warp & 3) + lane, half = warp >> 2;    // this thread: queries 32 half .. 32 half + 31 of an item
    const int kj = k0 + row;
    const uint32_t t_lane = tmem + ((uint32_t)(32 * (warp & 3)) << 16);
    float* rowv_all = reinterpret_cast<float*>(smem + KV_OFF_ROWV);      // [2][2][KT]: lse, delta / sqrt(d) negated
    bool ok = true;
    // this thread's share of an item's 64 lse values (rows 0..63) or 64 negated, scaled delta values (rows 64..127);
    // the value for item i + 1 is requested at the start of item i, so its latency is off the per-item path
    auto row_value = [&](int i) {
      const long long ro = ((long long)b * p.H + head_of(i)) * p.S;
      const int q = q0_of(i) + (row & (KT - 1));
      if (q >= p.S) return 0.f;
      return row < KT ? p.lse[ro + q] : -p.dsum[ro + q] * p.inv_sqrt_d;
    };
    float rv_next = half == 0 ? row_value(0) : 0.f;
    for (int i = 0; i < n_it; ++i) {
      const int q0 = q0_of(i);
      float* rowv = rowv_all + (i & 1) * 2 * KT;
      if (half == 0) {                                           // the first four warps stage the 128 values
        rowv[row] = rv_next;
        if (i + 1 < n_it) rv_next = row_value(i + 1);
      }
      // every row thread arrives: the buffer of item i + 2 is then written only after all have read item i's
      bar_arrive(bar_rv(i & 1));
      ok = bar_wait(bar_rv(i & 1), (uint32_t)((i >> 1) & 1), abort_flag, 0xF05u);
      if (ok) ok = bar_wait(bar_s(i & 1), (uint32_t)((i >> 1) & 1), abort_flag, 0xF10u);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      fence_after();
      const bool edge = q0 < k0 + QT || q0 + KT > p.S;         // the item crosses the diagonal or the sequence end
      // the mask costs three instructions per element: only items that need it take that path
      auto item = [&](auto edge_tag) {
        constexpr bool EDGE = decltype(edge_tag)::value;
        float t[32], d[32];
        ld32x2(t_lane + 32u * half, t_lane + 64u + 32u * half, t, d);
#pragma unroll
        for (int j4 = 0; j4 < 32; j4 += 4) {
          const float4 l4 = *reinterpret_cast<const float4*>(rowv + 32 * half + j4);          // the same address in every lane
          const float4 n4 = *reinterpret_cast<const float4*>(rowv + KT + 32 * half + j4);
          const float lq[4] = {l4.x, l4.y, l4.z, l4.w}, nq[4] = {n4.x, n4.y, n4.z, n4.w};
#pragma unroll
          for (int e = 0; e < 4; e += 2) {                       // two elements per multiply-add
            const int j = j4 + e, c = 32 * half + j;
            const float2 x = __ffma2_rn(make_float2(t[j], t[j + 1]), make_float2(p.scale_log2, p.scale_log2),
                                        make_float2(-lq[e], -lq[e + 1]));
            float2 pr = make_float2(ex2(x.x), ex2(x.y));
            if (EDGE) {
              if (!(kj <= q0 + c && q0 + c < p.S)) pr.x = 0.f;
              if (!(kj <= q0 + c + 1 && q0 + c + 1 < p.S)) pr.y = 0.f;
            }
            const float2 r = __fmul2_rn(pr, __ffma2_rn(make_float2(d[j], d[j + 1]), make_float2(p.inv_sqrt_d, p.inv_sqrt_d),
                                                       make_float2(nq[e], nq[e + 1])));
            t[j] = pr.x; t[j + 1] = pr.y;
            d[j] = r.x; d[j + 1] = r.y;
          }
        }
        // this thread's half of the rows of P^T and dS^T: A operands in tensor memory
        uint32_t pk[16];
#pragma unroll
        for (int w = 0; w < 16; ++w) pk[w] = pack2(t[2 * w], t[2 * w + 1]);
        st16(t_lane + 32u * half, pk);                           // over the first half of the columns just read
#pragma unroll
        for (int w = 0; w < 16; ++w) pk[w] = pack2(d[2 * w], d[2 * w + 1]);
        st16(t_lane + 64u + 32u * half, pk);
      };
      if (edge) item(std::true_type{}); else item(std::false_type{});
      wait_st();
      fence_before();
      bar_arrive(bar_pds(i & 1));
    }
    if (ok) {
      ok = bar_wait(bar_done((n_it - 1) & 1), (uint32_t)(((n_it - 1) >> 1) & 1), abort_flag, 0xF30u);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      fence_after();
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        uint4* dst = reinterpret_cast<uint4*>((which ? p.dk : p.dv) + (seq0 + kj) * p.ldk + g * HD);
        {
          float t[32];
          ld32(t_lane + 128u + 64u * which + 32u * half, t);
          if (kj < p.S) {
#pragma unroll
            for (int c = 0; c < 4; ++c)
              dst[4 * half + c] = make_uint4(pack2(t[8 * c], t[8 * c + 1]), pack2(t[8 * c + 2], t[8 * c + 3]),
                                             pack2(t[8 * c + 4], t[8 * c + 5]), pack2(t[8 * c + 6], t[8 * c + 7]));
          }
        }
      }
    }
  }
  __syncwarp();
  fence_before();
  __syncthreads();
  if (warp == 8) {
    fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)KV_TMEM) : "memory");
  }
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [rows, cols] BF16, row stride ld elements: boxes of 64 columns x box_rows rows, 128-byte swizzle
int head_map(faar_ctx* ctx, CUtensorMap* map, const void* ptr, long long rows, int cols, long long ld, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)HD, (cuuint32_t)box_rows};
  cuuint32_t es[2] = {1, 1};
  CUresult r = reinterpret_cast<EncodeFn>(ctx->encode_tiled)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims,
                                                             strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : (int)cudaErrorInvalidValue;
}

}  // namespace

int faar_launch_attention_fwd64_tc(faar_ctx* ctx, int B, int S, int H, int Hkv, const void* q, int64_t ldq, const void* k,
                                   const void* v, int64_t ldk, void* out, int64_t ldo, float* lse, float scale_log2) {
  static_assert(2 * SMEM <= 227 * 1024, "two CTAs per SM");
  const long long T = (long long)B * S;
  if (T > 0x7FFFFFFFll) return (int)cudaErrorInvalidValue;
  CUtensorMap tmQ, tmK, tmV;
  int e = head_map(ctx, &tmQ, q, T, H * HD, ldq, QT);
  if (!e) e = head_map(ctx, &tmK, k, T, Hkv * HD, ldk, KT);
  if (!e) e = head_map(ctx, &tmV, v, T, Hkv * HD, ldk, KT);
  if (e) return e;
  cudaError_t ce = cudaFuncSetAttribute(attn_fwd64_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (ce != cudaSuccess) return (int)ce;
  TcParams p;
  p.out = reinterpret_cast<__nv_bfloat16*>(out); p.lse = lse; p.ldo = ldo; p.B = B; p.S = S; p.H = H; p.Hkv = Hkv;
  p.scale_log2 = scale_log2;
  attn_fwd64_tc_kernel<<<dim3(((S + QT - 1) / QT) * H * B, 1, 1), THREADS, SMEM, ctx->stream>>>(tmQ, tmK, tmV, p);
  return (int)cudaGetLastError();
}

int faar_launch_attention_dq64_tc(faar_ctx* ctx, int B, int S, int H, int Hkv, const void* q, int64_t ldq, const void* k,
                                  const void* v, int64_t ldk, const void* dout, int64_t ldo, const float* lse,
                                  const float* dsum, void* dq, float scale_log2) {
  static_assert(2 * (DQ_SMEM + 1024) <= 227 * 1024, "two CTAs per SM");
  const long long T = (long long)B * S;
  if (T > 0x7FFFFFFFll) return (int)cudaErrorInvalidValue;
  CUtensorMap tmQ, tmDO, tmK, tmV;
  int e = head_map(ctx, &tmQ, q, T, H * HD, ldq, QT);
  if (!e) e = head_map(ctx, &tmDO, dout, T, H * HD, ldo, QT);
  if (!e) e = head_map(ctx, &tmK, k, T, Hkv * HD, ldk, KT);
  if (!e) e = head_map(ctx, &tmV, v, T, Hkv * HD, ldk, KT);
  if (e) return e;
  cudaError_t ce = cudaFuncSetAttribute(attn_dq64_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DQ_SMEM);
  if (ce != cudaSuccess) return (int)ce;
  TcBwdParams p = {};
  p.lse = lse; p.dsum = dsum; p.dq = reinterpret_cast<__nv_bfloat16*>(dq); p.ldq = ldq; p.ldk = ldk;
  p.B = B; p.S = S; p.H = H; p.Hkv = Hkv; p.scale_log2 = scale_log2; p.inv_sqrt_d = scale_log2 / 1.4426950408889634f;
  attn_dq64_tc_kernel<<<dim3(((S + QT - 1) / QT) * H * B, 1, 1), BWD_THREADS, DQ_SMEM, ctx->stream>>>(tmQ, tmDO, tmK, tmV, p);
  return (int)cudaGetLastError();
}

int faar_launch_attention_dkv64_tc(faar_ctx* ctx, int B, int S, int H, int Hkv, const void* q, int64_t ldq, const void* k,
                                   const void* v, int64_t ldk, const void* dout, int64_t ldo, const float* lse,
                                   const float* dsum, void* dk, void* dv, float scale_log2) {
  static_assert(KV_SMEM <= 227 * 1024, "shared memory budget");
  const long long T = (long long)B * S;
  if (T > 0x7FFFFFFFll) return (int)cudaErrorInvalidValue;
  CUtensorMap tmQ, tmDO, tmK, tmV;
  int e = head_map(ctx, &tmQ, q, T, H * HD, ldq, KT);
  if (!e) e = head_map(ctx, &tmDO, dout, T, H * HD, ldo, KT);
  if (!e) e = head_map(ctx, &tmK, k, T, Hkv * HD, ldk, QT);
  if (!e) e = head_map(ctx, &tmV, v, T, Hkv * HD, ldk, QT);
  if (e) return e;
  cudaError_t ce = cudaFuncSetAttribute(attn_dkv64_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, KV_SMEM);
  if (ce != cudaSuccess) return (int)ce;
  TcBwdParams p = {};
  p.lse = lse; p.dsum = dsum; p.dk = reinterpret_cast<__nv_bfloat16*>(dk); p.dv = reinterpret_cast<__nv_bfloat16*>(dv);
  p.ldq = ldq; p.ldk = ldk; p.B = B; p.S = S; p.H = H; p.Hkv = Hkv; p.scale_log2 = scale_log2;
  p.inv_sqrt_d = scale_log2 / 1.4426950408889634f;
  attn_dkv64_tc_kernel<<<dim3(((S + QT - 1) / QT) * Hkv * B, 1, 1), BWD_THREADS, KV_SMEM, ctx->stream>>>(tmQ, tmDO, tmK, tmV, p);
  return (int)cudaGetLastError();
}

// Reads and clears the status word of this module (synchronous copy: call after the stream has been synchronised).
int faar_attention_tc_status(uint32_t* code_out) {
  uint32_t v = 0, zero = 0;
  cudaError_t e = cudaMemcpyFromSymbol(&v, g_attn_status, sizeof(v));
  if (e == cudaSuccess && v) e = cudaMemcpyToSymbol(g_attn_status, &zero, sizeof(zero));
  *code_out = v;
  return (int)e;
}
