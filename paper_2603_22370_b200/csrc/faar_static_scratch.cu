// faar_round_loss_static: the Round Loss for callers that must not allocate.
//
// faar_round_loss takes its scratch (the per-block partial sums) from a workspace
// that the caller allocated.  Some callers cannot provide one: code that runs
// inside a region where device allocation is forbidden or would synchronise the
// device (a tight serving loop, a library hooked into somebody else's memory
// pool, a plugin that is handed raw pointers and nothing else).  For them the
// partial sums live in the file-scope device array below, which every GPU that
// loads the library holds until the process exits.
//
// One partial per 4096 consecutive elements of V, so the summation order -- and
// the result, bit for bit -- does not depend on the SM count of the device.
#include <mutex>

#include "faar_internal.cuh"

namespace {

constexpr int SL_THREADS = 256;
constexpr int SL_ELEMS_PER_BLOCK = 4096;                  // 256 threads x 4 float4
constexpr int SL_MAX_PARTIALS = 65536;                    // 256 KB of scratch per device
constexpr int64_t SL_MAX_N = (int64_t)SL_MAX_PARTIALS * SL_ELEMS_PER_BLOCK;   // 268 435 456 weights
constexpr int SL_MAX_DEVICES = 64;

// The scratch itself.  In host code this name is only a handle for
// cudaGetSymbolAddress: it is NOT a device address and must never be passed to a
// kernel directly.
static __device__ __align__(256) float g_round_partials[SL_MAX_PARTIALS];

// Device address of g_round_partials per device ordinal, resolved on first use.
float* g_partials_addr[SL_MAX_DEVICES] = {};
std::mutex g_addr_mutex;

// Block b sums 1 - (2v-1)^2 over elements [4096 b, 4096 (b+1)) in a fixed order.
__global__ void __launch_bounds__(SL_THREADS)
round_chunks_kernel(const float* __restrict__ V, int64_t N, float* __restrict__ partials) {
  const int64_t base = (int64_t)blockIdx.x * SL_ELEMS_PER_BLOCK;
  float acc = 0.f;
#pragma unroll
  for (int it = 0; it < SL_ELEMS_PER_BLOCK / (4 * SL_THREADS); ++it) {
    const int64_t e = base + ((int64_t)it * SL_THREADS + threadIdx.x) * 4;
    if (e + 4 <= N) {
      const float4 a = *reinterpret_cast<const float4*>(V + e);
      const float t0 = fmaf(2.f, a.x, -1.f), t1 = fmaf(2.f, a.y, -1.f);
      const float t2 = fmaf(2.f, a.z, -1.f), t3 = fmaf(2.f, a.w, -1.f);
      acc += (fmaf(-t0, t0, 1.f) + fmaf(-t1, t1, 1.f)) + (fmaf(-t2, t2, 1.f) + fmaf(-t3, t3, 1.f));
    } else {
      for (int64_t i = e; i < N; ++i) {
        const float t = fmaf(2.f, V[i], -1.f);
        acc += fmaf(-t, t, 1.f);
      }
    }
  }
  acc = faar_warp_sum(acc);
  __shared__ float s_sum[SL_THREADS / 32];
  if ((threadIdx.x & 31) == 0) s_sum[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int i = 0; i < SL_THREADS / 32; ++i) t += s_sum[i];
    partials[blockIdx.x] = t;
  }
}

// One block: the n partials in double, fixed order, times 1/N.
__global__ void __launch_bounds__(SL_THREADS)
round_total_kernel(const float* __restrict__ partials, int n, double inv_n, float* __restrict__ out) {
  __shared__ double sh[SL_THREADS];
  double acc = 0.0;
  for (int i = threadIdx.x; i < n; i += SL_THREADS) acc += (double)partials[i];
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int s = SL_THREADS / 2; s > 0; s >>= 1) {
    if (threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = (float)(sh[0] * inv_n);
}

struct CurrentDevice {
  int prev = -1;
  bool ok = true;
  explicit CurrentDevice(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; prev = -1; return; }
    if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess; else prev = -1;
  }
  ~CurrentDevice() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" int faar_round_loss_static(faar_ctx* ctx, const float* V, int64_t N, float* loss_round) {
  if (!ctx || !V || !loss_round) return FAAR_ERR_INVALID_ARG;
  if (N <= 0 || N > SL_MAX_N) return FAAR_ERR_SHAPE;          // beyond the fixed scratch: refuse, launch nothing
  if (reinterpret_cast<uintptr_t>(V) & 15u) return FAAR_ERR_ALIGN;
  if (ctx->device < 0 || ctx->device >= SL_MAX_DEVICES) return FAAR_ERR_INVALID_ARG;
  CurrentDevice cur(ctx->device);
  if (!cur.ok) { ctx->last_cuda_error = (int)cudaErrorInvalidDevice; return FAAR_ERR_CUDA; }

  float* partials;
  {
    // Set-up, once per device, with that device current: ask the runtime where this
    // device's copy of the array lives.
    std::lock_guard<std::mutex> lock(g_addr_mutex);
    if (!g_partials_addr[ctx->device]) {
      void* p = nullptr;
      cudaError_t e = cudaGetSymbolAddress(&p, g_round_partials);
      if (e != cudaSuccess || !p) { ctx->last_cuda_error = (int)e; return FAAR_ERR_CUDA; }
      g_partials_addr[ctx->device] = static_cast<float*>(p);
    }
    partials = g_partials_addr[ctx->device];
  }

  const int grid = (int)((N + SL_ELEMS_PER_BLOCK - 1) / SL_ELEMS_PER_BLOCK);
  // (not bracketed by the per-kernel timing events: creating an event is an allocation too)
  round_chunks_kernel<<<grid, SL_THREADS, 0, ctx->stream>>>(V, N, partials);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) {
    round_total_kernel<<<1, SL_THREADS, 0, ctx->stream>>>(partials, grid, 1.0 / (double)N, loss_round);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return FAAR_ERR_CUDA; }
  return FAAR_OK;
}

extern "C" int64_t faar_round_loss_static_max_n(void) { return SL_MAX_N; }
