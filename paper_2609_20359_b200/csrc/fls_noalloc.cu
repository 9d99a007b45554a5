// fls_reduce_norm_noalloc: the gradient reduction + global norm for callers that cannot allocate.
//
// Some users of this library are not allowed to call cudaMalloc at all: a plug-in inside a host
// application whose own pool already owns the whole device, a service that forbids allocation after
// start-up, or a latency-critical loop that cannot afford the device-wide synchronisation an allocation
// may cause.  The plan-based path needs a caller-provided workspace for its norm partials and ticket
// counter; this entry point needs none.  Its scratch lives in the file-scope __device__ array below,
// which every GPU that loads the library holds (about 256 KiB) until the process exits.
//
// The array is shared by all calls and keeps whatever the previous call left in it.  The only part that
// must start at zero, the ticket counter, is cleared on the caller's stream before every launch; the
// partials are fully rewritten before they are read.  Two calls that overlap on the GPU (different
// streams, or different host threads on the same device) race on the array: serialise them.
#include <type_traits>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <mutex>

#include "fls.h"
#include "fls_internal.h"

namespace {

constexpr int kThreads = 256;
constexpr int kVec = 8;
constexpr int kTile = kThreads * kVec;                        // 2048 elements
constexpr uint32_t kChunkTiles = 8;
constexpr uint64_t kChunkElems = uint64_t(kTile) * kChunkTiles;  // 16384 elements per norm partial
constexpr uint32_t kMaxChunks = FLS_NOALLOC_MAX_ELEMS / kChunkElems;
static_assert(uint64_t(kMaxChunks) * kChunkElems == FLS_NOALLOC_MAX_ELEMS, "maximum must be whole chunks");

struct Scratch {
  double partial[kMaxChunks];   // squared-norm partial of each 16384-element chunk
  unsigned int ticket;          // CTAs finished so far; must be zero when a launch starts
  unsigned int pad[63];
};

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(Scratch)];

struct Args {
  const void* grad[FLS_MAX_GRAD_BUFFERS];
  float* gbar;
  float* norm_coef;      // [0] = norm, [1] = clip coefficient
  Scratch* scratch;
  uint64_t n;
  uint32_t n_chunks;
  uint32_t K;
  uint64_t end_mask;     // bit k: buffer k closes a sharding group
  float k_float, inv_k;
  uint32_t k_is_pow2;
  double max_grad_norm;
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

template <bool F32>
__device__ __forceinline__ void load8(const void* base, uint64_t j, float (&x)[8]) {
  if constexpr (F32) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(static_cast<const float*>(base) + j));
    const float4 b = __ldcs(reinterpret_cast<const float4*>(static_cast<const float*>(base) + j + 4));
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  } else {
    const uint4 r = __ldcs(reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(base) + j));
    x[0] = bf16_lo(r.x); x[1] = bf16_hi(r.x); x[2] = bf16_lo(r.y); x[3] = bf16_hi(r.y);
    x[4] = bf16_lo(r.z); x[5] = bf16_hi(r.z); x[6] = bf16_lo(r.w); x[7] = bf16_hi(r.w);
  }
}
template <bool F32>
__device__ __forceinline__ float load1(const void* base, uint64_t j) {
  if constexpr (F32) return static_cast<const float*>(base)[j];
  return __uint_as_float(uint32_t(static_cast<const uint16_t*>(base)[j]) << 16);
}

// Same order and precision as the plan-based kernel: ascending buffers inside a sharding group, groups folded in
// ascending replica order, both levels starting from zero, one scaling by 1/K at the end.  bf16 gradients are added
// in fp32 (exact unless the addends span more than 16 binades); fp32 gradients are added in double and rounded to
// fp32 once, so that a mean that nearly cancels keeps its leading bits.
template <bool F32, int N>
__device__ __forceinline__ void mean_of(const Args& a, uint64_t j, float (&mean)[N]) {
  using A = typename std::conditional<F32, double, float>::type;
  A inner[N], outer[N];
#pragma unroll
  for (int e = 0; e < N; ++e) inner[e] = outer[e] = A(0);
  for (uint32_t k = 0; k < a.K; ++k) {
    float x[N];
    if constexpr (N == 8) load8<F32>(a.grad[k], j, x); else x[0] = load1<F32>(a.grad[k], j);
#pragma unroll
    for (int e = 0; e < N; ++e) inner[e] += x[e];
    if ((a.end_mask >> k) & 1ull) {
#pragma unroll
      for (int e = 0; e < N; ++e) { outer[e] += inner[e]; inner[e] = A(0); }
    }
  }
#pragma unroll
  for (int e = 0; e < N; ++e) {
    if constexpr (F32) mean[e] = float(a.k_is_pow2 ? outer[e] * double(a.inv_k) : __ddiv_rn(outer[e], double(a.k_float)));
    else mean[e] = a.k_is_pow2 ? outer[e] * a.inv_k : __fdiv_rn(outer[e], a.k_float);
  }
}

__device__ __forceinline__ double block_sum(double x, double* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();
  if (lane == 0) sh[warp] = x;
  __syncthreads();
  double t = 0.0;
  if (warp == 0) {
    t = lane < kThreads / 32 ? sh[lane] : 0.0;
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
  }
  return t;
}

template <bool F32>
__global__ void __launch_bounds__(kThreads) fls_reduce_norm_noalloc_kernel(const __grid_constant__ Args a) {
  __shared__ double sh[kThreads / 32];
  __shared__ bool is_last;
  for (uint32_t c = blockIdx.x; c < a.n_chunks; c += gridDim.x) {
    double dsum = 0.0;
    for (uint32_t t = 0; t < kChunkTiles; ++t) {
      const uint64_t j = uint64_t(c) * kChunkElems + uint64_t(t) * kTile + threadIdx.x * kVec;
      if (j + kVec <= a.n) {
        float g[8];
        mean_of<F32, 8>(a, j, g);
        float sq = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) sq = fmaf(g[e], g[e], sq);
        *reinterpret_cast<float4*>(a.gbar + j) = make_float4(g[0], g[1], g[2], g[3]);
        *reinterpret_cast<float4*>(a.gbar + j + 4) = make_float4(g[4], g[5], g[6], g[7]);
        dsum += double(sq);
      } else {
        for (uint64_t i = j; i < a.n && i < j + kVec; ++i) {
          float g[1];
          mean_of<F32, 1>(a, i, g);
          a.gbar[i] = g[0];
          dsum += double(g[0] * g[0]);
        }
      }
    }
    const double total = block_sum(dsum, sh);
    if (threadIdx.x == 0) a.scratch->partial[c] = total;
  }
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned int ticket = atomicAdd(&a.scratch->ticket, 1u);
    is_last = (ticket == gridDim.x - 1);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  double s = 0.0;
  for (uint32_t i = threadIdx.x; i < a.n_chunks; i += kThreads) s += __ldcg(a.scratch->partial + i);
  const double total = block_sum(s, sh);
  if (threadIdx.x == 0) {
    const double nrm = sqrt(total);
    double c = 1.0;
    if (a.max_grad_norm > 0.0) {
      c = a.max_grad_norm / (nrm + 1e-6);
      if (c >= 1.0) c = 1.0;
    }
    a.norm_coef[0] = float(nrm);
    a.norm_coef[1] = float(c);
    a.scratch->ticket = 0u;
  }
}

constexpr int kMaxDevices = 64;
std::mutex g_mu;
Scratch* g_dev_scratch[kMaxDevices] = {};
int g_dev_sms[kMaxDevices] = {};
int fail(int code, const char* msg) {
  fls::set_last_error(msg);   // read back with fls_last_error()
  return code;
}

}  // namespace

extern "C" int fls_reduce_norm_noalloc(const void* const* grads, uint32_t shard_dim, uint32_t replicate_dim,
                                       uint32_t grad_dtype, uint64_t n_elems, double max_grad_norm, float* gbar_out,
                                       float* norm_coef_out, void* cuda_stream) {
  if (!grads || !gbar_out || !norm_coef_out) return fail(FLS_EPTR, "fls_reduce_norm_noalloc: null pointer");
  if (shard_dim == 0 || replicate_dim == 0) return fail(FLS_EINVAL, "fls_reduce_norm_noalloc: shard_dim and replicate_dim must be >= 1");
  const uint64_t K = uint64_t(shard_dim) * replicate_dim;
  if (K > FLS_MAX_GRAD_BUFFERS) return fail(FLS_EINVAL, "fls_reduce_norm_noalloc: more than 64 gradient buffers");
  if (grad_dtype != FLS_GRAD_BF16 && grad_dtype != FLS_GRAD_F32) return fail(FLS_EINVAL, "fls_reduce_norm_noalloc: unknown grad_dtype");
  if (n_elems == 0) return fail(FLS_EINVAL, "fls_reduce_norm_noalloc: n_elems must be >= 1");
  if (n_elems > FLS_NOALLOC_MAX_ELEMS) {
    char msg[200];
    snprintf(msg, sizeof msg, "fls_reduce_norm_noalloc: n_elems = %llu exceeds the static scratch capacity of %llu elements",
             (unsigned long long)n_elems, (unsigned long long)FLS_NOALLOC_MAX_ELEMS);
    return fail(FLS_ESIZE, msg);
  }
  if (std::isnan(max_grad_norm)) return fail(FLS_EINVAL, "fls_reduce_norm_noalloc: max_grad_norm is NaN");
  for (uint64_t k = 0; k < K; ++k) {
    if (!grads[k]) return fail(FLS_EPTR, "fls_reduce_norm_noalloc: null gradient buffer");
    if (reinterpret_cast<uintptr_t>(grads[k]) % FLS_BUFFER_ALIGN) return fail(FLS_EALIGN, "fls_reduce_norm_noalloc: gradient buffer not 32-byte aligned");
  }
  if (reinterpret_cast<uintptr_t>(gbar_out) % FLS_BUFFER_ALIGN) return fail(FLS_EALIGN, "fls_reduce_norm_noalloc: gbar_out not 32-byte aligned");
  if (reinterpret_cast<uintptr_t>(norm_coef_out) % 8) return fail(FLS_EALIGN, "fls_reduce_norm_noalloc: norm_coef_out not 8-byte aligned");

  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(FLS_ECUDA, cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return fail(FLS_ECUDA, "fls_reduce_norm_noalloc: device index out of range");
  Scratch* scratch = nullptr;
  int sms = 0;
  {
    // first call on this device: resolve the device address of the static array (the symbol itself is
    // not an address the GPU can use) and remember it
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_dev_scratch[dev]) {
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
      if (e != cudaSuccess || !p) return fail(FLS_ECUDA, e != cudaSuccess ? cudaGetErrorString(e) : "cudaGetSymbolAddress returned null");
      int n = 0;
      e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return fail(FLS_ECUDA, cudaGetErrorString(e));
      g_dev_sms[dev] = n;
      g_dev_scratch[dev] = static_cast<Scratch*>(p);
    }
    scratch = g_dev_scratch[dev];
    sms = g_dev_sms[dev];
  }

  Args a{};
  for (uint64_t k = 0; k < K; ++k) {
    a.grad[k] = grads[k];
    if (k % shard_dim == shard_dim - 1) a.end_mask |= 1ull << k;
  }
  a.gbar = gbar_out;
  a.norm_coef = norm_coef_out;
  a.scratch = scratch;
  a.n = n_elems;
  a.n_chunks = uint32_t((n_elems + kChunkElems - 1) / kChunkElems);
  a.K = uint32_t(K);
  a.k_float = float(K);
  a.inv_k = 1.0f / float(K);
  a.k_is_pow2 = (K & (K - 1)) == 0 ? 1u : 0u;
  a.max_grad_norm = max_grad_norm;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // the array keeps the previous call's contents: the ticket must start at zero
  e = cudaMemsetAsync(&scratch->ticket, 0, sizeof(unsigned int), st);
  if (e != cudaSuccess) return fail(FLS_ECUDA, cudaGetErrorString(e));
  const unsigned grid = unsigned(std::min<uint64_t>(a.n_chunks, uint64_t(sms) * 4));
  if (grad_dtype == FLS_GRAD_F32)
    fls_reduce_norm_noalloc_kernel<true><<<grid, kThreads, 0, st>>>(a);
  else
    fls_reduce_norm_noalloc_kernel<false><<<grid, kThreads, 0, st>>>(a);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(FLS_ECUDA, cudaGetErrorString(e));
  return FLS_OK;
}
