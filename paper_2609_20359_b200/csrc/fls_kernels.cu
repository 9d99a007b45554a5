// sm_100a kernels of libfls.  All three are HBM streams: persistent grids of 256-thread CTAs walk
// 2048-element tiles; a thread owns 8 consecutive elements of a tile and moves them with 128-bit
// (bf16) and 256-bit (fp32) global accesses.  No shared-memory staging and no tensor cores: nothing
// here is a contraction, and each byte is touched once.
//
//   fls_reduce_kernel  : K gradient buffers -> mean gradient (fp32, shard order) + squared-norm partials;
//                    the last CTA to finish adds the partials in index order and writes the group's
//                    norm and clip coefficient (no floating-point atomics: the result does not depend
//                    on which CTA is last).
//   fls_adamw_kernel   : clip + AdamW on master/m/v in place + bf16 copy in unsharded order.
//   fls_fedavg_kernel  : weighted average of G copies written back to all G (+ bf16 copies).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "fls_kernels.h"

namespace fls {
namespace {

// ------------------------------------------------------------------------------------------------
// Global-memory accessors.  "stream": data touched once (evict-first, no L1 allocation).
// "keep": default policy, used for the reduced gradient that the next kernel reads back.
// ------------------------------------------------------------------------------------------------
struct alignas(32) F8 { float v[8]; };

#define FLS_O8(r) "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
__device__ __forceinline__ F8 ld8_stream(const float* p) {
  uint32_t u[8];
  asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];" : FLS_O8(u) : "l"(p));
  F8 r;
#pragma unroll
  for (int e = 0; e < 8; ++e) r.v[e] = __uint_as_float(u[e]);
  return r;
}
__device__ __forceinline__ F8 ld8_keep(const float* p) {
  uint32_t u[8];
  asm volatile("ld.global.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];" : FLS_O8(u) : "l"(p));
  F8 r;
#pragma unroll
  for (int e = 0; e < 8; ++e) r.v[e] = __uint_as_float(u[e]);
  return r;
}
#define FLS_U8(r) "r"(__float_as_uint(r.v[0])), "r"(__float_as_uint(r.v[1])), "r"(__float_as_uint(r.v[2])), "r"(__float_as_uint(r.v[3])), \
                  "r"(__float_as_uint(r.v[4])), "r"(__float_as_uint(r.v[5])), "r"(__float_as_uint(r.v[6])), "r"(__float_as_uint(r.v[7]))
__device__ __forceinline__ void st8_stream(float* p, const F8& r) {
  asm volatile("st.global.L1::no_allocate.L2::evict_first.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" :: "l"(p), FLS_U8(r) : "memory");
}
__device__ __forceinline__ void st8_keep(float* p, const F8& r) {
  asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" :: "l"(p), FLS_U8(r) : "memory");
}
__device__ __forceinline__ uint4 ld_b128_stream(const void* p) {
  uint4 r;
  // 128-bit accesses have no L2::evict_first form; .cs is the streaming (evict-first) cache operator
  asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}
__device__ __forceinline__ void st_b128_stream(void* p, const uint4& r) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w) : "memory");
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);   // round to nearest even
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint16_t to_bf16_bits(float x) {
  __nv_bfloat16 h = __float2bfloat16_rn(x);
  return *reinterpret_cast<uint16_t*>(&h);
}

// ------------------------------------------------------------------------------------------------
// Tile -> segment walk.  A CTA visits tiles in monotone order, so it only ever steps to a
// neighbouring segment; the current segment lives in registers.
// ------------------------------------------------------------------------------------------------
struct Walker {
  const Segment* segs;
  uint32_t i;
  Segment cur;
  __device__ __forceinline__ void init(const Segment* s, uint32_t n_seg, bool descending) {
    segs = s;
    i = descending ? n_seg - 1 : 0;
    cur = segs[i];
  }
  __device__ __forceinline__ void seek(uint64_t tile) {
    while (tile >= cur.tile_end) cur = segs[++i];
    while (tile < cur.tile_begin) cur = segs[--i];
  }
};

// Per-thread slice of a tile: n = number of valid elements (0..8), vec = whole 8 on the vector path.
struct Slice { uint64_t j, a; uint32_t n; bool vec; };
__device__ __forceinline__ Slice slice_of(const Segment& s, uint64_t tile) {
  Slice r;
  const uint64_t e0 = (tile - s.tile_begin) * kTile + threadIdx.x * kVec;
  const uint64_t rem = e0 < s.len ? s.len - e0 : 0;
  r.n = rem < kVec ? uint32_t(rem) : kVec;
  r.vec = s.aligned && r.n == kVec;
  r.j = s.j0 + e0;
  r.a = s.a0 + e0;
  return r;
}

// Fixed-shape block sum of one double per thread (shuffle tree inside a warp, then warp 0 over the
// per-warp results): same order every run.  Result valid in thread 0.
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

// ------------------------------------------------------------------------------------------------
// K1: gradient reduction in the paper's order + squared norm.
// ------------------------------------------------------------------------------------------------
template <int N, bool F32> struct Raw;
template <> struct Raw<8, false> { uint4 r; };
template <> struct Raw<8, true> { F8 r; };
template <> struct Raw<1, false> { uint16_t r; };
template <> struct Raw<1, true> { float r; };

__device__ __forceinline__ void load_raw(Raw<8, false>& x, const void* base, uint64_t j) {
  x.r = ld_b128_stream(static_cast<const uint16_t*>(base) + j);
}
__device__ __forceinline__ void load_raw(Raw<8, true>& x, const void* base, uint64_t j) {
  x.r = ld8_stream(static_cast<const float*>(base) + j);
}
__device__ __forceinline__ void load_raw(Raw<1, false>& x, const void* base, uint64_t j) {
  x.r = static_cast<const uint16_t*>(base)[j];
}
__device__ __forceinline__ void load_raw(Raw<1, true>& x, const void* base, uint64_t j) {
  x.r = static_cast<const float*>(base)[j];
}
__device__ __forceinline__ void unpack(const Raw<8, false>& x, float (&f)[8]) {
  f[0] = bf16_lo(x.r.x); f[1] = bf16_hi(x.r.x); f[2] = bf16_lo(x.r.y); f[3] = bf16_hi(x.r.y);
  f[4] = bf16_lo(x.r.z); f[5] = bf16_hi(x.r.z); f[6] = bf16_lo(x.r.w); f[7] = bf16_hi(x.r.w);
}
__device__ __forceinline__ void unpack(const Raw<8, true>& x, float (&f)[8]) {
#pragma unroll
  for (int e = 0; e < 8; ++e) f[e] = x.r.v[e];
}
__device__ __forceinline__ void unpack(const Raw<1, false>& x, float (&f)[1]) { f[0] = __uint_as_float(uint32_t(x.r) << 16); }
__device__ __forceinline__ void unpack(const Raw<1, true>& x, float (&f)[1]) { f[0] = x.r; }

// Mean of the K buffers at elements j .. j+N-1.  Buffers are consumed in ascending index k = rho*S +
// sigma, eight loads in flight at a time.  `inner` is the running sum of the current sharding group
// (the reduce-scatter level); when the group's last buffer has been added it is folded into `outer`
// (the all-reduce level across replicas).  Both start at zero, so every level is a plain ascending
// sum (0 + x is exact).  SG fixes the level structure at compile time so the hot loop holds only
// unpack + add:
//   SG =  0 : every batch of 8 lies inside one sharding group (FSDP, or S a multiple of 8); bit i of
//             fold_mask says that batch i closes a group.
//   SG = 1, 2, 4 : S == SG, a batch holds 8/SG whole groups.
//   SG = -1 : any other shape; bit k of end_mask says that buffer k closes a group.
template <int N, bool F32, int SG>
__device__ __forceinline__ void reduce_elems(const ReduceArgs& a, uint64_t j, float (&mean)[N]) {
  float inner[N], outer[N];
#pragma unroll
  for (int e = 0; e < N; ++e) inner[e] = outer[e] = 0.f;
  for (uint32_t k0 = 0; k0 < a.K; k0 += 8) {
    Raw<N, F32> raw[8];
#pragma unroll
    for (int b = 0; b < 8; ++b)
      if (k0 + b < a.K) load_raw(raw[b], a.grad[k0 + b], j);
    if constexpr (SG == 0) {
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        if (k0 + b < a.K) {
          float x[N];
          unpack(raw[b], x);
#pragma unroll
          for (int e = 0; e < N; ++e) inner[e] += x[e];
        }
      }
      if ((a.fold_mask >> (k0 >> 3)) & 1u) {
#pragma unroll
        for (int e = 0; e < N; ++e) { outer[e] += inner[e]; inner[e] = 0.f; }
      }
    } else if constexpr (SG > 0) {
#pragma unroll
      for (int g0 = 0; g0 < 8; g0 += SG) {
        if (k0 + g0 < a.K) {
          float s[N];
          unpack(raw[g0], s);
#pragma unroll
          for (int i = 1; i < SG; ++i) {
            float x[N];
            unpack(raw[g0 + i], x);
#pragma unroll
            for (int e = 0; e < N; ++e) s[e] += x[e];
          }
#pragma unroll
          for (int e = 0; e < N; ++e) outer[e] += s[e];
        }
      }
    } else {
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        const uint32_t k = k0 + b;
        if (k < a.K) {
          float x[N];
          unpack(raw[b], x);
#pragma unroll
          for (int e = 0; e < N; ++e) inner[e] += x[e];
          if ((a.end_mask >> k) & 1ull) {
#pragma unroll
            for (int e = 0; e < N; ++e) { outer[e] += inner[e]; inner[e] = 0.f; }
          }
        }
      }
    }
  }
  // one scaling by 1/K after the last level: a multiply when 1/K is exact, else an IEEE division
  if (a.k_is_pow2) {
#pragma unroll
    for (int e = 0; e < N; ++e) mean[e] = outer[e] * a.inv_k;
  } else {
#pragma unroll
    for (int e = 0; e < N; ++e) mean[e] = __fdiv_rn(outer[e], a.k_float);
  }
}

template <bool F32, int SG>
__global__ void __launch_bounds__(kThreads, 2) fls_reduce_kernel(const __grid_constant__ ReduceArgs a) {
  __shared__ double sh[kThreads / 32];
  __shared__ bool is_last;
  double dsum = 0.0;
  if (blockIdx.x < a.n_tiles) {
    Walker w;
    w.init(a.segs, a.n_seg, a.descending);
    for (uint64_t lin = blockIdx.x; lin < a.n_tiles; lin += gridDim.x) {
      const uint64_t tile = a.descending ? a.n_tiles - 1 - lin : lin;
      w.seek(tile);
      const Slice s = slice_of(w.cur, tile);
      if (s.vec) {
        float g[8];
        reduce_elems<8, F32, SG>(a, s.j, g);
        F8 o;
        float sq = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) { o.v[e] = g[e]; sq = fmaf(g[e], g[e], sq); }
        st8_keep(a.gbar + s.a, o);
        dsum += double(sq);
      } else {
        for (uint32_t e = 0; e < s.n; ++e) {
          float g[1];
          reduce_elems<1, F32, -1>(a, s.j + e, g);
          a.gbar[s.a + e] = g[0];
          dsum += double(g[0] * g[0]);
        }
      }
    }
  }
  // CTA partial -> workspace; the CTA that takes the last ticket adds all partials in index order.
  double total = block_sum(dsum, sh);
  if (threadIdx.x == 0) {
    a.partials[blockIdx.x] = total;
    __threadfence();
    const uint32_t ticket = atomicAdd(a.ticket, 1u);
    is_last = (ticket == gridDim.x - 1);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  double s = 0.0;
  for (uint32_t i = threadIdx.x; i < gridDim.x; i += kThreads) s += __ldcg(a.partials + i);
  total = block_sum(s, sh);
  if (threadIdx.x == 0) {
    const double nrm = sqrt(total);
    double c = 1.0;
    if (a.max_grad_norm > 0.0) {
      c = a.max_grad_norm / (nrm + 1e-6);
      if (c >= 1.0) c = 1.0;            // NaN compares false and stays NaN: non-finite norms propagate
    }
    *a.normsq_out = total;
    *a.norm_out = float(nrm);
    *a.coef_out = float(c);
    if (!isfinite(nrm)) atomicOr(a.status, uint32_t(FLS_STATUS_NONFINITE_NORM));
    *a.ticket = 0u;                      // ready for the next launch (stream order)
  }
}

// ------------------------------------------------------------------------------------------------
// K2: clip + AdamW + bf16 copy.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void adamw_one(const AdamArgs& a, float c, float gbar, float& th, float& m, float& v) {
  const float g = c * gbar;
  th = th * a.decay;                                        // decoupled weight decay: theta (1 - lr wd)
  m = fmaf(a.beta1, m, a.omb1 * g);
  v = fmaf(a.beta2, v, a.omb2 * (g * g));
  const float denom = fmaf(sqrtf(v), a.inv_sqrt_bc2, a.eps);  // sqrt(v / (1 - beta2^t)) + eps
  th = fmaf(-a.step_size, __fdiv_rn(m, denom), th);         // step_size = lr / (1 - beta1^t)
}

__global__ void __launch_bounds__(kThreads, 3) fls_adamw_kernel(const __grid_constant__ AdamArgs a) {
  if (blockIdx.x >= a.n_tiles) return;
  const float c = __ldcg(a.coef);
  Walker w;
  w.init(a.segs, a.n_seg, a.descending);
  for (uint64_t lin = blockIdx.x; lin < a.n_tiles; lin += gridDim.x) {
    const uint64_t tile = a.descending ? a.n_tiles - 1 - lin : lin;
    w.seek(tile);
    const Slice s = slice_of(w.cur, tile);
    if (s.vec) {
      const F8 g = ld8_keep(a.gbar + s.a);
      F8 th = ld8_stream(a.theta + s.a);
      F8 m = ld8_stream(a.m + s.a);
      F8 v = ld8_stream(a.v + s.a);
#pragma unroll
      for (int e = 0; e < 8; ++e) adamw_one(a, c, g.v[e], th.v[e], m.v[e], v.v[e]);
      st8_stream(a.theta + s.a, th);
      st8_stream(a.m + s.a, m);
      st8_stream(a.v + s.a, v);
      uint4 p;
      p.x = pack_bf16x2(th.v[0], th.v[1]); p.y = pack_bf16x2(th.v[2], th.v[3]);
      p.z = pack_bf16x2(th.v[4], th.v[5]); p.w = pack_bf16x2(th.v[6], th.v[7]);
      st_b128_stream(a.pbf16 + s.j, p);
    } else {
      for (uint32_t e = 0; e < s.n; ++e) {
        float th = a.theta[s.a + e], m = a.m[s.a + e], v = a.v[s.a + e];
        adamw_one(a, c, a.gbar[s.a + e], th, m, v);
        a.theta[s.a + e] = th; a.m[s.a + e] = m; a.v[s.a + e] = v;
        a.pbf16[s.j + e] = to_bf16_bits(th);
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// K3: FedAvg.  x_bar = sum_g w_g x_g, ascending g, written to all G copies.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 2) fls_fedavg_kernel(const __grid_constant__ FedavgArgs a) {
  if (blockIdx.x >= a.n_tiles) return;
  Walker w;
  w.init(a.segs, a.n_seg, a.descending);
  for (uint64_t lin = blockIdx.x; lin < a.n_tiles; lin += gridDim.x) {
    const uint64_t tile = a.descending ? a.n_tiles - 1 - lin : lin;
    w.seek(tile);
    const Slice s = slice_of(w.cur, tile);
    if (s.vec) {
      F8 acc;
#pragma unroll
      for (int e = 0; e < 8; ++e) acc.v[e] = 0.f;
      for (uint32_t g0 = 0; g0 < a.G; g0 += 8) {
        F8 raw[8];
#pragma unroll
        for (int b = 0; b < 8; ++b)
          if (g0 + b < a.G) raw[b] = ld8_stream(a.x[g0 + b] + s.a);
#pragma unroll
        for (int b = 0; b < 8; ++b) {
          const uint32_t g = g0 + b;
          if (g < a.G) {
            const float wg = a.w[g];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc.v[e] = fmaf(wg, raw[b].v[e], acc.v[e]);   // acc starts at 0: the first term is w_0 x_0
          }
        }
      }
      for (uint32_t g = 0; g < a.G; ++g) st8_stream(a.x[g] + s.a, acc);
      if (a.write_bf16) {
        uint4 p;
        p.x = pack_bf16x2(acc.v[0], acc.v[1]); p.y = pack_bf16x2(acc.v[2], acc.v[3]);
        p.z = pack_bf16x2(acc.v[4], acc.v[5]); p.w = pack_bf16x2(acc.v[6], acc.v[7]);
        for (uint32_t g = 0; g < a.G; ++g) st_b128_stream(a.pbf16[g] + s.j, p);
      }
    } else {
      for (uint32_t e = 0; e < s.n; ++e) {
        float acc = 0.f;
        for (uint32_t g = 0; g < a.G; ++g) {
          const float x = a.x[g][s.a + e];
          acc = fmaf(a.w[g], x, acc);
        }
        for (uint32_t g = 0; g < a.G; ++g) a.x[g][s.a + e] = acc;
        if (a.write_bf16) {
          const uint16_t b = to_bf16_bits(acc);
          for (uint32_t g = 0; g < a.G; ++g) a.pbf16[g][s.j + e] = b;
        }
      }
    }
  }
}

}  // namespace

template <bool F32>
static void launch_reduce_t(const ReduceArgs& a, int sg, unsigned grid, cudaStream_t st) {
  switch (sg) {
    case 0: fls_reduce_kernel<F32, 0><<<grid, kThreads, 0, st>>>(a); break;
    case 1: fls_reduce_kernel<F32, 1><<<grid, kThreads, 0, st>>>(a); break;
    case 2: fls_reduce_kernel<F32, 2><<<grid, kThreads, 0, st>>>(a); break;
    case 4: fls_reduce_kernel<F32, 4><<<grid, kThreads, 0, st>>>(a); break;
    default: fls_reduce_kernel<F32, -1><<<grid, kThreads, 0, st>>>(a); break;
  }
}

cudaError_t launch_reduce(const ReduceArgs& a, bool f32, int sg, unsigned grid, cudaStream_t st) {
  if (f32)
    launch_reduce_t<true>(a, sg, grid, st);
  else
    launch_reduce_t<false>(a, sg, grid, st);
  return cudaGetLastError();
}

cudaError_t launch_adamw(const AdamArgs& a, unsigned grid, cudaStream_t st) {
  fls_adamw_kernel<<<grid, kThreads, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_fedavg(const FedavgArgs& a, unsigned grid, cudaStream_t st) {
  fls_fedavg_kernel<<<grid, kThreads, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace fls
