// sm_100a kernels of libfls.  All of them are HBM streams over 2048-element tiles; a group of 256
// threads owns a tile, a thread owns 8 consecutive elements of it and moves them with 128-bit (bf16)
// and 256-bit (fp32) global accesses.  By default the grid covers the whole buffer in one pass (no
// grid-stride loop): the hardware scheduler hands out CTAs in order, so the tiles in flight form a
// compact window that moves through memory and the SMs stay balanced, which measured 5-15 % faster
// than persistent grid-stride CTAs.  The kernels are kept small in registers (32-80) so that 768-2048
// threads are resident per SM; that, not unrolling, is what keeps enough loads in flight.
// No shared-memory staging and no tensor cores: nothing here is a contraction, and each byte is touched
// once.
//
//   fls_reduce_kernel       : K gradient buffers -> mean gradient (fp32, shard order) + squared-norm partials,
//                             added up over a fixed tree (warp, CTA, chunk of CTAs, grid) by whoever arrives
//                             last at each level; the last of all writes the group's norm and clip coefficient
//                             (no floating-point atomics, no block-wide barrier: the result does not depend on
//                             the order of arrival).  Also the norm-only pass of the recompute route, and, with
//                             the group in blockIdx.y, the reduction of all groups of a small plan at once.
//   fls_adamw_kernel        : clip + AdamW on master/m/v in place + bf16 copy in unsharded order
//                             (fls_adamw_batch_kernel: all groups of a small plan in one grid).
//   fls_reduce_adamw_kernel : AdamW that forms the mean gradient itself (recompute route; redo kernel of a
//                             speculative step).
//   fls_step_noclip_kernel  : reduce + norm + AdamW in one pass (plans without clipping; first kernel of a
//                             speculative step).
//   fls_fedavg_kernel       : weighted average of G copies written back to all copies (+ bf16 copies), optionally
//                             through an outer SGD step on a global copy.
//   fls_adamw_fedavg_kernel : AdamW of every group and FedAvg of the results in one pass (aggregation steps).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "fls_kernels.h"

namespace fls {
namespace {

// ------------------------------------------------------------------------------------------------
// Global-memory accessors.  "stream": data touched once, or for the last time (evict-first, no L1 allocation).
// "keep": stores of the part of the reduced gradient that the next kernel reads first.
// ------------------------------------------------------------------------------------------------
struct alignas(32) F8 { float v[8]; };

#define FLS_O8(r) "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
#define FLS_U8(r) "r"(__float_as_uint(r.v[0])), "r"(__float_as_uint(r.v[1])), "r"(__float_as_uint(r.v[2])), "r"(__float_as_uint(r.v[3])), \
                  "r"(__float_as_uint(r.v[4])), "r"(__float_as_uint(r.v[5])), "r"(__float_as_uint(r.v[6])), "r"(__float_as_uint(r.v[7]))
__device__ __forceinline__ F8 ld8_stream(const float* p) {
  uint32_t u[8];
  asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];" : FLS_O8(u) : "l"(p));
  F8 r;
#pragma unroll
  for (int e = 0; e < 8; ++e) r.v[e] = __uint_as_float(u[e]);
  return r;
}
__device__ __forceinline__ void st8_stream(float* p, const F8& r) {
  asm volatile("st.global.L1::no_allocate.L2::evict_first.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" :: "l"(p), FLS_U8(r) : "memory");
}
// the reduced gradient is the one stream that is read again (by the next kernel): its last part, which that
// kernel reads first, is stored with "evict last" so that it is still in L2 by then
__device__ __forceinline__ void st8_keep(float* p, const F8& r) {
  asm volatile("st.global.L2::evict_last.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" :: "l"(p), FLS_U8(r) : "memory");
}
// 128-bit accesses have no L2::evict_first form; .cs is the streaming (evict-first) cache operator
__device__ __forceinline__ uint4 ld_b128_stream(const void* p) {
  uint4 r;
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
__device__ __forceinline__ uint4 pack_bf16x8(const F8& x) {
  uint4 p;
  p.x = pack_bf16x2(x.v[0], x.v[1]); p.y = pack_bf16x2(x.v[2], x.v[3]);
  p.z = pack_bf16x2(x.v[4], x.v[5]); p.w = pack_bf16x2(x.v[6], x.v[7]);
  return p;
}
__device__ __forceinline__ uint16_t to_bf16_bits(float x) {
  __nv_bfloat16 h = __float2bfloat16_rn(x);
  return *reinterpret_cast<uint16_t*>(&h);
}

// ------------------------------------------------------------------------------------------------
// Programmatic dependent launch.  Inside one API call every kernel but the first is launched with
// programmatic stream serialization: its CTAs may start while the previous kernel's last CTAs are still
// running.  A kernel first issues the loads that its direct predecessor does not write, then waits
// (dep_wait) for that predecessor to have completed and flushed, and only then touches what the
// predecessor wrote or still reads.  A thread lets its successor go (dep_launch) only AFTER its own
// dep_wait: "the successor has started" then implies "my predecessor has completed", so at most two
// kernels of the chain ever overlap and the early loads can only race with the direct predecessor.  The
// first kernel of a call is launched normally and is therefore ordered after everything the caller
// enqueued before.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ------------------------------------------------------------------------------------------------
// Tile -> segment.  A segment is a run that is contiguous in both index orders.
// ------------------------------------------------------------------------------------------------
// Index of the segment that holds `tile`: bisection over the tile_end table, read from the kernel
// parameters when the table is small enough to travel there, else from global memory.
__device__ __forceinline__ uint32_t find_segment(const SegIndex& ix, uint32_t tile) {
  uint32_t lo = 0, hi = ix.n_seg - 1;
  if (ix.in_params) {
    while (lo < hi) {
      const uint32_t mid = (lo + hi) >> 1;
      if (ix.tile_end[mid] <= tile) lo = mid + 1; else hi = mid;
    }
  } else {
    while (lo < hi) {
      const uint32_t mid = (lo + hi) >> 1;
      if (__ldg(&ix.segs[mid].tile_end) <= uint64_t(tile)) lo = mid + 1; else hi = mid;
    }
  }
  return lo;
}

// Per-thread slice of a tile: n = number of valid elements (0..8), vec = whole 8 on the vector path.
// `lane` is the thread's index inside the 256-thread group that owns the tile.
struct Slice { uint64_t j, a, e; uint32_t n; bool vec; };   // e: position of the first element inside its segment
__device__ __forceinline__ Slice slice_of(const Segment* sg, uint32_t tile, uint32_t lane) {
  Slice r;
  const uint64_t e0 = (uint64_t(tile) - __ldg(&sg->tile_begin)) * kTile + lane * kVec;
  const uint64_t len = __ldg(&sg->len);
  const uint64_t rem = e0 < len ? len - e0 : 0;
  r.n = rem < kVec ? uint32_t(rem) : kVec;
  r.vec = __ldg(&sg->aligned) && r.n == kVec;
  r.j = __ldg(&sg->j0) + e0;
  r.a = __ldg(&sg->a0) + e0;
  r.e = e0;
  return r;
}

// Segment cursor of a CTA that visits several tiles in monotone order (persistent launch shapes).
struct Walker {
  const Segment* segs;
  uint32_t i;
  uint64_t begin, end;
  __device__ __forceinline__ void init(const SegIndex& ix, uint32_t tile) {
    segs = ix.segs;
    i = find_segment(ix, tile);
    begin = __ldg(&segs[i].tile_begin);
    end = __ldg(&segs[i].tile_end);
  }
  __device__ __forceinline__ const Segment* seek(uint32_t tile) {
    while (uint64_t(tile) >= end) { ++i; begin = end; end = __ldg(&segs[i].tile_end); }
    while (uint64_t(tile) < begin) { --i; end = begin; begin = __ldg(&segs[i].tile_begin); }
    return segs + i;
  }
};

// Sum over the lanes of a warp in a fixed (butterfly) order: every lane ends with the same bits.
__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
  return x;
}

// Release / acquire on one word in global memory (device scope): what was written before the store is visible to
// whoever sees the stored value with the load.
__device__ __forceinline__ void st_release(uint32_t* p, uint32_t v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
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
// sum (0 + x is exact).  KT and SG fix the shape at compile time so the hot path holds only
// load + unpack + add:
//   KT = K for K in {1, 2, 4, 8} (the buffer loop is unrolled and the pointers are read straight from
//        the kernel parameters), 0 for any other K (batches of 8 with a run-time bound);
//   SG =  0 : every batch of 8 lies inside one sharding group (FSDP, or S a multiple of 8); bit i of
//             fold_mask says that batch i closes a group.
//   SG = 1, 2, 4 : S == SG, a batch holds whole groups of SG buffers.
//   SG = -1 : any other shape; bit k of end_mask says that buffer k closes a group.
//   SG = -2 : as -1, with every partial sum and the final mean rounded to bf16 (the bf16-wire emulation).
// Ring order (SG < 0 only, a.ring set): the q-th buffer visited is not buffer q but the one a ring would add
// q-th.  For an element owned by rank s after the reduce-scatter and lying in sub-chunk c of the all-reduce
// across replicas (sc = s | c << 16), the shard level adds sigma = s+1, s+2, ..., s (mod S) inside each replica
// and the replicate level adds rho = c+1, ..., c (mod R): the owner's contribution comes last at both levels.
__device__ __forceinline__ float round_bf16(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

__device__ __forceinline__ uint32_t ring_buffer(const ReduceArgs& a, uint32_t sc, uint32_t q) {
  const uint32_t lvl = q / a.S, pos = q - lvl * a.S;
  uint32_t sigma = (sc & 0xFFFFu) + 1 + pos, rho = (sc >> 16) + 1 + lvl;
  if (sigma >= a.S) sigma -= a.S;
  if (rho >= a.R) rho -= a.R;
  return rho * a.S + sigma;
}

// Accumulator of the sums.  bf16 gradients are added in fp32: their 8-bit significands leave 16 spare bits, so
// the running sums are exact unless the addends span more than 16 binades.  fp32 gradients are added in double and
// rounded to fp32 once, after the scaling: an fp32 running sum of fp32 addends rounds at every step, by up to
// 2^-24 of the LARGEST addend, and where the addends cancel that error is large relative to the mean -- AdamW
// divides by sqrt(v)+eps, so a mean of 1e-9 that is off by 1e-10 moves theta by more than the parity tolerance.
template <bool F32> struct AccOf { using type = float; };
template <> struct AccOf<true> { using type = double; };

// one scaling by 1/K after the last level: a multiply when 1/K is exact, else an IEEE division
template <int N, typename A>
__device__ __forceinline__ void scale_mean(const ReduceArgs& a, const A (&outer)[N], float (&mean)[N]) {
  if (a.k_is_pow2) {
#pragma unroll
    for (int e = 0; e < N; ++e) mean[e] = float(outer[e] * A(a.inv_k));
  } else {
#pragma unroll
    for (int e = 0; e < N; ++e) {
      if constexpr (sizeof(A) == 8) mean[e] = float(__ddiv_rn(outer[e], double(a.k_float)));
      else mean[e] = __fdiv_rn(outer[e], a.k_float);
    }
  }
}

// Static K (KT = K in {1, 2, 4, 8}, SG in {0, 1, 2, 4}): the mean of KT values already loaded.
template <int N, bool F32, int KT, int SG>
__device__ __forceinline__ void combine_loaded(const ReduceArgs& a, const Raw<N, F32> (&raw)[KT], float (&mean)[N]) {
  static_assert(KT > 0 && SG >= 0, "static shapes only");
  using A = typename AccOf<F32 && (KT > 1)>::type;      // a single buffer is its own mean in any precision
  A outer[N];
#pragma unroll
  for (int e = 0; e < N; ++e) outer[e] = A(0);
  if constexpr (SG == 0) {
    A inner[N];
#pragma unroll
    for (int e = 0; e < N; ++e) inner[e] = A(0);
#pragma unroll
    for (int b = 0; b < KT; ++b) {
      float x[N];
      unpack(raw[b], x);
#pragma unroll
      for (int e = 0; e < N; ++e) inner[e] += x[e];
    }
#pragma unroll
    for (int e = 0; e < N; ++e) outer[e] += inner[e];
  } else {
#pragma unroll
    for (int g0 = 0; g0 < KT; g0 += SG) {
      A s[N];
      {
        float x[N];
        unpack(raw[g0], x);
#pragma unroll
        for (int e = 0; e < N; ++e) s[e] = x[e];
      }
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
  scale_mean<N, A>(a, outer, mean);
}

// gk0: index of the group's first buffer in a.grad (0 except in a batched launch).
template <int N, bool F32, int KT, int SG>
__device__ __forceinline__ void reduce_elems(const ReduceArgs& a, uint64_t j, float (&mean)[N], uint32_t sc = 0, uint32_t gk0 = 0) {
  if constexpr (KT > 0 && SG >= 0) {
    Raw<N, F32> raw[KT];
#pragma unroll
    for (int b = 0; b < KT; ++b) load_raw(raw[b], a.grad[gk0 + b], j);
    combine_loaded<N, F32, KT, SG>(a, raw, mean);
  } else {
    // run-time K: batches of 8 buffers
    using A = typename AccOf<F32>::type;
    const uint32_t K = a.K;
    A inner[N], outer[N];
#pragma unroll
    for (int e = 0; e < N; ++e) inner[e] = outer[e] = A(0);
#pragma unroll 1
    for (uint32_t k0 = 0; k0 < K; k0 += 8) {
      Raw<N, F32> raw[8];
      if (SG < 0 && a.ring) {
#pragma unroll
        for (int b = 0; b < 8; ++b)
          if (k0 + b < K) load_raw(raw[b], a.grad[gk0 + ring_buffer(a, sc, k0 + b)], j);
      } else {
#pragma unroll
        for (int b = 0; b < 8; ++b)
          if (k0 + b < K) load_raw(raw[b], a.grad[gk0 + k0 + b], j);
      }
      if constexpr (SG == 0) {
#pragma unroll
        for (int b = 0; b < 8; ++b) {
          if (k0 + b < K) {
            float x[N];
            unpack(raw[b], x);
#pragma unroll
            for (int e = 0; e < N; ++e) inner[e] += x[e];
          }
        }
        if ((a.fold_mask >> (k0 >> 3)) & 1u) {
#pragma unroll
          for (int e = 0; e < N; ++e) { outer[e] += inner[e]; inner[e] = A(0); }
        }
      } else if constexpr (SG > 0) {
#pragma unroll
        for (int g0 = 0; g0 < 8; g0 += SG) {
          if (k0 + g0 < K) {
            A s[N];
            {
              float x[N];
              unpack(raw[g0], x);
#pragma unroll
              for (int e = 0; e < N; ++e) s[e] = x[e];
            }
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
          if (k < K) {
            float x[N];
            unpack(raw[b], x);
#pragma unroll
            for (int e = 0; e < N; ++e) inner[e] = (SG == -2) ? A(round_bf16(float(inner[e] + x[e]))) : inner[e] + x[e];
            if ((a.end_mask >> k) & 1ull) {
#pragma unroll
              for (int e = 0; e < N; ++e) { outer[e] = (SG == -2) ? A(round_bf16(float(outer[e] + inner[e]))) : outer[e] + inner[e]; inner[e] = A(0); }
            }
          }
        }
      }
    }
    scale_mean<N, A>(a, outer, mean);
    if constexpr (SG == -2) {
#pragma unroll
      for (int e = 0; e < N; ++e) mean[e] = round_bf16(mean[e]);
    }
  }
}

// element-wise path of one thread's slice (unaligned runs and ragged tails); kept out of line so that
// it does not cost the vector path registers
// ring order (a.ring): seg is the slice's segment (it names the owning rank and the all-reduce sub-chunk length) and
// pos the position of the slice's first element inside it; otherwise both are ignored
template <bool F32, bool WIRE>
__device__ __noinline__ float reduce_slice_scalar(const ReduceArgs& a, uint64_t j, uint64_t addr, uint32_t n, const Segment* seg,
                                                  uint64_t pos, uint32_t gk0, float* gbar) {
  float sq = 0.f;
  uint32_t shard = 0;
  uint64_t sub_len = 1;
  if (a.ring) {
    shard = uint32_t(__ldg(&seg->shard));
    sub_len = __ldg(&seg->sub_len);
  }
  for (uint32_t e = 0; e < n; ++e) {
    float g[1];
    const uint32_t sc = a.ring ? (shard | uint32_t((pos + e) / sub_len) << 16) : 0u;
    reduce_elems<1, F32, 0, WIRE ? -2 : -1>(a, j + e, g, sc, gk0);
    if (a.store_gbar) gbar[addr + e] = g[0];
    sq = fmaf(g[0], g[0], sq);
  }
  return sq;
}

// End of every kernel that computes the norm.  The squared norm is added up over a fixed tree, so the result
// does not depend on the order in which warps or CTAs finish (no floating-point atomics), and without any
// block-wide barrier, so that a warp that is done never waits for the slowest warp of its CTA:
//   thread: fp32 sum of its 8 squares -> warp: butterfly in double -> CTA: the LAST WARP TO ARRIVE (a shared
//   counter) adds the warp sums in index order -> chunk of kNormChunk consecutive CTAs: the last CTA of the chunk
//   to arrive (one global counter per chunk) adds the chunk's CTA partials in index order -> grid: the last chunk
//   to arrive (the ticket) adds the chunk sums in index order, writes the group's norm and clip coefficient and
//   re-arms the ticket; every chunk counter is re-armed by the warp that closes the chunk.  A grid of at most
//   4 * kNormChunk CTAs forms a single chunk, whose closing warp finishes the job (one level less for small plans).
// The caller must have zeroed *arrived (shared) behind a __syncthreads() at the start of the kernel.
constexpr unsigned kNormChunk = kNormChunkCtas;

// Lane's share of an ordered sum: x[lane] + x[lane + 32] + x[lane + 64] + ... in that order.  Sixteen loads are
// issued before the first add (a plain loop would wait for each L2 round trip in turn: 16 of them for 512 partials,
// which is most of the run time of a kernel that lasts 10 us); entries past n count as +0, which changes nothing.
__device__ __noinline__ double lane_sum(const double* x, unsigned n, unsigned lane) {
  double c = 0.0;
  for (unsigned i0 = 0; i0 < n; i0 += 32 * 16) {
    double v[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const unsigned i = i0 + u * 32 + lane;
      v[u] = i < n ? __ldcg(x + i) : 0.0;
    }
#pragma unroll
    for (int u = 0; u < 16; ++u) c += v[u];
  }
  return c;
}

// y: the group of a batched launch (0 otherwise); it selects the group's own tree arrays, ticket and output slots.
template <int THREADS>
__device__ __forceinline__ void finish_norm(const ReduceArgs& a, float sq, unsigned* arrived, uint32_t y = 0) {
  constexpr int W = THREADS / 32;
  __shared__ double sh[W];
  const double x = warp_sum(double(sq));
  const unsigned lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  unsigned t = 0;
  if (lane == 0) {
    sh[warp] = x;
    __threadfence_block();
    t = atomicAdd(arrived, 1u);
  }
  if (__shfl_sync(0xFFFFFFFFu, t, 0) != W - 1) return;
  __threadfence_block();
  const double cta = warp_sum(lane < W ? sh[lane] : 0.0);
  // chunks of kNormChunk CTAs; a grid of up to 4 * kNormChunk CTAs is one chunk (one level less for small plans)
  const unsigned per_chunk = gridDim.x <= 4 * kNormChunk ? gridDim.x : kNormChunk;
  const unsigned chunk = blockIdx.x / per_chunk, n_chunks = (gridDim.x + per_chunk - 1) / per_chunk;
  const unsigned chunk_size = min(per_chunk, gridDim.x - chunk * per_chunk);
  double* const partials = a.partials + size_t(y) * gridDim.x;
  double* const chunk_partials = a.chunk_partials + size_t(y) * a.tree_stride;
  uint32_t* const chunk_count = a.chunk_count + size_t(y) * a.tree_stride;
  if (lane == 0) {
    partials[blockIdx.x] = cta;
    __threadfence();
    t = atomicAdd(chunk_count + chunk, 1u);
  }
  if (__shfl_sync(0xFFFFFFFFu, t, 0) != chunk_size - 1) return;
  __threadfence();
  double c = warp_sum(lane_sum(partials + size_t(chunk) * per_chunk, chunk_size, lane));
  if (lane == 0) chunk_count[chunk] = 0u;     // ready for the next launch (stream order)
  double total = c;
  if (n_chunks > 1) {                    // (a grid of one chunk is complete here: its sum is the total)
    if (lane == 0) {
      chunk_partials[chunk] = c;
      __threadfence();
      t = atomicAdd(a.ticket + y, 1u);
    }
    if (__shfl_sync(0xFFFFFFFFu, t, 0) != n_chunks - 1) return;
    __threadfence();
    total = warp_sum(lane_sum(chunk_partials, n_chunks, lane));
  }
  if (lane == 0) {
    const double nrm = sqrt(total);
    double c1 = 1.0;
    if (a.max_grad_norm > 0.0) {
      c1 = a.max_grad_norm / (nrm + 1e-6);
      if (c1 >= 1.0) c1 = 1.0;          // NaN compares false and stays NaN: non-finite norms propagate
    }
    a.normsq_out[y] = total;
    a.norm_out[y] = float(nrm);
    a.coef_out[y] = float(c1);
    if (!isfinite(nrm)) atomicOr(a.status, uint32_t(FLS_STATUS_NONFINITE_NORM));
    if (a.spec_counts) atomicAdd(a.spec_counts + (float(c1) == 1.0f ? 0 : 1), 1u);   // speculative step: kept / redone
    a.ticket[y] = 0u;                    // ready for the next launch (stream order)
    if (a.ready) st_release(a.ready + y, a.launch_id);   // resident step: the group's CTAs are waiting for this
  }
}

// Start of the same kernels: arm the CTA's arrival counter.
__device__ __forceinline__ void begin_norm(unsigned* arrived) {
  if (threadIdx.x == 0) *arrived = 0u;
  __syncthreads();
}

// One pass, no loop: a CTA of THREADS threads owns U * THREADS/256 consecutive tiles (each group of 256
// threads takes every (THREADS/256)-th of them, U in all) and the grid covers the whole buffer.  MINB resident
// CTAs per SM fix the register budget: 256 x 8 (32 registers) for the flat order with K = 4 or 8, 256 x 5 (48
// registers, what the kernel needs without spilling) for the two-level orders, which carry a second set of
// accumulators; 256 x 2 for a run-time K.
// Small CTAs turn over independently (no warp waits for the slowest of 32); they became the fastest shape once
// the norm epilogue lost its block-wide barriers.
// With K = 1 or 2 a thread would have only one or two 16-byte loads in flight, so those shapes take U > 1 tiles
// per thread (256 x 4 CTAs, 64 registers) and issue the loads of all of them before the first add.
template <bool F32, int KT, int SG>
__device__ __forceinline__ float reduce_one_tile(const ReduceArgs& a, uint32_t tile, uint32_t lane, uint32_t gk0, float* gbar) {
  float sq = 0.f;
  const Segment* seg = a.idx.segs + find_segment(a.idx, tile);
  const Slice s = slice_of(seg, tile, lane);
  bool vec = s.vec;
  uint32_t sc = 0;
  if (SG < 0 && a.ring) {
    // the eight elements of a vector access must share one all-reduce sub-chunk, else they go one by one
    const uint64_t sub_len = __ldg(&seg->sub_len);
    const uint64_t c0 = s.e / sub_len;
    vec = vec && (s.e + kVec - 1) / sub_len == c0;
    sc = uint32_t(__ldg(&seg->shard)) | uint32_t(c0) << 16;
  }
  if (vec) {
    float g[8];
    reduce_elems<8, F32, KT, SG>(a, s.j, g, sc, gk0);
    F8 o;
#pragma unroll
    for (int e = 0; e < 8; ++e) { o.v[e] = g[e]; sq = fmaf(g[e], g[e], sq); }
    if (a.store_gbar) {
      dep_wait();                        // the previous group's AdamW kernel may still be reading the scratch
      if (tile >= a.keep_from_tile) st8_keep(gbar + s.a, o); else st8_stream(gbar + s.a, o);
    }
  } else if (s.n) {
    dep_wait();
    sq = reduce_slice_scalar<F32, SG == -2>(a, s.j, s.a, s.n, seg, s.e, gk0, gbar);
  }
  return sq;
}

// BATCH: the grid's y dimension runs over the groups (see ReduceArgs); otherwise one group per launch.
template <bool F32, int KT, int SG, int THREADS, int MINB, int U, bool BATCH = false>
__global__ void __launch_bounds__(THREADS, MINB) fls_reduce_kernel(const __grid_constant__ ReduceArgs a) {
  constexpr uint32_t T = THREADS / kThreads;
  __shared__ unsigned arrived;
  begin_norm(&arrived);
  const uint32_t y = BATCH ? blockIdx.y : 0u;
  const uint32_t gk0 = BATCH ? y * uint32_t(KT) : 0u;
  float* const gbar = BATCH ? a.gbar + size_t(y) * a.gbar_stride : a.gbar;
  const uint32_t lane = threadIdx.x % kThreads;
  const uint32_t first = blockIdx.x * (T * U) + threadIdx.x / kThreads;   // this thread's tiles: first + u*T
  float sq = 0.f;
  if constexpr (U == 1) {
    if (first < a.idx.n_tiles) sq = reduce_one_tile<F32, KT, SG>(a, first, lane, gk0, gbar);
  } else {
    static_assert(KT > 0 && SG >= 0, "several tiles per thread only for a static K");
    // fast path: all U tiles lie in one aligned segment and are full, so their addresses are a stride apart
    const uint32_t last = first + (U - 1) * T;
    bool fast = false;
    uint64_t j0 = 0, a0 = 0;
    if (last < a.idx.n_tiles) {
      const Segment* sg = a.idx.segs + find_segment(a.idx, first);
      const uint64_t begin = __ldg(&sg->tile_begin);
      if (uint64_t(last) < __ldg(&sg->tile_end) && __ldg(&sg->aligned) &&
          (uint64_t(last) - begin + 1) * kTile <= __ldg(&sg->len)) {
        const uint64_t e0 = (uint64_t(first) - begin) * kTile + lane * kVec;
        j0 = __ldg(&sg->j0) + e0;
        a0 = __ldg(&sg->a0) + e0;
        fast = true;
      }
    }
    if (fast) {
      constexpr uint64_t stride = uint64_t(T) * kTile;
      Raw<8, F32> raw[U][KT];
#pragma unroll
      for (int u = 0; u < U; ++u)
#pragma unroll
        for (int b = 0; b < KT; ++b) load_raw(raw[u][b], a.grad[gk0 + b], j0 + u * stride);
      if (a.store_gbar) dep_wait();
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float g[8];
        combine_loaded<8, F32, KT, SG>(a, raw[u], g);
        F8 o;
        float s8 = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) { o.v[e] = g[e]; s8 = fmaf(g[e], g[e], s8); }
        sq += s8;
        if (a.store_gbar) {
          if (first + u * T >= a.keep_from_tile) st8_keep(gbar + a0 + u * stride, o); else st8_stream(gbar + a0 + u * stride, o);
        }
      }
    } else {
      for (int u = 0; u < U; ++u) {
        const uint32_t tile = first + u * T;
        if (tile < a.idx.n_tiles) sq += reduce_one_tile<F32, KT, SG>(a, tile, lane, gk0, gbar);
      }
    }
  }
  dep_wait();                            // partials, ticket and the norm slots belong to the predecessor until now
  dep_launch();
  finish_norm<THREADS>(a, sq, &arrived, y);
}

// ------------------------------------------------------------------------------------------------
// K2: clip + AdamW + bf16 copy.
// ------------------------------------------------------------------------------------------------
template <class A>
__device__ __forceinline__ void adamw_one(const A& a, float c, float gbar, float& th, float& m, float& v) {
  const float g = c * gbar;
  th = th * a.decay;                                        // decoupled weight decay: theta (1 - lr wd)
  m = fmaf(a.beta1, m, a.omb1 * g);
  v = fmaf(a.beta2, v, a.omb2 * (g * g));
  const float denom = fmaf(sqrtf(v), a.inv_sqrt_bc2, a.eps);  // sqrt(v / (1 - beta2^t)) + eps
  th = fmaf(-a.step_size, __fdiv_rn(m, denom), th);         // step_size = lr / (1 - beta1^t)
}

// Body of the AdamW kernel for one group's state; A is AdamArgs or AdamBatchArgs (layout, direction, scalars).
template <class A>
__device__ __forceinline__ void adamw_tiles(const A& a, float* theta, float* m_, float* v_, uint16_t* pbf16, const float* gbar,
                                            const float* coef) {
  const uint32_t n_tiles = a.idx.n_tiles;
  if (blockIdx.x >= n_tiles) { dep_wait(); dep_launch(); return; }
  float c = 0.f;
  bool waited = false;
  Walker w;
  w.init(a.idx, a.descending ? n_tiles - 1 - blockIdx.x : blockIdx.x);
  for (uint32_t lin = blockIdx.x; lin < n_tiles; lin += gridDim.x) {
    const uint32_t tile = a.descending ? n_tiles - 1 - lin : lin;
    const Slice s = slice_of(w.seek(tile), tile, threadIdx.x);
    if (s.vec) {
      // theta, m and v of this group are not touched by the reduce kernel: fetch them before waiting for it
      F8 th = ld8_stream(theta + s.a);
      F8 m = ld8_stream(m_ + s.a);
      F8 v = ld8_stream(v_ + s.a);
      if (!waited) { dep_wait(); dep_launch(); c = __ldcg(coef); waited = true; }
      const F8 g = ld8_stream(gbar + s.a);      // last use: evict-first also releases the lines K1 stored "evict last"
#pragma unroll
      for (int e = 0; e < 8; ++e) adamw_one(a, c, g.v[e], th.v[e], m.v[e], v.v[e]);
      st8_stream(theta + s.a, th);
      st8_stream(m_ + s.a, m);
      st8_stream(v_ + s.a, v);
      st_b128_stream(pbf16 + s.j, pack_bf16x8(th));
    } else if (s.n) {
      if (!waited) { dep_wait(); dep_launch(); c = __ldcg(coef); waited = true; }
      for (uint32_t e = 0; e < s.n; ++e) {
        float th = theta[s.a + e], m = m_[s.a + e], v = v_[s.a + e];
        adamw_one(a, c, gbar[s.a + e], th, m, v);
        theta[s.a + e] = th; m_[s.a + e] = m; v_[s.a + e] = v;
        pbf16[s.j + e] = to_bf16_bits(th);
      }
    }
  }
  if (!waited) { dep_wait(); dep_launch(); }
}

#ifndef FLS_ADAMW_MINB
#define FLS_ADAMW_MINB 3
#endif
#ifndef FLS_FUSED_MINB
#define FLS_FUSED_MINB 3
#endif
__global__ void __launch_bounds__(kThreads, FLS_ADAMW_MINB) fls_adamw_kernel(const __grid_constant__ AdamArgs a) {
  adamw_tiles(a, a.theta, a.m, a.v, a.pbf16, a.gbar, a.coef);
}

// The same for all groups in one grid (small plans, where one launch per group would be launch-bound).
__global__ void __launch_bounds__(kThreads, FLS_ADAMW_MINB) fls_adamw_batch_kernel(const __grid_constant__ AdamBatchArgs a) {
  const uint32_t y = blockIdx.y;
  adamw_tiles(a, a.theta[y], a.m[y], a.v[y], a.pbf16[y], a.gbar + size_t(y) * a.gbar_stride, a.coef + y);
}

// AdamW with the mean gradient formed in place (recompute plan).  With few gradient bytes per element
// (K * e_g < 8) reading the gradients a second time is cheaper than writing the fp32 mean and reading it
// back; reduce_elems is the same code the norm pass ran, so the gradient and the result are the same bits.
template <bool F32>
__device__ __noinline__ void reduce_adamw_slice_scalar(const ReduceAdamArgs& p, float c, uint64_t j, uint64_t addr, uint32_t n) {
  const AdamArgs& a = p.a;
  for (uint32_t e = 0; e < n; ++e) {
    float g[1];
    reduce_elems<1, F32, 0, -1>(p.r, j + e, g);
    float th = a.theta[addr + e], m = a.m[addr + e], v = a.v[addr + e];
    adamw_one(a, c, g[0], th, m, v);
    a.theta_out[addr + e] = th; a.m_out[addr + e] = m; a.v_out[addr + e] = v;
    a.pbf16[j + e] = to_bf16_bits(th);
  }
}

// skip_if_unclipped: this launch is the second kernel of a speculative step.  The first one applied AdamW with
// coefficient 1 while it computed the norm; if the coefficient turned out to be 1 its result stands and this
// kernel has nothing to do; otherwise it redoes the step with the real coefficient, reading the same (untouched)
// input state and overwriting the same output buffers.
template <bool F32, int KT, int SG>
__global__ void __launch_bounds__(kThreads, KT == 0 ? 2 : ((F32 && KT > 1) ? 3 : 4)) fls_reduce_adamw_kernel(const __grid_constant__ ReduceAdamArgs p) {
  const AdamArgs& a = p.a;
  const uint32_t n_tiles = a.idx.n_tiles;
  if (blockIdx.x >= n_tiles) { dep_wait(); dep_launch(); return; }
  float c = 0.f;
  bool waited = false;
  if (p.skip_if_unclipped) {
    dep_wait();
    dep_launch();
    c = __ldcg(a.coef);
    waited = true;
    if (c == 1.0f) return;
  }
  Walker w;
  w.init(a.idx, a.descending ? n_tiles - 1 - blockIdx.x : blockIdx.x);
  for (uint32_t lin = blockIdx.x; lin < n_tiles; lin += gridDim.x) {
    const uint32_t tile = a.descending ? n_tiles - 1 - lin : lin;
    const Slice s = slice_of(w.seek(tile), tile, threadIdx.x);
    if (s.vec) {
      // nothing read here is written by the norm pass: all loads can precede the wait for it
      F8 th = ld8_stream(a.theta + s.a);
      F8 m = ld8_stream(a.m + s.a);
      F8 v = ld8_stream(a.v + s.a);
      float g[8];
      reduce_elems<8, F32, KT, SG>(p.r, s.j, g);
      if (!waited) { dep_wait(); dep_launch(); c = __ldcg(a.coef); waited = true; }
#pragma unroll
      for (int e = 0; e < 8; ++e) adamw_one(a, c, g[e], th.v[e], m.v[e], v.v[e]);
      st8_stream(a.theta_out + s.a, th);
      st8_stream(a.m_out + s.a, m);
      st8_stream(a.v_out + s.a, v);
      st_b128_stream(a.pbf16 + s.j, pack_bf16x8(th));
    } else if (s.n) {
      if (!waited) { dep_wait(); dep_launch(); c = __ldcg(a.coef); waited = true; }
      reduce_adamw_slice_scalar<F32>(p, c, s.j, s.a, s.n);
    }
  }
  if (!waited) { dep_wait(); dep_launch(); }
}

// Whole step in one pass, for plans without clipping: the clip coefficient is 1 whatever the norm turns out
// to be, so AdamW does not have to wait for it.  Plans that clip use the same kernel as the first half of a
// speculative step: it writes the new state to the plan's second buffer set (theta_out, m_out, v_out) and the
// coefficient it computes at the end tells the follow-up kernel whether the guess "1" held.  One 256-thread CTA per tile forms the mean gradient, applies
// AdamW and contributes to the norm (still reported): K*e_g + 26 bytes per element instead of K*e_g + 34.
// theta, m and v come out bit-identical to the two-pass route (there the gradient is multiplied by exactly 1).
// (4 CTAs per SM measured best for a static K: 2 and 3 leave loads in flight on the table, 5 and 6 spill; the
// run-time-K form holds a batch of eight raw loads next to the state and needs the registers of 2 CTAs per SM)
template <bool F32, int KT, int SG>
__global__ void __launch_bounds__(kThreads, KT == 0 ? 2 : ((F32 && KT > 1) ? 3 : 4)) fls_step_noclip_kernel(const __grid_constant__ ReduceAdamArgs p) {
  const AdamArgs& a = p.a;
  __shared__ unsigned arrived;
  begin_norm(&arrived);
  float sq = 0.f;
  const uint32_t tile = blockIdx.x;        // the grid covers every tile exactly once
  const Slice s = slice_of(a.idx.segs + find_segment(a.idx, tile), tile, threadIdx.x);
  if (s.vec) {
    // nothing read here is written by the kernel before this one in the call (another group's step)
    F8 th = ld8_stream(a.theta + s.a);
    F8 m = ld8_stream(a.m + s.a);
    F8 v = ld8_stream(a.v + s.a);
    float g[8];
    reduce_elems<8, F32, KT, SG>(p.r, s.j, g);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      sq = fmaf(g[e], g[e], sq);
      adamw_one(a, 1.0f, g[e], th.v[e], m.v[e], v.v[e]);
    }
    dep_wait();
    st8_stream(a.theta_out + s.a, th);
    st8_stream(a.m_out + s.a, m);
    st8_stream(a.v_out + s.a, v);
    st_b128_stream(a.pbf16 + s.j, pack_bf16x8(th));
  } else if (s.n) {
    dep_wait();
    for (uint32_t e = 0; e < s.n; ++e) {
      float g[1];
      reduce_elems<1, F32, 0, -1>(p.r, s.j + e, g);
      sq = fmaf(g[0], g[0], sq);
      float th = a.theta[s.a + e], m = a.m[s.a + e], v = a.v[s.a + e];
      adamw_one(a, 1.0f, g[0], th, m, v);
      a.theta_out[s.a + e] = th; a.m_out[s.a + e] = m; a.v_out[s.a + e] = v;
      a.pbf16[s.j + e] = to_bf16_bits(th);
    }
  }
  dep_wait();
  dep_launch();
  finish_norm<kThreads>(p.r, sq, &arrived);
}

// Whole step of ALL groups in one kernel, for plans small enough that every CTA of the grid is resident at once
// (cooperative launch; group = blockIdx.y).  Phase 1: the CTA forms the mean gradient of its T tiles (x, x + gridDim.x,
// ...), keeps it in shared memory (thread-private slots, no barrier needed) and contributes to the group's norm.
// Then it fetches the state of its first tile and waits until the warp that completes the group's norm tree has
// published the clip coefficient (ready[y] == launch_id).  Phase 2: AdamW on the same tiles with the stashed mean
// gradient.  Per element K*e_g + 26 bytes, one launch per step instead of two per group.
// The wait is bounded: after wait_limit polls the CTA records FLS_STATUS_WAIT_EXPIRED and returns without
// touching the state (all CTAs are resident, so this happens only if the grid lost a CTA to an error).
// Mean gradient, AdamW arithmetic and the per-thread sums of squares are those of the other routes; the norm's
// tree groups T tiles per CTA instead of one, so in double it can differ from the two-pass route's in the last bits.
template <bool F32, int KT, int SG>
__global__ void __launch_bounds__(kThreads, (F32 && KT > 1) ? 3 : 4) fls_step_resident_kernel(const __grid_constant__ ResidentArgs p) {
  extern __shared__ float4 stash[];        // [T][2][kThreads]
  __shared__ unsigned arrived;
  __shared__ unsigned go;
  const ReduceArgs& a = p.r;
  const uint32_t y = blockIdx.y, gk0 = y * a.K, T = p.tiles_per_cta, n_tiles = a.idx.n_tiles;
  begin_norm(&arrived);
  float sq = 0.f;
  for (uint32_t i = 0; i < T; ++i) {
    const uint32_t tile = blockIdx.x + i * gridDim.x;
    if (tile >= n_tiles) break;
    const Slice s = slice_of(a.idx.segs + find_segment(a.idx, tile), tile, threadIdx.x);
    float g[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) g[e] = 0.f;
    if (s.vec) {
      reduce_elems<8, F32, KT, SG>(a, s.j, g, 0, gk0);
      float s8 = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) s8 = fmaf(g[e], g[e], s8);
      sq += s8;
    } else {
      for (uint32_t e = 0; e < s.n; ++e) {
        float t[1];
        reduce_elems<1, F32, 0, -1>(a, s.j + e, t, 0, gk0);
#pragma unroll
        for (int q = 0; q < 8; ++q) if (q == int(e)) g[q] = t[0];
        sq = fmaf(t[0], t[0], sq);
      }
    }
    stash[(i * 2 + 0) * kThreads + threadIdx.x] = make_float4(g[0], g[1], g[2], g[3]);
    stash[(i * 2 + 1) * kThreads + threadIdx.x] = make_float4(g[4], g[5], g[6], g[7]);
  }
  finish_norm<kThreads>(a, sq, &arrived, y);

  // state of the first tile: nothing of it depends on the norm, so the loads go out before the wait
  float* const theta = p.theta[y];
  float* const m_ = p.m[y];
  float* const v_ = p.v[y];
  uint16_t* const pbf16 = p.pbf16[y];
  Slice s0 = slice_of(a.idx.segs + find_segment(a.idx, blockIdx.x), blockIdx.x, threadIdx.x);   // blockIdx.x < n_tiles
  F8 th0, m0, v0;
  if (s0.vec) {
    th0 = ld8_stream(theta + s0.a);
    m0 = ld8_stream(m_ + s0.a);
    v0 = ld8_stream(v_ + s0.a);
  }
  if (threadIdx.x == 0) {
    unsigned ok = 1;
    uint32_t polls = 0;
    while (ld_acquire(a.ready + y) != p.expect_id) {
      if (++polls > p.wait_limit) { ok = 0; break; }
      __nanosleep(64);
    }
    if (!ok) atomicOr(a.status, uint32_t(FLS_STATUS_WAIT_EXPIRED));
    go = ok;
  }
  __syncthreads();
  if (!go) return;
  const float c = __ldcg(a.coef_out + y);
  // AdamW on tile i of this CTA with the stashed mean gradient; th, m, v: the thread's state if the slice is a vector
  auto apply = [&](uint32_t i, const Slice& s, F8& th, F8& m, F8& v) {
    const float4 ga = stash[(i * 2 + 0) * kThreads + threadIdx.x], gb = stash[(i * 2 + 1) * kThreads + threadIdx.x];
    const float g[8] = {ga.x, ga.y, ga.z, ga.w, gb.x, gb.y, gb.z, gb.w};
    if (s.vec) {
#pragma unroll
      for (int e = 0; e < 8; ++e) adamw_one(p, c, g[e], th.v[e], m.v[e], v.v[e]);
      st8_stream(theta + s.a, th);
      st8_stream(m_ + s.a, m);
      st8_stream(v_ + s.a, v);
      st_b128_stream(pbf16 + s.j, pack_bf16x8(th));
    } else {
      for (uint32_t e = 0; e < s.n; ++e) {
        float ge = 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q) if (q == int(e)) ge = g[q];
        float t1 = theta[s.a + e], m1 = m_[s.a + e], v1 = v_[s.a + e];
        adamw_one(p, c, ge, t1, m1, v1);
        theta[s.a + e] = t1; m_[s.a + e] = m1; v_[s.a + e] = v1;
        pbf16[s.j + e] = to_bf16_bits(t1);
      }
    }
  };
  apply(0, s0, th0, m0, v0);
  for (uint32_t i = 1; i < T; ++i) {
    const uint32_t tile = blockIdx.x + i * gridDim.x;
    if (tile >= n_tiles) break;
    const Slice s = slice_of(a.idx.segs + find_segment(a.idx, tile), tile, threadIdx.x);
    F8 th, m, v;
    if (s.vec) { th = ld8_stream(theta + s.a); m = ld8_stream(m_ + s.a); v = ld8_stream(v_ + s.a); }
    apply(i, s, th, m, v);
  }
}

// ------------------------------------------------------------------------------------------------
// K3: FedAvg.  x_bar = sum_g w_g x_g, ascending g from zero, written to all G copies.
// GT = G for G in {1, 2, 4, 8} (unrolled, pointers straight from the kernel parameters), else 0.
// ------------------------------------------------------------------------------------------------
// Outer optimizer on one element: xbar becomes the new global value.  delta = x_global - xbar,
// buf = momentum*buf + delta, d = delta + momentum*buf (Nesterov) or buf, x_global -= outer_lr*d.
__device__ __forceinline__ float outer_step(const FedavgArgs& a, float xbar, float xg, float& buf) {
  const float delta = xg - xbar;
  buf = fmaf(a.momentum, buf, delta);
  const float d = a.nesterov ? fmaf(a.momentum, buf, delta) : buf;
  return fmaf(-a.outer_lr, d, xg);
}

__device__ __noinline__ void fedavg_slice_scalar(const FedavgArgs& a, uint64_t j, uint64_t addr, uint32_t n) {
  for (uint32_t e = 0; e < n; ++e) {
    float acc = 0.f;
    for (uint32_t g = 0; g < a.G; ++g) acc = fmaf(a.w[g], a.x[g][addr + e], acc);
    if (a.x_global) {
      float b = a.outer_buf[addr + e];
      acc = outer_step(a, acc, a.x_global[addr + e], b);
      a.x_global[addr + e] = acc;
      a.outer_buf[addr + e] = b;
    }
    for (uint32_t g = 0; g < a.G; ++g) a.x[g][addr + e] = acc;
    for (uint32_t i = 0; i < a.n_extra; ++i) a.x_extra[i][addr + e] = acc;
    if (a.write_bf16) {
      const uint16_t b = to_bf16_bits(acc);
      for (uint32_t g = 0; g < a.G; ++g) a.pbf16[g][j + e] = b;
      for (uint32_t i = 0; i < a.n_extra; ++i) a.pbf16_extra[i][j + e] = b;
    }
  }
}

#ifndef FLS_FEDAVG_BATCH
#define FLS_FEDAVG_BATCH 8               // copies loaded before the first use (G = 8 and run-time G)
#define FLS_FEDAVG_BATCH_MINB 2
#endif
template <int GT, int MINB>
__global__ void __launch_bounds__(kThreads, MINB) fls_fedavg_kernel(const __grid_constant__ FedavgArgs a) {
  constexpr int B = (GT == 0 || GT > FLS_FEDAVG_BATCH) ? FLS_FEDAVG_BATCH : GT;
  const uint32_t G = GT ? uint32_t(GT) : a.G;
  const uint32_t n_tiles = a.idx.n_tiles;
  dep_wait();                            // the copies being averaged were just written by the predecessor
  dep_launch();
  if (blockIdx.x >= n_tiles) return;
  Walker w;
  w.init(a.idx, a.descending ? n_tiles - 1 - blockIdx.x : blockIdx.x);
  for (uint32_t lin = blockIdx.x; lin < n_tiles; lin += gridDim.x) {
    const uint32_t tile = a.descending ? n_tiles - 1 - lin : lin;
    const Slice s = slice_of(w.seek(tile), tile, threadIdx.x);
    if (s.vec) {
      F8 acc;
#pragma unroll
      for (int e = 0; e < 8; ++e) acc.v[e] = 0.f;
#pragma unroll 1
      for (uint32_t g0 = 0; g0 < G; g0 += B) {
        F8 raw[B];
#pragma unroll
        for (int b = 0; b < B; ++b)
          if (GT || g0 + b < G) raw[b] = ld8_stream(a.x[g0 + b] + s.a);
#pragma unroll
        for (int b = 0; b < B; ++b) {
          if (GT || g0 + b < G) {
            const float wg = a.w[g0 + b];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc.v[e] = fmaf(wg, raw[b].v[e], acc.v[e]);   // acc starts at 0: first term w_0 x_0
          }
        }
      }
      if (a.x_global) {
        const F8 xg = ld8_stream(a.x_global + s.a);
        F8 b = ld8_stream(a.outer_buf + s.a);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc.v[e] = outer_step(a, acc.v[e], xg.v[e], b.v[e]);
        st8_stream(a.x_global + s.a, acc);
        st8_stream(a.outer_buf + s.a, b);
      }
      if constexpr (GT != 0) {
#pragma unroll
        for (int g = 0; g < GT; ++g) st8_stream(a.x[g] + s.a, acc);
      } else {
        for (uint32_t g = 0; g < G; ++g) st8_stream(a.x[g] + s.a, acc);
      }
      // the broadcast inside each group: the other replicas' copies receive the same values
      for (uint32_t i = 0; i < a.n_extra; ++i) st8_stream(a.x_extra[i] + s.a, acc);
      if (a.write_bf16) {
        const uint4 p = pack_bf16x8(acc);
        if constexpr (GT != 0) {
#pragma unroll
          for (int g = 0; g < GT; ++g) st_b128_stream(a.pbf16[g] + s.j, p);
        } else {
          for (uint32_t g = 0; g < G; ++g) st_b128_stream(a.pbf16[g] + s.j, p);
        }
        for (uint32_t i = 0; i < a.n_extra; ++i) st_b128_stream(a.pbf16_extra[i] + s.j, p);
      }
    } else if (s.n) {
      fedavg_slice_scalar(a, s.j, s.a, s.n);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// K2+K3 fused for aggregation steps: AdamW on every group's element, then the weighted average of the G
// results, written to all G copies.  The arithmetic and its order are those of fls_adamw_kernel followed by
// fls_fedavg_kernel (each group's new theta is rounded to fp32 before it enters the fma chain), so the
// results are bit-identical to the two-kernel sequence; what is saved is FedAvg's own pass over the
// parameters.  m and v stay per group unless the plan averages the optimizer state.
// ------------------------------------------------------------------------------------------------
__device__ __noinline__ void fused_slice_scalar(const FusedArgs& a, uint64_t j, uint64_t addr, uint32_t n) {
  for (uint32_t e = 0; e < n; ++e) {
    float ath = 0.f, am = 0.f, av = 0.f;
    for (uint32_t g = 0; g < a.G; ++g) {
      float th = a.theta[g][addr + e], m = a.m[g][addr + e], v = a.v[g][addr + e];
      adamw_one(a, __ldcg(a.coefs + g), a.gbar[g][addr + e], th, m, v);
      ath = fmaf(a.w[g], th, ath);
      if (a.avg_opt_state) { am = fmaf(a.w[g], m, am); av = fmaf(a.w[g], v, av); }
      else {
        a.m[g][addr + e] = m; a.v[g][addr + e] = v;
        for (uint32_t r = 0; r + 1 < a.replicas; ++r) {
          const uint32_t i = g * (a.replicas - 1) + r;
          a.m_extra[i][addr + e] = m; a.v_extra[i][addr + e] = v;
        }
      }
    }
    const uint16_t b = to_bf16_bits(ath);
    for (uint32_t g = 0; g < a.G; ++g) {
      a.theta[g][addr + e] = ath;
      a.pbf16[g][j + e] = b;
      if (a.avg_opt_state) { a.m[g][addr + e] = am; a.v[g][addr + e] = av; }
    }
    for (uint32_t i = 0; i < a.G * (a.replicas - 1); ++i) {
      a.theta_extra[i][addr + e] = ath;
      a.pbf16_extra[i][j + e] = b;
      if (a.avg_opt_state) { a.m_extra[i][addr + e] = am; a.v_extra[i][addr + e] = av; }
    }
  }
}

template <bool OPT>
__global__ void __launch_bounds__(kThreads, FLS_FUSED_MINB) fls_adamw_fedavg_kernel(const __grid_constant__ FusedArgs a) {
  const uint32_t n_tiles = a.idx.n_tiles;
  if (blockIdx.x >= n_tiles) { dep_wait(); dep_launch(); return; }
  bool waited = false;
  Walker w;
  w.init(a.idx, a.descending ? n_tiles - 1 - blockIdx.x : blockIdx.x);
  for (uint32_t lin = blockIdx.x; lin < n_tiles; lin += gridDim.x) {
    const uint32_t tile = a.descending ? n_tiles - 1 - lin : lin;
    const Slice s = slice_of(w.seek(tile), tile, threadIdx.x);
    if (s.vec) {
      F8 ath, am, av;
#pragma unroll
      for (int e = 0; e < 8; ++e) ath.v[e] = am.v[e] = av.v[e] = 0.f;
#pragma unroll 1
      for (uint32_t g = 0; g < a.G; ++g) {
        // theta, m, v are not written by the reduce kernels: group 0's can be fetched before the wait
        F8 th = ld8_stream(a.theta[g] + s.a);
        F8 m = ld8_stream(a.m[g] + s.a);
        F8 v = ld8_stream(a.v[g] + s.a);
        if (!waited) { dep_wait(); dep_launch(); waited = true; }
        const F8 gb = ld8_stream(a.gbar[g] + s.a);
        const float c = __ldcg(a.coefs + g), wg = a.w[g];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          adamw_one(a, c, gb.v[e], th.v[e], m.v[e], v.v[e]);
          ath.v[e] = fmaf(wg, th.v[e], ath.v[e]);
          if (OPT) { am.v[e] = fmaf(wg, m.v[e], am.v[e]); av.v[e] = fmaf(wg, v.v[e], av.v[e]); }
        }
        if (!OPT) {
          st8_stream(a.m[g] + s.a, m); st8_stream(a.v[g] + s.a, v);
          // the group's other replicas ran the same update on the same gradient: they get the same moments
          for (uint32_t r = 0; r + 1 < a.replicas; ++r) {
            const uint32_t i = g * (a.replicas - 1) + r;
            st8_stream(a.m_extra[i] + s.a, m); st8_stream(a.v_extra[i] + s.a, v);
          }
        }
      }
      const uint4 p = pack_bf16x8(ath);
      for (uint32_t g = 0; g < a.G; ++g) {
        st8_stream(a.theta[g] + s.a, ath);
        st_b128_stream(a.pbf16[g] + s.j, p);
        if (OPT) { st8_stream(a.m[g] + s.a, am); st8_stream(a.v[g] + s.a, av); }
      }
      for (uint32_t i = 0; i < a.G * (a.replicas - 1); ++i) {     // the broadcast to the other replicas of every group
        st8_stream(a.theta_extra[i] + s.a, ath);
        st_b128_stream(a.pbf16_extra[i] + s.j, p);
        if (OPT) { st8_stream(a.m_extra[i] + s.a, am); st8_stream(a.v_extra[i] + s.a, av); }
      }
    } else if (s.n) {
      if (!waited) { dep_wait(); dep_launch(); waited = true; }
      fused_slice_scalar(a, s.j, s.a, s.n);
    }
  }
  if (!waited) { dep_wait(); dep_launch(); }
}

// ------------------------------------------------------------------------------------------------
// Launchers.
// ------------------------------------------------------------------------------------------------
#ifndef FLS_FLAT_THREADS
#define FLS_FLAT_THREADS 256
#define FLS_FLAT_MINB 8
#endif
#ifndef FLS_LEVEL_THREADS
#define FLS_LEVEL_THREADS 256
#define FLS_LEVEL_MINB 5
#endif
constexpr int kFlatThreads = FLS_FLAT_THREADS, kFlatMinB = FLS_FLAT_MINB;       // SG == 0 with a static K
constexpr int kLevelThreads = FLS_LEVEL_THREADS, kLevelMinB = FLS_LEVEL_MINB;   // two-level orders with a static K
// fp32 gradients: double accumulators (twice the registers) and 32-byte loads, so fewer resident CTAs
constexpr int kFlatMinB32 = 5, kLevelMinB32 = 4;
constexpr int kAnyThreads = 256, kAnyMinB = 2;         // run-time K: batches of 8 loads need the registers
#ifndef FLS_FEW_THREADS
#define FLS_FEW_THREADS 256
#define FLS_FEW_MINB 4
#endif
constexpr int kFewThreads = FLS_FEW_THREADS, kFewMinB = FLS_FEW_MINB;   // K = 1 or 2: several tiles per thread (see tiles_per_thread)

// tiles per thread so that 8 (bf16) or 4 (fp32, 32-byte) loads are in flight per thread; 1 for K >= 4
template <bool F32, int KT> constexpr int tiles_per_thread() { return (KT == 1 || KT == 2) ? (F32 ? 4 : 8) / KT : 1; }

// Launch, with programmatic stream serialization if `overlap` (see dep_wait / dep_launch above).
template <typename Args>
void launch_k(void (*kernel)(Args), const Args& a, unsigned grid, unsigned threads, cudaStream_t st, bool overlap) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kernel, a);
}

// tiles one CTA of the reduce kernel covers, for the shape that launch_reduce_shape picks
inline unsigned reduce_tiles_per_cta(const ReduceArgs& a, int sg, bool f32) {
  const bool static_k = sg >= 0 && (a.K == 1 || a.K == 2 || a.K == 4 || a.K == 8);
  if (!static_k) return kAnyThreads / kThreads;
  if (a.K <= 2) return (kFewThreads / kThreads) * ((f32 ? 4u : 8u) / a.K);
  return (sg == 0 ? kFlatThreads : kLevelThreads) / kThreads;
}

template <bool F32, int KT, int SG>
void launch_reduce_shape(const ReduceArgs& a, unsigned grid, cudaStream_t st, bool ov) {
  if constexpr (KT == 0)
    launch_k(fls_reduce_kernel<F32, KT, SG, kAnyThreads, kAnyMinB, 1>, a, grid, kAnyThreads, st, ov);
  else if constexpr (KT <= 2)
    launch_k(fls_reduce_kernel<F32, KT, SG, kFewThreads, kFewMinB, tiles_per_thread<F32, KT>()>, a, grid, kFewThreads, st, ov);
  else if constexpr (SG == 0)
    launch_k(fls_reduce_kernel<F32, KT, SG, kFlatThreads, F32 ? kFlatMinB32 : kFlatMinB, 1>, a, grid, kFlatThreads, st, ov);
  else
    launch_k(fls_reduce_kernel<F32, KT, SG, kLevelThreads, F32 ? kLevelMinB32 : kLevelMinB, 1>, a, grid, kLevelThreads, st, ov);
}

template <bool F32, int KT>
void launch_reduce_k(const ReduceArgs& a, int sg, unsigned grid, cudaStream_t st, bool ov) {
  // only the level structures that can occur with KT buffers are instantiated (SG divides KT)
  if (sg == 0) { launch_reduce_shape<F32, KT, 0>(a, grid, st, ov); return; }
  if constexpr (KT == 0 || KT >= 2) { if (sg == 1) { launch_reduce_shape<F32, KT, 1>(a, grid, st, ov); return; } }
  if constexpr (KT == 0 || KT >= 4) { if (sg == 2) { launch_reduce_shape<F32, KT, 2>(a, grid, st, ov); return; } }
  if constexpr (KT == 0 || KT == 8) { if (sg == 4) { launch_reduce_shape<F32, KT, 4>(a, grid, st, ov); return; } }
  if constexpr (KT == 0 && !F32) { if (sg == -2) { launch_reduce_shape<F32, 0, -2>(a, grid, st, ov); return; } }
  launch_reduce_shape<F32, 0, -1>(a, grid, st, ov);
}

template <bool F32>
void launch_reduce_t(const ReduceArgs& a, int sg, unsigned grid, cudaStream_t st, bool ov) {
  if (sg >= 0) {
    switch (a.K) {
      case 1: launch_reduce_k<F32, 1>(a, sg, grid, st, ov); return;
      case 2: launch_reduce_k<F32, 2>(a, sg, grid, st, ov); return;
      case 4: launch_reduce_k<F32, 4>(a, sg, grid, st, ov); return;
      case 8: launch_reduce_k<F32, 8>(a, sg, grid, st, ov); return;
      default: break;
    }
  }
  launch_reduce_k<F32, 0>(a, sg, grid, st, ov);
}

}  // namespace

unsigned reduce_grid(const ReduceArgs& a, int sg, bool f32) {
  const unsigned tiles_per_cta = reduce_tiles_per_cta(a, sg, f32);
  return (a.idx.n_tiles + tiles_per_cta - 1) / tiles_per_cta;
}

namespace {
template <typename Args>
void launch_k2(void (*kernel)(Args), const Args& a, unsigned grid_x, unsigned grid_y, unsigned threads, cudaStream_t st, bool overlap) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid_x, grid_y);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kernel, a);
}

template <bool F32, int KT, int SG>
void launch_reduce_batch_shape(const ReduceArgs& a, unsigned grid, unsigned groups, cudaStream_t st, bool ov) {
  if constexpr (SG == 0)
    launch_k2(fls_reduce_kernel<F32, KT, SG, kFlatThreads, F32 ? kFlatMinB32 : kFlatMinB, 1, true>, a, grid, groups, kFlatThreads, st, ov);
  else
    launch_k2(fls_reduce_kernel<F32, KT, SG, kLevelThreads, F32 ? kLevelMinB32 : kLevelMinB, 1, true>, a, grid, groups, kLevelThreads, st, ov);
}

// K = 1 or 2 (norm-only passes of recompute plans): the several-tiles-per-thread shape of launch_reduce_shape
template <bool F32, int KT, int SG>
void launch_reduce_batch_few(const ReduceArgs& a, unsigned grid, unsigned groups, cudaStream_t st, bool ov) {
  launch_k2(fls_reduce_kernel<F32, KT, SG, kFewThreads, kFewMinB, tiles_per_thread<F32, KT>(), true>, a, grid, groups, kFewThreads, st, ov);
}

template <bool F32>
void launch_reduce_batch_t(const ReduceArgs& a, int sg, unsigned grid, unsigned groups, cudaStream_t st, bool ov) {
  if (a.K == 1) {
    launch_reduce_batch_few<F32, 1, 0>(a, grid, groups, st, ov);
  } else if (a.K == 2) {
    if (sg == 0) launch_reduce_batch_few<F32, 2, 0>(a, grid, groups, st, ov);
    else launch_reduce_batch_few<F32, 2, 1>(a, grid, groups, st, ov);
  } else if (a.K == 4) {
    if (sg == 0) launch_reduce_batch_shape<F32, 4, 0>(a, grid, groups, st, ov);
    else if (sg == 1) launch_reduce_batch_shape<F32, 4, 1>(a, grid, groups, st, ov);
    else launch_reduce_batch_shape<F32, 4, 2>(a, grid, groups, st, ov);
  } else {
    if (sg == 0) launch_reduce_batch_shape<F32, 8, 0>(a, grid, groups, st, ov);
    else if (sg == 1) launch_reduce_batch_shape<F32, 8, 1>(a, grid, groups, st, ov);
    else if (sg == 2) launch_reduce_batch_shape<F32, 8, 2>(a, grid, groups, st, ov);
    else launch_reduce_batch_shape<F32, 8, 4>(a, grid, groups, st, ov);
  }
}
}  // namespace

bool reduce_batchable(uint32_t K, int sg) {
  return (K == 4 && (sg == 0 || sg == 1 || sg == 2)) || (K == 8 && (sg == 0 || sg == 1 || sg == 2 || sg == 4));
}
bool norm_pass_batchable(uint32_t K, int sg) { return (K == 1 && sg == 0) || (K == 2 && (sg == 0 || sg == 1)); }

cudaError_t launch_reduce_batch(const ReduceArgs& a, bool f32, int sg, unsigned groups, cudaStream_t st, bool overlap) {
  const unsigned grid = reduce_grid(a, sg, f32);
  if (f32)
    launch_reduce_batch_t<true>(a, sg, grid, groups, st, overlap);
  else
    launch_reduce_batch_t<false>(a, sg, grid, groups, st, overlap);
  return cudaGetLastError();
}

cudaError_t launch_adamw_batch(const AdamBatchArgs& a, unsigned grid, unsigned groups, cudaStream_t st, bool overlap) {
  launch_k2(fls_adamw_batch_kernel, a, grid, groups, kThreads, st, overlap);
  return cudaGetLastError();
}

cudaError_t launch_reduce(const ReduceArgs& a, bool f32, int sg, cudaStream_t st, bool overlap) {
  const unsigned grid = reduce_grid(a, sg, f32);
  if (f32)
    launch_reduce_t<true>(a, sg, grid, st, overlap);
  else
    launch_reduce_t<false>(a, sg, grid, st, overlap);
  return cudaGetLastError();
}

namespace {
template <bool F32, int KT>
void launch_noclip_k(const ReduceAdamArgs& a, int sg, unsigned grid, cudaStream_t st, bool ov) {
  if (sg == 0) { launch_k(fls_step_noclip_kernel<F32, KT, 0>, a, grid, kThreads, st, ov); return; }
  if constexpr (KT == 0 || KT >= 2) { if (sg == 1) { launch_k(fls_step_noclip_kernel<F32, KT, 1>, a, grid, kThreads, st, ov); return; } }
  if constexpr (KT == 0 || KT >= 4) { if (sg == 2) { launch_k(fls_step_noclip_kernel<F32, KT, 2>, a, grid, kThreads, st, ov); return; } }
  if constexpr (KT == 0 || KT == 8) { if (sg == 4) { launch_k(fls_step_noclip_kernel<F32, KT, 4>, a, grid, kThreads, st, ov); return; } }
  launch_k(fls_step_noclip_kernel<F32, 0, -1>, a, grid, kThreads, st, ov);
}
template <bool F32>
void launch_noclip_t(const ReduceAdamArgs& a, int sg, unsigned grid, cudaStream_t st, bool ov) {
  if (sg >= 0) {
    switch (a.r.K) {
      case 1: launch_noclip_k<F32, 1>(a, sg, grid, st, ov); return;
      case 2: launch_noclip_k<F32, 2>(a, sg, grid, st, ov); return;
      case 4: launch_noclip_k<F32, 4>(a, sg, grid, st, ov); return;
      case 8: launch_noclip_k<F32, 8>(a, sg, grid, st, ov); return;
      default: break;
    }
  }
  launch_noclip_k<F32, 0>(a, sg, grid, st, ov);
}
}  // namespace

// Single pass for plans without clipping; the grid is one CTA per tile (= the number of norm partials).
cudaError_t launch_step_noclip(const ReduceAdamArgs& a, bool f32, int sg, cudaStream_t st, bool overlap) {
  const unsigned grid = a.a.idx.n_tiles;
  if (f32)
    launch_noclip_t<true>(a, sg, grid, st, overlap);
  else
    launch_noclip_t<false>(a, sg, grid, st, overlap);
  return cudaGetLastError();
}

namespace {
using ResidentKernel = void (*)(ResidentArgs);
template <bool F32, int KT>
ResidentKernel resident_kernel_k(int sg) {
  if (sg == 0) return fls_step_resident_kernel<F32, KT, 0>;
  if constexpr (KT >= 2) { if (sg == 1) return fls_step_resident_kernel<F32, KT, 1>; }
  if constexpr (KT >= 4) { if (sg == 2) return fls_step_resident_kernel<F32, KT, 2>; }
  if constexpr (KT == 8) { if (sg == 4) return fls_step_resident_kernel<F32, KT, 4>; }
  return nullptr;
}
template <bool F32>
ResidentKernel resident_kernel_t(uint32_t K, int sg) {
  switch (K) {
    case 1: return resident_kernel_k<F32, 1>(sg);
    case 2: return resident_kernel_k<F32, 2>(sg);
    case 4: return resident_kernel_k<F32, 4>(sg);
    case 8: return resident_kernel_k<F32, 8>(sg);
    default: return nullptr;
  }
}
ResidentKernel resident_kernel(bool f32, uint32_t K, int sg) {
  return f32 ? resident_kernel_t<true>(K, sg) : resident_kernel_t<false>(K, sg);
}
}  // namespace

bool resident_shape_ok(uint32_t K, int sg) { return resident_kernel(false, K, sg) != nullptr; }

cudaError_t resident_max_ctas(bool f32, uint32_t K, int sg, size_t smem_bytes, int sm_count, unsigned* out) {
  *out = 0;
  ResidentKernel k = resident_kernel(f32, K, sg);
  if (!k) return cudaErrorInvalidValue;
  // allow the kernel the device's whole opt-in shared memory once and for all: plans with different tile counts share it
  int dev = 0, optin = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  if (smem_bytes + 256 > size_t(optin)) return cudaSuccess;      // (static shared memory included) does not fit: 0 CTAs
  e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - 256);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, kThreads, smem_bytes);
  if (e != cudaSuccess) return e;
  *out = unsigned(per_sm) * unsigned(sm_count);
  return cudaSuccess;
}

// Cooperative launch: the driver refuses the launch unless the whole grid can be resident at once, which is what
// lets the CTAs of a group wait for one another inside the kernel.
cudaError_t launch_step_resident(const ResidentArgs& a, bool f32, int sg, unsigned grid_x, unsigned groups, cudaStream_t st) {
  ResidentKernel k = resident_kernel(f32, a.r.K, sg);
  if (!k) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid_x, groups);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = size_t(a.tiles_per_cta) * kTile * sizeof(float);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k, a);
}

cudaError_t launch_reduce_adamw(const ReduceAdamArgs& a, bool f32, int sg, unsigned grid, cudaStream_t st, bool overlap) {
  // static shapes for the recompute plan (K * e_g < 8: bf16 with K <= 3, fp32 with K = 1); any other K, which only
  // the redo of a speculative step brings here, takes the run-time-K form
  const uint32_t K = a.r.K;
  if (f32 && K == 1) {
    launch_k(fls_reduce_adamw_kernel<true, 1, 0>, a, grid, kThreads, st, overlap);
  } else if (f32 && sg == 0) {
    launch_k(fls_reduce_adamw_kernel<true, 0, 0>, a, grid, kThreads, st, overlap);
  } else if (f32 && sg == 1) {
    launch_k(fls_reduce_adamw_kernel<true, 0, 1>, a, grid, kThreads, st, overlap);
  } else if (f32) {
    launch_k(fls_reduce_adamw_kernel<true, 0, -1>, a, grid, kThreads, st, overlap);
  } else if (K == 1) {
    launch_k(fls_reduce_adamw_kernel<false, 1, 0>, a, grid, kThreads, st, overlap);
  } else if (K == 2 && sg == 0) {
    launch_k(fls_reduce_adamw_kernel<false, 2, 0>, a, grid, kThreads, st, overlap);
  } else if (K == 2 && sg == 1) {
    launch_k(fls_reduce_adamw_kernel<false, 2, 1>, a, grid, kThreads, st, overlap);
  } else if (sg == 0) {
    launch_k(fls_reduce_adamw_kernel<false, 0, 0>, a, grid, kThreads, st, overlap);
  } else if (sg == 1) {
    launch_k(fls_reduce_adamw_kernel<false, 0, 1>, a, grid, kThreads, st, overlap);
  } else {
    launch_k(fls_reduce_adamw_kernel<false, 0, -1>, a, grid, kThreads, st, overlap);
  }
  return cudaGetLastError();
}

cudaError_t launch_adamw(const AdamArgs& a, unsigned grid, cudaStream_t st, bool overlap) {
  launch_k(fls_adamw_kernel, a, grid, kThreads, st, overlap);
  return cudaGetLastError();
}

cudaError_t launch_fedavg(const FedavgArgs& a, unsigned grid, cudaStream_t st, bool overlap) {
  switch (a.G) {
    case 1: launch_k(fls_fedavg_kernel<1, 6>, a, grid, kThreads, st, overlap); break;
    case 2: launch_k(fls_fedavg_kernel<2, 5>, a, grid, kThreads, st, overlap); break;
    case 4: launch_k(fls_fedavg_kernel<4, 4>, a, grid, kThreads, st, overlap); break;
    case 8: launch_k(fls_fedavg_kernel<8, FLS_FEDAVG_BATCH_MINB>, a, grid, kThreads, st, overlap); break;
    default: launch_k(fls_fedavg_kernel<0, FLS_FEDAVG_BATCH_MINB>, a, grid, kThreads, st, overlap); break;
  }
  return cudaGetLastError();
}

cudaError_t launch_adamw_fedavg(const FusedArgs& a, unsigned grid, cudaStream_t st, bool overlap) {
  if (a.avg_opt_state)
    launch_k(fls_adamw_fedavg_kernel<true>, a, grid, kThreads, st, overlap);
  else
    launch_k(fls_adamw_fedavg_kernel<false>, a, grid, kThreads, st, overlap);
  return cudaGetLastError();
}

}  // namespace fls
