// Kernel argument blocks and launchers (implemented in fls_kernels.cu).
#pragma once
#include <cuda_runtime.h>

#include "fls_internal.h"

namespace fls {

constexpr int FLS_MAX_FUSED_EXTRA = 32;    // extra state copies (G*(R_rep-1)) the fused aggregation kernel can serve

// Where the tiles of each segment end, for the tile -> segment search.  Small tables (the usual case)
// are also copied here so that the search runs out of the kernel parameters (constant bank) instead of
// global memory; the segment record itself is then one global load.
struct SegIndex {
  const Segment* segs;                     // device
  uint32_t n_seg;
  uint32_t n_tiles;
  uint32_t in_params;                      // 1: tile_end[] below is filled
  uint32_t tile_end[kParamSegs];
};

struct ReduceArgs {
  const void* grad[FLS_MAX_GRAD_BUFFERS];  // device, K buffers of this group, index rho*S + sigma (batched launch: the
                                           // buffers of all groups, index g*K + rho*S + sigma)
  float* gbar;                             // device, reduced gradient (shard order)
  // Batched launch (gridDim.y = groups, K in {4, 8}): group y = blockIdx.y uses grad[y*K ..], gbar + y*gbar_stride,
  // entries y*gridDim.x.. of partials, y*tree_stride.. of the chunk arrays, and entry y of ticket, norm_out, coef_out,
  // normsq_out.  A plain launch is the case y = 0.
  uint64_t gbar_stride;                    // elements
  uint32_t tree_stride;                    // chunks per group
  SegIndex idx;
  uint32_t K;
  float k_float, inv_k;                    // K and 1/K as float: the mean is scaled by 1/K once
  uint32_t k_is_pow2;                      // 1/K exact: multiply; otherwise divide
  uint32_t keep_from_tile;                 // tiles from this one on store the mean gradient with L2::evict_last (the
                                           // AdamW kernel reads them first), the others with evict_first
  uint32_t fold_mask;                      // bit i set: the i-th batch of 8 buffers closes a sharding group
  uint64_t end_mask;                       // bit k set: buffer k closes a sharding group
  double* partials;                        // device, one per CTA
  double* chunk_partials;                  // device, one per chunk of 256 CTAs
  uint32_t* chunk_count;                   // device, one per chunk, zero between launches
  uint32_t* ticket;                        // device, zero between launches
  float* norm_out;
  float* coef_out;
  double* normsq_out;
  uint32_t* status;
  double max_grad_norm;
  int store_gbar;                          // 0: norm only (the recompute plan: the mean gradient is formed again in AdamW)
  // ring order (generic kernels only): visit the buffers as a ring reduce-scatter / all-reduce would
  uint32_t ring;                           // 0: ascending buffer index at both levels
  uint32_t S, R;                           // shard_dim, replicate_dim (used by the ring order)
  uint32_t* spec_counts;                   // device, 2 counters (coefficient == 1, != 1) or null: speculative steps only
  // resident step only (null otherwise): the warp that finishes group y's norm publishes ready[y] = launch_id after the
  // coefficient, which releases the group's CTAs waiting in the same kernel
  uint32_t* ready;
  uint32_t launch_id;
};

struct AdamArgs {
  const float* gbar;
  float *theta, *m, *v;                    // state read (and, in fls_adamw_kernel, updated in place)
  float *theta_out, *m_out, *v_out;        // where the kernels that form the gradient themselves store the new state
                                           // (the same three pointers, or the other buffer set of a speculative plan)
  uint16_t* pbf16;
  SegIndex idx;
  int descending;
  const float* coef;                       // device, written by the reduce kernel of the same group
  float decay, beta1, omb1, beta2, omb2, step_size, inv_sqrt_bc2, eps;
};

// AdamW of all groups in one grid (gridDim.y = groups): group y = blockIdx.y.
struct AdamBatchArgs {
  float* theta[FLS_MAX_GROUPS];
  float* m[FLS_MAX_GROUPS];
  float* v[FLS_MAX_GROUPS];
  uint16_t* pbf16[FLS_MAX_GROUPS];
  const float* gbar;                       // group 0's reduced gradient
  uint64_t gbar_stride;                    // elements between the groups' reduced gradients
  const float* coef;                       // group 0's clip coefficient; group y's is coef[y]
  SegIndex idx;
  int descending;
  float decay, beta1, omb1, beta2, omb2, step_size, inv_sqrt_bc2, eps;
};

// Whole step of all groups in ONE cooperative kernel (small plans): every CTA reduces its tiles, keeps the mean gradient
// in shared memory, waits until its group's norm is complete and applies AdamW.
struct ResidentArgs {
  ReduceArgs r;                            // batched form (all groups' buffers; gbar unused, store_gbar = 0)
  float* theta[FLS_MAX_GROUPS];
  float* m[FLS_MAX_GROUPS];
  float* v[FLS_MAX_GROUPS];
  uint16_t* pbf16[FLS_MAX_GROUPS];
  float decay, beta1, omb1, beta2, omb2, step_size, inv_sqrt_bc2, eps;
  uint32_t tiles_per_cta;                  // T: CTA x takes tiles x, x + gridDim.x, ... (T of them at most)
  uint32_t wait_limit;                     // polls of ready[y] before a CTA gives up (FLS_STATUS_WAIT_EXPIRED)
  uint32_t expect_id;                      // what ready[y] must hold for the wait to end (= r.launch_id)
};

// AdamW that forms the mean gradient itself from the K gradient buffers (recompute plan, small K).
struct ReduceAdamArgs {
  ReduceArgs r;                            // gradient pointers, level structure, 1/K (its outputs are not used)
  AdamArgs a;                              // state pointers, scalars (its gbar is not used)
  int skip_if_unclipped;                   // second kernel of a speculative step: return at once if the coefficient is 1
};

struct FedavgArgs {
  float* x[FLS_MAX_GROUPS];                // device, the G copies (in/out)
  uint16_t* pbf16[FLS_MAX_GROUPS];         // device, the G bf16 copies (out), used if write_bf16
  float w[FLS_MAX_GROUPS];
  // plans with one state copy per replica: x[] holds replica 0 of every group (the one that aggregates); the
  // average is also stored ("broadcast") to the other copies listed here
  float* x_extra[FLS_MAX_GROUPS];
  uint16_t* pbf16_extra[FLS_MAX_GROUPS];
  uint32_t n_extra;
  SegIndex idx;
  uint32_t G;
  int write_bf16;
  int descending;
  // outer optimizer (both null: plain FedAvg)
  float* x_global;                         // device, in/out
  float* outer_buf;                        // device, in/out: momentum buffer
  float outer_lr, momentum;
  int nesterov;
};

// AdamW of all G groups + FedAvg of the results in one pass (G <= FLS_MAX_FUSED_GROUPS).
struct FusedArgs {
  const float* gbar[FLS_MAX_FUSED_GROUPS];  // device, one reduced gradient per group
  float* theta[FLS_MAX_FUSED_GROUPS];
  float* m[FLS_MAX_FUSED_GROUPS];
  float* v[FLS_MAX_FUSED_GROUPS];
  uint16_t* pbf16[FLS_MAX_FUSED_GROUPS];
  float w[FLS_MAX_FUSED_GROUPS];
  // plans with one state copy per replica: the arrays above hold replica 0 of every group; copy r >= 1 of group g
  // is entry g*(R-1) + r-1 of the arrays below (R = replicas)
  float* theta_extra[FLS_MAX_FUSED_EXTRA];
  float* m_extra[FLS_MAX_FUSED_EXTRA];
  float* v_extra[FLS_MAX_FUSED_EXTRA];
  uint16_t* pbf16_extra[FLS_MAX_FUSED_EXTRA];
  uint32_t replicas;                       // 1: no extra copies
  const float* coefs;                      // device, G clip coefficients written by the reduce kernels
  SegIndex idx;
  uint32_t G;
  int avg_opt_state;                       // m and v are averaged too
  int descending;
  float decay, beta1, omb1, beta2, omb2, step_size, inv_sqrt_bc2, eps;
};

// sg: level structure of the reduction (see reduce_elems): 0, 1, 2, 4 or -1 for the generic form;
// -2: the generic form with every partial sum and the mean rounded to bf16 (bf16 gradients only).
// The reduce kernel has one launch shape; reduce_grid() is its grid (= number of norm partials it writes).
unsigned reduce_grid(const ReduceArgs& a, int sg, bool f32);
// overlap: launch with programmatic stream serialization, so that the kernel's first CTAs may start during
// the tail of the kernel launched just before it on the same stream (which must be one of these three).
cudaError_t launch_reduce(const ReduceArgs& a, bool f32, int sg, cudaStream_t st, bool overlap);
// All groups in one grid; only for K in {4, 8} with a static level structure (reduce_batchable).
bool reduce_batchable(uint32_t K, int sg);
// K = 1 or 2: launch_reduce_batch serves them too, for the norm-only passes of recompute plans (store_gbar = 0)
bool norm_pass_batchable(uint32_t K, int sg);
cudaError_t launch_reduce_batch(const ReduceArgs& a, bool f32, int sg, unsigned groups, cudaStream_t st, bool overlap);
cudaError_t launch_adamw_batch(const AdamBatchArgs& a, unsigned grid, unsigned groups, cudaStream_t st, bool overlap);
cudaError_t launch_step_noclip(const ReduceAdamArgs& a, bool f32, int sg, cudaStream_t st, bool overlap);
// Resident step: static K in {1, 2, 4, 8} with a static level structure only (resident_shape_ok).  The launch is
// cooperative: grid_x * groups CTAs must be resident at once; resident_max_ctas gives that bound for a given amount
// of dynamic shared memory (tiles_per_cta * kTile * 4 bytes) on the current device.
bool resident_shape_ok(uint32_t K, int sg);
cudaError_t resident_max_ctas(bool f32, uint32_t K, int sg, size_t smem_bytes, int sm_count, unsigned* out);
cudaError_t launch_step_resident(const ResidentArgs& a, bool f32, int sg, unsigned grid_x, unsigned groups, cudaStream_t st);
cudaError_t launch_reduce_adamw(const ReduceAdamArgs& a, bool f32, int sg, unsigned grid, cudaStream_t st, bool overlap);
cudaError_t launch_adamw(const AdamArgs& a, unsigned grid, cudaStream_t st, bool overlap);
cudaError_t launch_fedavg(const FedavgArgs& a, unsigned grid, cudaStream_t st, bool overlap);
cudaError_t launch_adamw_fedavg(const FusedArgs& a, unsigned grid, cudaStream_t st, bool overlap);

}  // namespace fls
