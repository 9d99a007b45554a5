// Kernel argument blocks and launchers (implemented in fls_kernels.cu).
#pragma once
#include <cuda_runtime.h>

#include "fls_internal.h"

namespace fls {

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
  const void* grad[FLS_MAX_GRAD_BUFFERS];  // device, K buffers of this group, index rho*S + sigma
  float* gbar;                             // device, reduced gradient (shard order)
  SegIndex idx;
  uint32_t K;
  float k_float, inv_k;                    // K and 1/K as float: the mean is scaled by 1/K once
  uint32_t k_is_pow2;                      // 1/K exact: multiply; otherwise divide
  uint32_t fold_mask;                      // bit i set: the i-th batch of 8 buffers closes a sharding group
  uint64_t end_mask;                       // bit k set: buffer k closes a sharding group
  double* partials;                        // device, one per CTA
  uint32_t* ticket;                        // device, zero between launches
  float* norm_out;
  float* coef_out;
  double* normsq_out;
  uint32_t* status;
  double max_grad_norm;
  int store_gbar;                          // 0: norm only (the recompute plan: the mean gradient is formed again in AdamW)
};

struct AdamArgs {
  const float* gbar;
  float *theta, *m, *v;
  uint16_t* pbf16;
  SegIndex idx;
  int descending;
  const float* coef;                       // device, written by the reduce kernel of the same group
  float decay, beta1, omb1, beta2, omb2, step_size, inv_sqrt_bc2, eps;
};

// AdamW that forms the mean gradient itself from the K gradient buffers (recompute plan, small K).
struct ReduceAdamArgs {
  ReduceArgs r;                            // gradient pointers, level structure, 1/K (its outputs are not used)
  AdamArgs a;                              // state pointers, scalars (its gbar is not used)
};

struct FedavgArgs {
  float* x[FLS_MAX_GROUPS];                // device, the G copies (in/out)
  uint16_t* pbf16[FLS_MAX_GROUPS];         // device, the G bf16 copies (out), used if write_bf16
  float w[FLS_MAX_GROUPS];
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
cudaError_t launch_step_noclip(const ReduceAdamArgs& a, bool f32, int sg, cudaStream_t st, bool overlap);
cudaError_t launch_reduce_adamw(const ReduceAdamArgs& a, bool f32, int sg, unsigned grid, cudaStream_t st, bool overlap);
cudaError_t launch_adamw(const AdamArgs& a, unsigned grid, cudaStream_t st, bool overlap);
cudaError_t launch_fedavg(const FedavgArgs& a, unsigned grid, cudaStream_t st, bool overlap);
cudaError_t launch_adamw_fedavg(const FusedArgs& a, unsigned grid, cudaStream_t st, bool overlap);

}  // namespace fls
