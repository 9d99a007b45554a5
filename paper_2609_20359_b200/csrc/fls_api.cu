// C ABI of libfls (see include/fls.h for the contract of every call).
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <limits>
#include <new>
#include <string>
#include <vector>

#include "fls_kernels.h"

using namespace fls;

namespace {

thread_local std::string g_err;

int fail(int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_err = buf;
  return code;
}

int cuda_fail(cudaError_t e, const char* what) {
  return fail(FLS_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}

struct TimedLaunch {
  cudaEvent_t begin, end;
  int kernel;
};

struct Range {
  uintptr_t lo, hi;
  const char* what;
  int index;
  bool output;
};

}  // namespace

constexpr uint64_t kBatchScratchBytes = 24ull << 20;
constexpr uint64_t kResidentAutoBytes = 16ull << 20;   // mean gradients of all groups up to which the resident step is chosen automatically

struct fls_plan {
  fls_plan_desc desc{};
  std::vector<uint64_t> units;
  Layout lay;
  uint32_t K = 0;
  uint32_t R_state = 1;     // state copies per group: R_rep with FLS_STATE_PER_REPLICA, else 1
  uint32_t n_copies = 0;    // G * R_state: entries of master / m / v / pbf16
  bool ring = false;
  uint64_t end_mask = 0;
  uint32_t fold_mask = 0;
  int reduce_sg = -1;

  bool bound = false;
  int device = -1;
  int sm_count = 0;
  std::vector<const void*> grads;
  std::vector<float*> master, m, v;      // current state of every copy (index g*R_state + rho)
  std::vector<uint16_t*> pbf16;
  std::vector<float*> master2, m2, v2;   // second buffer set of a speculative plan (the one not current)
  std::vector<Range> ranges;             // everything bound, for overlap checks of later additions
  bool speculative = false;
  bool fused_plan = false;               // fls_sync_step_fedavg may fuse the aggregation into the optimizer kernel
  int batch_mode = -1;                   // groups in one grid: -1 automatic (small plans), 0 never, 1 whenever possible
  int resident_mode = -1;                // whole step in one cooperative kernel: -1 automatic, 0 never, 1 whenever it fits
  uint32_t res_tiles = 0, res_grid = 0;  // tiles per CTA and grid.x of the resident step on the bound device (0: does not fit)
  uint32_t res_seq = 0;                  // id of the last resident launch (what the ready words are compared with)
  uint32_t res_wait_limit = 1u << 22;    // polls (64 ns apart at least) before a CTA gives up
  bool res_hold_back = false;            // test hook: the next resident launch waits for an id nobody publishes
  uint64_t l2_keep_bytes = 64ull << 20;  // tail of the reduced gradient stored with L2 evict-last
  char* ws = nullptr;

  uint64_t step = 0;
  uint64_t launches = 0;
  int ctas_per_sm[FLS_KERNEL_COUNT] = {0, 0, 0, 0};   // 0: the grid covers every tile once (no grid-stride loop)
  int descending[FLS_KERNEL_COUNT] = {0, 1, 0, 1};   // AdamW starts where the reduce kernel stopped: those lines are still in L2

  bool overlap = true;     // programmatic dependent launch between the kernels of one call
  bool recompute = false;  // K * e_g < 8: the norm pass stores nothing and AdamW forms the mean gradient again
  bool single_pass = false;  // no clipping: reduce + norm + AdamW in one kernel
  bool profiling = false;
  std::vector<TimedLaunch> timed;
  std::vector<cudaEvent_t> event_pool;

  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_begin = nullptr;
  std::vector<cudaEvent_t> ev_copied;

  const Segment* d_segs() const { return reinterpret_cast<const Segment*>(ws + kWsSegments); }
  float* d_gbar(uint32_t slot = 0) const { return reinterpret_cast<float*>(ws + lay.ws_scratch_offset + lay.scratch_stride * slot); }
  uint32_t last_slot = 0;   // where the last processed group's reduced gradient lives
  bool gbar_valid = false;  // false after a step of a recompute plan: nothing was stored
  float* d_norms() const { return reinterpret_cast<float*>(ws + kWsNorms); }
  float* d_coefs() const { return reinterpret_cast<float*>(ws + kWsCoefs); }
  double* d_normsq() const { return reinterpret_cast<double*>(ws + kWsNormSq); }
  double* d_partials() const { return reinterpret_cast<double*>(ws + lay.ws_partials_offset); }
  double* d_chunk_partials() const { return reinterpret_cast<double*>(ws + lay.ws_chunk_partials_offset); }
  uint32_t* d_chunk_count() const { return reinterpret_cast<uint32_t*>(ws + lay.ws_chunk_count_offset); }
  uint32_t* d_status() const { return reinterpret_cast<uint32_t*>(ws + kWsStatus); }
  uint32_t* d_ticket() const { return reinterpret_cast<uint32_t*>(ws + kWsTickets); }
  uint32_t* d_spec_counts() const { return reinterpret_cast<uint32_t*>(ws + kWsStatus) + 2; }
  uint32_t* d_ready() const { return reinterpret_cast<uint32_t*>(ws + kWsReady); }
  // One grid for all groups (instead of one launch per group) needs a reduced-gradient slot per group, a level structure
  // the batched kernels are built for, the default two-pass route and one state copy per group.  Automatic: only when all
  // the reduced gradients together take at most 24 MiB (a fifth of the L2), i.e. when a launch per group would be launch-bound;
  // larger plans keep the per-group sequence, whose reduced gradient is still in L2 when AdamW reads it.
  bool can_batch() const {
    return desc.groups > 1 && lay.scratch_slots >= desc.groups && uint64_t(desc.groups) * K <= FLS_MAX_GRAD_BUFFERS &&
           reduce_batchable(K, reduce_sg) && plain_reduce() && !single_pass && !recompute && !speculative;
  }
  bool batching() const {
    if (batch_mode == 0 || !can_batch()) return false;
    return batch_mode > 0 || uint64_t(desc.groups) * lay.n_padded * 4 <= kBatchScratchBytes;
  }
  // The whole step as one cooperative kernel: a shape the resident kernel is built for, the plain reduction, clipping on
  // (without it every group's step is one kernel already) and a grid that fits the bound device (res_tiles > 0).
  bool can_resident() const {
    return res_tiles > 0 && resident_shape_ok(K, reduce_sg) && uint64_t(desc.groups) * K <= FLS_MAX_GRAD_BUFFERS &&
           plain_reduce() && !single_pass && !speculative;
  }
  bool resident() const {
    if (resident_mode == 0 || !can_resident()) return false;
    return resident_mode > 0 || uint64_t(desc.groups) * lay.n_padded * 4 <= kResidentAutoBytes;
  }
  // Recompute plans (K * e_g < 8) with several groups: the norm-only passes of all groups can share one grid, followed by
  // one AdamW kernel per group, instead of alternating a short norm pass and a long AdamW kernel per group.
  bool can_norm_first() const {
    return desc.groups > 1 && recompute && !single_pass && !speculative && plain_reduce() &&
           norm_pass_batchable(K, reduce_sg) && uint64_t(desc.groups) * K <= FLS_MAX_GRAD_BUFFERS;
  }
  bool norm_first() const { return batch_mode != 0 && can_norm_first(); }
  // how fls_sync_step currently gets from the gradients to the new state (for the HBM byte count)
  // the routes that form the mean gradient inside the AdamW kernel exist for fp32 partial sums in ascending order
  // and one state copy per group
  bool plain_reduce() const { return desc.reduce_wire == FLS_WIRE_F32 && !ring && R_state == 1; }
  int route() const { return speculative || single_pass || resident() ? 2 : (recompute ? 1 : 0); }

  SegIndex seg_index() const {
    SegIndex ix{};
    ix.segs = d_segs();
    ix.n_seg = uint32_t(lay.segments.size());
    ix.n_tiles = uint32_t(lay.n_tiles);
    ix.in_params = ix.n_seg <= uint32_t(kParamSegs) ? 1u : 0u;
    if (ix.in_params)
      for (uint32_t i = 0; i < ix.n_seg; ++i) ix.tile_end[i] = uint32_t(lay.segments[i].tile_end);
    return ix;
  }

  // grid of the AdamW / FedAvg kernels (the reduce kernel has a single launch shape of its own)
  unsigned grid_for(int kernel) const {
    uint64_t g = ctas_per_sm[kernel] > 0 ? uint64_t(sm_count) * uint64_t(ctas_per_sm[kernel]) : lay.n_tiles;
    g = std::min<uint64_t>(g, lay.n_tiles);
    return unsigned(std::max<uint64_t>(g, 1));
  }

  cudaEvent_t take_event() {
    if (!event_pool.empty()) {
      cudaEvent_t e = event_pool.back();
      event_pool.pop_back();
      return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
  }
};

namespace {

// Brackets one kernel launch with events when profiling is on.
template <typename F>
cudaError_t timed_launch(fls_plan* p, int kernel, cudaStream_t st, F&& launch) {
  TimedLaunch t{nullptr, nullptr, kernel};
  if (p->profiling) {
    t.begin = p->take_event();
    t.end = p->take_event();
    if (!t.begin || !t.end) return cudaErrorMemoryAllocation;
    cudaEventRecord(t.begin, st);
  }
  cudaError_t e = launch();
  if (p->profiling) {
    cudaEventRecord(t.end, st);
    p->timed.push_back(t);
  }
  if (e == cudaSuccess) p->launches++;
  return e;
}

struct AdamScalars { float decay, beta1, omb1, beta2, omb2, step_size, inv_sqrt_bc2, eps; };

// Scalars of the AdamW step, in double on the host, handed to the kernels as fp32.
AdamScalars adam_scalars(const fls_plan_desc& d, double lr, uint64_t t_new) {
  const double bc1 = 1.0 - std::pow(d.beta1, double(t_new));
  const double bc2 = 1.0 - std::pow(d.beta2, double(t_new));
  AdamScalars s;
  s.decay = float(1.0 - lr * d.weight_decay);
  s.beta1 = float(d.beta1);
  s.omb1 = float(1.0 - d.beta1);
  s.beta2 = float(d.beta2);
  s.omb2 = float(1.0 - d.beta2);
  s.step_size = float(lr / bc1);
  s.inv_sqrt_bc2 = float(1.0 / std::sqrt(bc2));
  s.eps = float(d.eps);
  return s;
}

void set_adam_scalars(AdamArgs* aa, const AdamScalars& sc) {
  aa->decay = sc.decay; aa->beta1 = sc.beta1; aa->omb1 = sc.omb1; aa->beta2 = sc.beta2; aa->omb2 = sc.omb2;
  aa->step_size = sc.step_size; aa->inv_sqrt_bc2 = sc.inv_sqrt_bc2; aa->eps = sc.eps;
}

// The part of the reduce kernel's arguments that does not depend on the group.
ReduceArgs common_reduce_args(const fls_plan* p) {
  const fls_plan_desc& d = p->desc;
  ReduceArgs ra{};
  ra.idx = p->seg_index();
  ra.K = p->K;
  ra.k_float = float(p->K);
  ra.inv_k = 1.0f / float(p->K);
  ra.k_is_pow2 = (p->K & (p->K - 1)) == 0 ? 1u : 0u;
  ra.fold_mask = p->fold_mask;
  ra.end_mask = p->end_mask;
  ra.status = p->d_status();
  ra.max_grad_norm = d.max_grad_norm;
  ra.ring = p->ring ? 1u : 0u;
  ra.S = d.shard_dim;
  ra.R = d.replicate_dim;
  ra.spec_counts = nullptr;
  ra.gbar_stride = p->lay.scratch_stride / 4;
  ra.tree_stride = uint32_t(p->lay.n_chunks);
  return ra;
}

// Tiles from which on the reduced gradient is stored "evict last": the AdamW kernel walks it from its end.
uint32_t keep_from_tile(const fls_plan* p, bool reader_descends) {
  const uint64_t keep_tiles = std::min<uint64_t>(p->lay.n_tiles, p->l2_keep_bytes / (uint64_t(kTile) * 4));
  return reader_descends ? uint32_t(p->lay.n_tiles - keep_tiles) : uint32_t(p->lay.n_tiles);
}

// One group's reduce (+ AdamW) launches.  chain: the previous operation on `st` is a kernel of this same call,
// so this group's first kernel may overlap its tail.  slot: which reduced-gradient buffer of the workspace
// receives the mean gradient; with_adamw = false stops after the reduction (the fused aggregation applies AdamW
// to all groups afterwards).
int run_group(fls_plan* p, uint32_t g, double lr, uint64_t t_new, cudaStream_t st, bool chain, uint32_t slot = 0,
              bool with_adamw = true) {
  const fls_plan_desc& d = p->desc;
  const uint32_t c0 = g * p->R_state;      // the group's first state copy
  ReduceArgs ra = common_reduce_args(p);
  for (uint32_t k = 0; k < p->K; ++k) ra.grad[k] = p->grads[size_t(g) * p->K + k];
  ra.gbar = p->d_gbar(slot);
  p->last_slot = slot;
  ra.partials = p->d_partials() + size_t(g) * p->lay.n_tiles;
  ra.chunk_partials = p->d_chunk_partials() + size_t(g) * p->lay.n_chunks;
  ra.chunk_count = p->d_chunk_count() + size_t(g) * p->lay.n_chunks;
  ra.ticket = p->d_ticket() + g;
  ra.norm_out = p->d_norms() + g;
  ra.coef_out = p->d_coefs() + g;
  ra.normsq_out = p->d_normsq() + g;
  // keep the end of the reduced gradient in L2 for the AdamW kernel, stream the rest; before a fused aggregation nothing
  // is kept (that kernel reads G reduced gradients: keeping their ends measured slower)
  ra.keep_from_tile = keep_from_tile(p, with_adamw && p->descending[FLS_KERNEL_ADAMW]);
  const bool speculate = p->speculative && with_adamw;
  const bool single = (p->single_pass || speculate) && with_adamw;
  const bool recompute = p->recompute && with_adamw && !single;   // the fused aggregation needs the stored gradients
  ra.store_gbar = (recompute || single) ? 0 : 1;
  p->gbar_valid = ra.store_gbar != 0;
  const bool f32 = d.grad_dtype == FLS_GRAD_F32;
  const bool overlap = p->overlap && !p->profiling;   // event records between kernels would serialise anyway
  const AdamScalars sc = adam_scalars(d, lr, t_new);
  AdamArgs aa{};
  aa.gbar = p->d_gbar(slot);
  aa.theta = aa.theta_out = p->master[c0];
  aa.m = aa.m_out = p->m[c0];
  aa.v = aa.v_out = p->v[c0];
  aa.pbf16 = p->pbf16[c0];
  aa.idx = ra.idx;
  aa.descending = p->descending[FLS_KERNEL_ADAMW];
  aa.coef = p->d_coefs() + g;
  set_adam_scalars(&aa, sc);
  if (single) {
    // The coefficient is 1 (no clipping) or guessed to be 1 (speculative): one kernel does the whole step of the
    // group.  A speculative step writes the other buffer set and is followed by a kernel that redoes the step with
    // the real coefficient if the guess was wrong; either way the other set holds the new state afterwards.
    ReduceAdamArgs rp{};
    rp.r = ra;
    rp.a = aa;
    if (speculate) {
      rp.r.spec_counts = p->d_spec_counts();
      rp.a.theta_out = p->master2[g];
      rp.a.m_out = p->m2[g];
      rp.a.v_out = p->v2[g];
    }
    cudaError_t e1 = timed_launch(p, FLS_KERNEL_ADAMW, st, [&] { return launch_step_noclip(rp, f32, p->reduce_sg, st, overlap && chain); });
    if (e1 != cudaSuccess) return cuda_fail(e1, "single-pass step kernel launch");
    if (speculate) {
      rp.r.spec_counts = nullptr;
      rp.skip_if_unclipped = 1;
      const unsigned grid = unsigned(std::min<uint64_t>(p->lay.n_tiles, uint64_t(std::max(p->sm_count, 1)) * 8));
      e1 = timed_launch(p, FLS_KERNEL_ADAMW, st, [&] { return launch_reduce_adamw(rp, f32, p->reduce_sg, grid, st, overlap); });
      if (e1 != cudaSuccess) return cuda_fail(e1, "speculative redo kernel launch");
      std::swap(p->master[g], p->master2[g]);
      std::swap(p->m[g], p->m2[g]);
      std::swap(p->v[g], p->v2[g]);
    }
    return FLS_OK;
  }
  cudaError_t e = timed_launch(p, FLS_KERNEL_REDUCE, st, [&] { return launch_reduce(ra, f32, p->reduce_sg, st, overlap && chain); });
  if (e != cudaSuccess) return cuda_fail(e, "reduce kernel launch");
  if (!with_adamw) return FLS_OK;

  if (recompute) {
    ReduceAdamArgs rp{};
    rp.r = ra;
    rp.a = aa;
    e = timed_launch(p, FLS_KERNEL_ADAMW, st,
                     [&] { return launch_reduce_adamw(rp, f32, p->reduce_sg, p->grid_for(FLS_KERNEL_ADAMW), st, overlap); });
    if (e != cudaSuccess) return cuda_fail(e, "adamw kernel launch");
    return FLS_OK;
  }
  // every state copy of the group (one, or one per replica) takes the same update; consecutive passes over the
  // reduced gradient alternate direction so that each starts where the one before stopped
  for (uint32_t r = 0; r < p->R_state; ++r) {
    aa.theta = aa.theta_out = p->master[c0 + r];
    aa.m = aa.m_out = p->m[c0 + r];
    aa.v = aa.v_out = p->v[c0 + r];
    aa.pbf16 = p->pbf16[c0 + r];
    aa.descending = p->descending[FLS_KERNEL_ADAMW] ^ int(r & 1u);
    e = timed_launch(p, FLS_KERNEL_ADAMW, st, [&] { return launch_adamw(aa, p->grid_for(FLS_KERNEL_ADAMW), st, overlap); });
    if (e != cudaSuccess) return cuda_fail(e, "adamw kernel launch");
  }
  return FLS_OK;
}

// All groups in two launches (one reduce grid, one AdamW grid with the groups in the y dimension) instead of two per
// group; with_adamw = false stops after the reduction (fused aggregation).  Same arithmetic, same results.
int run_groups_batched(fls_plan* p, double lr, uint64_t t_new, cudaStream_t st, bool with_adamw) {
  const fls_plan_desc& d = p->desc;
  const uint32_t G = d.groups;
  ReduceArgs ra = common_reduce_args(p);
  for (uint32_t i = 0; i < G * p->K; ++i) ra.grad[i] = p->grads[i];
  ra.gbar = p->d_gbar(0);
  p->last_slot = G - 1;
  p->gbar_valid = true;
  ra.partials = p->d_partials();
  ra.chunk_partials = p->d_chunk_partials();
  ra.chunk_count = p->d_chunk_count();
  ra.ticket = p->d_ticket();
  ra.norm_out = p->d_norms();
  ra.coef_out = p->d_coefs();
  ra.normsq_out = p->d_normsq();
  ra.keep_from_tile = keep_from_tile(p, true);      // small plans: everything fits in L2 anyway
  ra.store_gbar = 1;
  const bool f32 = d.grad_dtype == FLS_GRAD_F32;
  const bool overlap = p->overlap && !p->profiling;
  cudaError_t e = timed_launch(p, FLS_KERNEL_REDUCE, st, [&] { return launch_reduce_batch(ra, f32, p->reduce_sg, G, st, false); });
  if (e != cudaSuccess) return cuda_fail(e, "batched reduce kernel launch");
  if (!with_adamw) return FLS_OK;
  const AdamScalars sc = adam_scalars(d, lr, t_new);
  AdamBatchArgs ab{};
  for (uint32_t g = 0; g < G; ++g) {
    ab.theta[g] = p->master[g];
    ab.m[g] = p->m[g];
    ab.v[g] = p->v[g];
    ab.pbf16[g] = p->pbf16[g];
  }
  ab.gbar = p->d_gbar(0);
  ab.gbar_stride = ra.gbar_stride;
  ab.coef = p->d_coefs();
  ab.idx = ra.idx;
  ab.descending = p->descending[FLS_KERNEL_ADAMW];
  ab.decay = sc.decay; ab.beta1 = sc.beta1; ab.omb1 = sc.omb1; ab.beta2 = sc.beta2; ab.omb2 = sc.omb2;
  ab.step_size = sc.step_size; ab.inv_sqrt_bc2 = sc.inv_sqrt_bc2; ab.eps = sc.eps;
  e = timed_launch(p, FLS_KERNEL_ADAMW, st, [&] { return launch_adamw_batch(ab, p->grid_for(FLS_KERNEL_ADAMW), G, st, overlap); });
  if (e != cudaSuccess) return cuda_fail(e, "batched adamw kernel launch");
  return FLS_OK;
}

// Recompute plans: one grid computes the norms (and clip coefficients) of all groups, then every group's AdamW kernel
// forms the mean gradient again from the gradients.  Same arithmetic as the per-group sequence, G + 1 launches
// instead of 2 G, and the long kernels follow one another directly.
int run_groups_norm_first(fls_plan* p, double lr, uint64_t t_new, cudaStream_t st) {
  const fls_plan_desc& d = p->desc;
  const uint32_t G = d.groups;
  ReduceArgs ra = common_reduce_args(p);
  for (uint32_t i = 0; i < G * p->K; ++i) ra.grad[i] = p->grads[i];
  ra.gbar = p->d_gbar(0);
  ra.store_gbar = 0;
  p->gbar_valid = false;
  ra.partials = p->d_partials();
  ra.chunk_partials = p->d_chunk_partials();
  ra.chunk_count = p->d_chunk_count();
  ra.ticket = p->d_ticket();
  ra.norm_out = p->d_norms();
  ra.coef_out = p->d_coefs();
  ra.normsq_out = p->d_normsq();
  ra.keep_from_tile = uint32_t(p->lay.n_tiles);
  const bool f32 = d.grad_dtype == FLS_GRAD_F32;
  const bool overlap = p->overlap && !p->profiling;
  cudaError_t e = timed_launch(p, FLS_KERNEL_REDUCE, st, [&] { return launch_reduce_batch(ra, f32, p->reduce_sg, G, st, false); });
  if (e != cudaSuccess) return cuda_fail(e, "batched norm kernel launch");
  const AdamScalars sc = adam_scalars(d, lr, t_new);
  for (uint32_t g = 0; g < G; ++g) {
    ReduceAdamArgs rp{};
    rp.r = common_reduce_args(p);
    for (uint32_t k = 0; k < p->K; ++k) rp.r.grad[k] = p->grads[size_t(g) * p->K + k];
    rp.a.theta = rp.a.theta_out = p->master[g];
    rp.a.m = rp.a.m_out = p->m[g];
    rp.a.v = rp.a.v_out = p->v[g];
    rp.a.pbf16 = p->pbf16[g];
    rp.a.idx = rp.r.idx;
    rp.a.descending = p->descending[FLS_KERNEL_ADAMW];
    rp.a.coef = p->d_coefs() + g;
    set_adam_scalars(&rp.a, sc);
    e = timed_launch(p, FLS_KERNEL_ADAMW, st,
                     [&] { return launch_reduce_adamw(rp, f32, p->reduce_sg, p->grid_for(FLS_KERNEL_ADAMW), st, overlap); });
    if (e != cudaSuccess) return cuda_fail(e, "adamw kernel launch");
  }
  return FLS_OK;
}

// Tiles per CTA and grid.x with which the resident step fits the current device: the smallest number of tiles per CTA
// (8 KB of shared memory each) for which all G * ceil(n_tiles / T) CTAs can be resident at once; 0, 0 if none does.
void plan_resident_shape(fls_plan* p) {
  p->res_tiles = p->res_grid = 0;
  if (!resident_shape_ok(p->K, p->reduce_sg) || p->lay.n_tiles == 0) return;
  const bool f32 = p->desc.grad_dtype == FLS_GRAD_F32;
  for (uint32_t T = 1; T <= 27; ++T) {
    unsigned cap = 0;
    if (resident_max_ctas(f32, p->K, p->reduce_sg, size_t(T) * kTile * 4, p->sm_count, &cap) != cudaSuccess) {
      cudaGetLastError();
      return;
    }
    if (cap == 0) return;
    const uint64_t gx = (p->lay.n_tiles + T - 1) / T;
    if (gx * p->desc.groups <= cap) {
      p->res_tiles = T;
      p->res_grid = uint32_t(gx);
      return;
    }
  }
}

// The step of all groups as one cooperative kernel (see fls_plan_set_resident).
int run_resident(fls_plan* p, double lr, uint64_t t_new, cudaStream_t st, bool* fell_back) {
  *fell_back = false;
  const fls_plan_desc& d = p->desc;
  const uint32_t G = d.groups;
  ResidentArgs a{};
  a.r = common_reduce_args(p);
  for (uint32_t i = 0; i < G * p->K; ++i) a.r.grad[i] = p->grads[i];
  a.r.gbar = nullptr;
  a.r.store_gbar = 0;
  p->gbar_valid = false;
  a.r.partials = p->d_partials();
  a.r.chunk_partials = p->d_chunk_partials();
  a.r.chunk_count = p->d_chunk_count();
  a.r.ticket = p->d_ticket();
  a.r.norm_out = p->d_norms();
  a.r.coef_out = p->d_coefs();
  a.r.normsq_out = p->d_normsq();
  a.r.keep_from_tile = uint32_t(p->lay.n_tiles);
  if (++p->res_seq == 0) p->res_seq = 1;            // the ready words start at zero
  a.r.launch_id = p->res_seq;
  a.r.ready = p->d_ready();
  for (uint32_t g = 0; g < G; ++g) {
    a.theta[g] = p->master[g];
    a.m[g] = p->m[g];
    a.v[g] = p->v[g];
    a.pbf16[g] = p->pbf16[g];
  }
  const AdamScalars sc = adam_scalars(d, lr, t_new);
  a.decay = sc.decay; a.beta1 = sc.beta1; a.omb1 = sc.omb1; a.beta2 = sc.beta2; a.omb2 = sc.omb2;
  a.step_size = sc.step_size; a.inv_sqrt_bc2 = sc.inv_sqrt_bc2; a.eps = sc.eps;
  a.tiles_per_cta = p->res_tiles;
  a.wait_limit = p->res_wait_limit;
  // test hook (one launch): the waiters expect an id that nobody publishes, so every wait runs out
  a.expect_id = p->res_hold_back ? (a.r.launch_id ^ 0x80000000u) : a.r.launch_id;
  p->res_hold_back = false;
  const bool f32 = d.grad_dtype == FLS_GRAD_F32;
  cudaError_t e = timed_launch(p, FLS_KERNEL_ADAMW, st,
                               [&] { return launch_step_resident(a, f32, p->reduce_sg, p->res_grid, G, st); });
  if (e == cudaErrorCooperativeLaunchTooLarge) {
    // the device would not hold the grid after all (its occupancy differs from what bind computed): nothing ran;
    // give the route up for this binding and let the caller take the usual one
    cudaGetLastError();
    p->res_tiles = p->res_grid = 0;
    *fell_back = true;
    return FLS_OK;
  }
  if (e != cudaSuccess) return cuda_fail(e, "resident step kernel launch");
  return FLS_OK;
}

// Every range must be non-null, aligned device memory of the current device.  Outputs may overlap nothing;
// gradient buffers may only overlap each other (a caller may feed one buffer to several replicas).
int check_ranges(const std::vector<Range>& ranges, int dev) {
  for (const Range& r : ranges) {
    if (r.lo == 0) return fail(FLS_EPTR, "%s[%d] is null", r.what, r.index);
    if (r.lo % FLS_BUFFER_ALIGN != 0) return fail(FLS_EALIGN, "%s[%d] is not %d-byte aligned", r.what, r.index, FLS_BUFFER_ALIGN);
    cudaPointerAttributes attr{};
    cudaError_t e = cudaPointerGetAttributes(&attr, reinterpret_cast<const void*>(r.lo));
    if (e != cudaSuccess) {
      cudaGetLastError();
      return fail(FLS_EPTR, "%s[%d]: %s", r.what, r.index, cudaGetErrorString(e));
    }
    if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged)
      return fail(FLS_EPTR, "%s[%d] is not device memory", r.what, r.index);
    if (attr.type == cudaMemoryTypeDevice && attr.device != dev)
      return fail(FLS_EPTR, "%s[%d] lives on device %d, current device is %d", r.what, r.index, attr.device, dev);
  }
  std::vector<size_t> order(ranges.size());
  for (size_t i = 0; i < order.size(); ++i) order[i] = i;
  std::sort(order.begin(), order.end(), [&](size_t x, size_t y) { return ranges[x].lo < ranges[y].lo; });
  for (size_t q = 0; q < order.size(); ++q) {
    const Range& r0 = ranges[order[q]];
    for (size_t w = q + 1; w < order.size() && ranges[order[w]].lo < r0.hi; ++w) {
      const Range& r1 = ranges[order[w]];
      if (r0.output || r1.output)
        return fail(FLS_EPTR, "%s[%d] overlaps %s[%d]", r0.what, r0.index, r1.what, r1.index);
    }
  }
  return FLS_OK;
}

bool step_preamble(fls_plan* p, double* lr) {
  if (std::isnan(*lr)) *lr = p->desc.lr;
  return *lr >= 0.0 && std::isfinite(*lr);
}

}  // namespace

namespace fls {
void set_last_error(const char* msg) { g_err = msg ? msg : ""; }
}  // namespace fls

extern "C" {

const char* fls_last_error(void) { return g_err.c_str(); }

int fls_plan_create(const fls_plan_desc* desc, fls_plan** out) {
  if (out) *out = nullptr;
  if (!desc || !out) return fail(FLS_EINVAL, "fls_plan_create: null argument");
  const fls_plan_desc& d = *desc;
  if (d.groups == 0 || d.shard_dim == 0 || d.replicate_dim == 0 || d.sync_period == 0 || d.align_elems == 0)
    return fail(FLS_EINVAL, "groups, shard_dim, replicate_dim, sync_period and align_elems must be >= 1");
  if (d.groups > FLS_MAX_GROUPS) return fail(FLS_EINVAL, "groups = %u exceeds %d", d.groups, FLS_MAX_GROUPS);
  const uint64_t K = uint64_t(d.shard_dim) * d.replicate_dim;
  if (K > FLS_MAX_GRAD_BUFFERS)
    return fail(FLS_EINVAL, "shard_dim*replicate_dim = %llu exceeds %d", (unsigned long long)K, FLS_MAX_GRAD_BUFFERS);
  if (d.grad_dtype != FLS_GRAD_BF16 && d.grad_dtype != FLS_GRAD_F32) return fail(FLS_EINVAL, "unknown grad_dtype %u", d.grad_dtype);
  if (!(d.fedavg_what & FLS_AVG_PARAMS) || (d.fedavg_what & ~uint32_t(FLS_AVG_PARAMS | FLS_AVG_OPT_STATE | FLS_AVG_FUSED)))
    return fail(FLS_EINVAL, "fedavg_what must be FLS_AVG_PARAMS, optionally | FLS_AVG_OPT_STATE | FLS_AVG_FUSED");
  if (d.reduce_wire != FLS_WIRE_F32 && d.reduce_wire != FLS_WIRE_BF16) return fail(FLS_EINVAL, "unknown reduce_wire %u", d.reduce_wire);
  if (d.reduce_wire == FLS_WIRE_BF16 && d.grad_dtype != FLS_GRAD_BF16)
    return fail(FLS_EINVAL, "FLS_WIRE_BF16 needs bf16 gradients");
  if (d.reduce_order != FLS_ORDER_ASCENDING && d.reduce_order != FLS_ORDER_RING) return fail(FLS_EINVAL, "unknown reduce_order %u", d.reduce_order);
  if (d.state_copies != FLS_STATE_PER_GROUP && d.state_copies != FLS_STATE_PER_REPLICA)
    return fail(FLS_EINVAL, "unknown state_copies %u", d.state_copies);
  if (d.state_copies == FLS_STATE_PER_REPLICA && uint64_t(d.groups) * d.replicate_dim > FLS_MAX_STATE_COPIES)
    return fail(FLS_EINVAL, "groups*replicate_dim = %llu exceeds %d state copies", (unsigned long long)(uint64_t(d.groups) * d.replicate_dim),
                FLS_MAX_STATE_COPIES);
  if (!(d.beta1 >= 0.0 && d.beta1 < 1.0) || !(d.beta2 >= 0.0 && d.beta2 < 1.0)) return fail(FLS_EINVAL, "betas must lie in [0, 1)");
  if (!(d.eps > 0.0) || !std::isfinite(d.eps)) return fail(FLS_EINVAL, "eps must be positive");
  if (!(d.lr >= 0.0) || !std::isfinite(d.lr)) return fail(FLS_EINVAL, "lr must be finite and >= 0");
  if (!std::isfinite(d.weight_decay) || d.weight_decay < 0.0) return fail(FLS_EINVAL, "weight_decay must be finite and >= 0");
  if (std::isnan(d.max_grad_norm)) return fail(FLS_EINVAL, "max_grad_norm is NaN");
  if (d.n_params == 0) return fail(FLS_EINVAL, "n_params must be >= 1");

  std::vector<uint64_t> units;
  if (d.n_units == 0 && d.unit_numel == nullptr) {
    units.push_back(d.n_params);
  } else {
    if (d.n_units == 0 || d.unit_numel == nullptr) return fail(FLS_EINVAL, "n_units and unit_numel must be given together");
    units.assign(d.unit_numel, d.unit_numel + d.n_units);
  }
  unsigned __int128 sum = 0;
  for (uint64_t n : units) sum += n;
  if (sum != d.n_params) return fail(FLS_EINVAL, "sum(unit_numel) differs from n_params");

  fls_plan* p = new (std::nothrow) fls_plan();
  if (!p) return fail(FLS_EINVAL, "out of host memory");
  p->desc = d;
  p->units = units;
  p->desc.unit_numel = nullptr;   // the caller's table is not kept; p->units is the copy
  p->desc.n_units = uint32_t(units.size());
  p->ring = d.reduce_order == FLS_ORDER_RING;
  p->R_state = d.state_copies == FLS_STATE_PER_REPLICA ? d.replicate_dim : 1;
  p->n_copies = d.groups * p->R_state;
  const bool fused = (d.fedavg_what & FLS_AVG_FUSED) && d.groups <= FLS_MAX_FUSED_GROUPS &&
                     uint64_t(d.groups) * (p->R_state - 1) <= uint64_t(FLS_MAX_FUSED_EXTRA);
  // one reduced-gradient slot per group for the fused aggregation and for small plans (whose groups share a grid)
  unsigned __int128 padded_bound = 0;
  for (uint64_t n : units) padded_bound += n + uint64_t(d.shard_dim) * d.align_elems;
  const bool small = padded_bound * 4 * d.groups <= kBatchScratchBytes;
  p->fused_plan = fused;
  const std::string msg = build_layout(units, d.shard_dim, d.align_elems, (fused || small) ? d.groups : 1, p->ring ? d.replicate_dim : 0,
                                       d.groups, &p->lay);
  if (!msg.empty()) {
    delete p;
    return fail(FLS_EINVAL, "layout: %s", msg.c_str());
  }
  p->K = uint32_t(K);
  // level structure of the gradient reduction: which buffers / batches of 8 close a sharding group
  for (uint32_t k = 0; k < p->K; ++k)
    if (k % d.shard_dim == d.shard_dim - 1) p->end_mask |= 1ull << k;
  const uint32_t S = d.shard_dim;
  if (d.replicate_dim == 1 || S % 8 == 0) {
    p->reduce_sg = 0;
    for (uint32_t k0 = 0; k0 < p->K; k0 += 8)
      if (std::min(k0 + 8, p->K) % S == 0) p->fold_mask |= 1u << (k0 / 8);
  } else if (S == 1 || S == 2 || S == 4) {
    p->reduce_sg = int(S);
  } else {
    p->reduce_sg = -1;
  }
  if (p->ring) p->reduce_sg = -1;                          // generic kernel: the visiting order depends on the element
  if (d.reduce_wire == FLS_WIRE_BF16) p->reduce_sg = -2;   // generic kernel, bf16 rounding after every sum
  // fewer than 8 gradient bytes per element: a second read of the gradients costs less than the fp32 round trip
  p->recompute = p->plain_reduce() && K * (d.grad_dtype == FLS_GRAD_F32 ? 4 : 2) < 8;
  // without clipping the coefficient is 1 whatever the norm: the step needs no second pass at all
  p->single_pass = p->plain_reduce() && !(d.max_grad_norm > 0.0);
  *out = p;
  return FLS_OK;
}

int fls_plan_query(const fls_plan* plan, fls_layout* out) {
  if (!plan || !out) return fail(FLS_EINVAL, "fls_plan_query: null argument");
  out->n_padded = plan->lay.n_padded;
  out->shard_numel = plan->lay.shard_numel;
  out->n_units = uint32_t(plan->units.size());
  out->grad_buffers = plan->K;
  out->unit_offset = plan->lay.unit_offset.data();
  out->unit_shard_numel = plan->lay.unit_shard_numel.data();
  out->unit_shard_offset = plan->lay.unit_shard_offset.data();
  out->workspace_bytes = plan->lay.workspace_bytes;
  out->n_segments = uint32_t(plan->lay.segments.size());
  out->vector_path = plan->lay.vector_path ? 1u : 0u;
  out->n_state_copies = plan->n_copies;
  out->reserved = 0;
  return FLS_OK;
}

int fls_plan_bind(fls_plan* p, const fls_buffers* b) {
  if (!p || !b) return fail(FLS_EINVAL, "fls_plan_bind: null argument");
  if (!b->grads || !b->master || !b->m || !b->v || !b->param_bf16 || !b->workspace)
    return fail(FLS_EPTR, "fls_plan_bind: null pointer table or workspace");
  if (b->workspace_bytes < p->lay.workspace_bytes)
    return fail(FLS_ESIZE, "workspace has %llu bytes, %llu needed", (unsigned long long)b->workspace_bytes,
                (unsigned long long)p->lay.workspace_bytes);
  const uint32_t G = p->desc.groups, K = p->K, C = p->n_copies;
  const uint64_t N = p->lay.n_padded;
  const uint64_t eg = p->desc.grad_dtype == FLS_GRAD_F32 ? 4 : 2;

  std::vector<Range> ranges;
  auto add = [&](const void* ptr, uint64_t bytes, const char* what, int idx, bool output) {
    ranges.push_back(Range{reinterpret_cast<uintptr_t>(ptr), reinterpret_cast<uintptr_t>(ptr) + bytes, what, idx, output});
  };
  for (uint32_t i = 0; i < G * K; ++i) add(b->grads[i], N * eg, "grads", int(i), false);
  for (uint32_t g = 0; g < C; ++g) {
    add(b->master[g], N * 4, "master", int(g), true);
    add(b->m[g], N * 4, "m", int(g), true);
    add(b->v[g], N * 4, "v", int(g), true);
    add(b->param_bf16[g], N * 2, "param_bf16", int(g), true);
  }
  add(b->workspace, p->lay.workspace_bytes, "workspace", 0, true);

  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
  int rc = check_ranges(ranges, dev);
  if (rc != FLS_OK) return rc;

  int sms = 0;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
  p->device = dev;
  p->sm_count = sms;
  p->grads.assign(b->grads, b->grads + size_t(G) * K);
  p->master.assign(b->master, b->master + C);
  p->m.assign(b->m, b->m + C);
  p->v.assign(b->v, b->v + C);
  p->pbf16.resize(C);
  for (uint32_t g = 0; g < C; ++g) p->pbf16[g] = static_cast<uint16_t*>(b->param_bf16[g]);
  p->ws = static_cast<char*>(b->workspace);
  p->ranges = ranges;
  p->master2.clear(); p->m2.clear(); p->v2.clear();   // a new binding drops the second buffer set
  p->speculative = false;
  p->res_seq = 0;                  // the ready words are zeroed below
  plan_resident_shape(p);

  e = cudaMemset(p->ws, 0, size_t(kWsSegments));
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemset(workspace head)");
  e = cudaMemset(p->ws + p->lay.ws_chunk_count_offset, 0, size_t(p->lay.ws_chunk_count_bytes));
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemset(norm counters)");
  e = cudaMemcpy(p->ws + kWsSegments, p->lay.segments.data(), p->lay.segments.size() * sizeof(Segment), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy(segment table)");
  e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceSynchronize");
  if (!p->copy_stream) {
    e = cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamCreate");
    e = cudaEventCreateWithFlags(&p->ev_begin, cudaEventDisableTiming);
    if (e != cudaSuccess) return cuda_fail(e, "cudaEventCreate");
    p->ev_copied.resize(G, nullptr);
    for (uint32_t g = 0; g < G; ++g) {
      e = cudaEventCreateWithFlags(&p->ev_copied[g], cudaEventDisableTiming);
      if (e != cudaSuccess) return cuda_fail(e, "cudaEventCreate");
    }
  }
  p->bound = true;
  return FLS_OK;
}

int fls_sync_step(fls_plan* p, double lr, void* cuda_stream, int* fedavg_due) {
  if (!p) return fail(FLS_EINVAL, "fls_sync_step: null plan");
  if (!p->bound) return fail(FLS_ESTATE, "fls_sync_step: plan has no buffers bound");
  if (!step_preamble(p, &lr)) return fail(FLS_EINVAL, "fls_sync_step: lr must be finite and >= 0");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const uint64_t t_new = p->step + 1;
  bool fell_back = true;
  if (p->resident()) {
    const int rc = run_resident(p, lr, t_new, st, &fell_back);
    if (rc != FLS_OK) return rc;
  }
  if (!fell_back) {
    // done: the resident kernel did the whole step
  } else if (p->batching()) {
    const int rc = run_groups_batched(p, lr, t_new, st, true);
    if (rc != FLS_OK) return rc;
  } else if (p->norm_first()) {
    const int rc = run_groups_norm_first(p, lr, t_new, st);
    if (rc != FLS_OK) return rc;
  } else {
    for (uint32_t g = 0; g < p->desc.groups; ++g) {
      const int rc = run_group(p, g, lr, t_new, st, g > 0);
      if (rc != FLS_OK) return rc;
    }
  }
  p->step = t_new;
  if (fedavg_due) *fedavg_due = (t_new % p->desc.sync_period == 0) ? 1 : 0;
  return FLS_OK;
}

int fls_sync_step_host(fls_plan* p, const void* const* host_grads, double lr, void* cuda_stream, float* host_norms,
                       int* fedavg_due) {
  if (!p || !host_grads) return fail(FLS_EINVAL, "fls_sync_step_host: null argument");
  if (!p->bound) return fail(FLS_ESTATE, "fls_sync_step_host: plan has no buffers bound");
  if (!step_preamble(p, &lr)) return fail(FLS_EINVAL, "fls_sync_step_host: lr must be finite and >= 0");
  const uint32_t G = p->desc.groups, K = p->K;
  for (uint32_t i = 0; i < G * K; ++i)
    if (!host_grads[i]) return fail(FLS_EPTR, "host_grads[%u] is null", i);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const uint64_t bytes = p->lay.n_padded * (p->desc.grad_dtype == FLS_GRAD_F32 ? 4ull : 2ull);
  const uint64_t t_new = p->step + 1;
  // the copies may not overtake work already queued on the caller's stream that still reads the buffers
  cudaError_t e = cudaEventRecord(p->ev_begin, st);
  if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
  e = cudaStreamWaitEvent(p->copy_stream, p->ev_begin, 0);
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamWaitEvent");
  for (uint32_t g = 0; g < G; ++g) {
    for (uint32_t k = 0; k < K; ++k) {
      e = cudaMemcpyAsync(const_cast<void*>(p->grads[size_t(g) * K + k]), host_grads[size_t(g) * K + k], bytes,
                          cudaMemcpyHostToDevice, p->copy_stream);
      if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(host gradients)");
    }
    e = cudaEventRecord(p->ev_copied[g], p->copy_stream);
    if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    e = cudaStreamWaitEvent(st, p->ev_copied[g], 0);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamWaitEvent");
    const int rc = run_group(p, g, lr, t_new, st, false);   // an event wait precedes every group here
    if (rc != FLS_OK) return rc;
  }
  if (host_norms) {
    e = cudaMemcpyAsync(host_norms, p->d_norms(), sizeof(float) * G, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(norms)");
  }
  e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  p->step = t_new;
  if (fedavg_due) *fedavg_due = (t_new % p->desc.sync_period == 0) ? 1 : 0;
  return FLS_OK;
}

namespace {
struct OuterOpt { float* x_global; float* buf; double lr, momentum; int nesterov; };

int fedavg_impl(fls_plan* p, const uint64_t* sample_counts, void* cuda_stream, const OuterOpt* outer, const char* who) {
  const uint32_t G = p->desc.groups;
  long double total = 0;
  for (uint32_t g = 0; g < G; ++g) total += sample_counts ? (long double)sample_counts[g] : 1.0L;
  if (!(total > 0)) return fail(FLS_EINVAL, "%s: all sample counts are zero", who);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  FedavgArgs fa{};
  for (uint32_t g = 0; g < G; ++g) {
    const double n = sample_counts ? double(sample_counts[g]) : 1.0;
    fa.w[g] = float(n / double(total));
  }
  fa.idx = p->seg_index();
  fa.G = G;
  fa.descending = p->descending[FLS_KERNEL_FEDAVG];
  const int n_arrays = (p->desc.fedavg_what & FLS_AVG_OPT_STATE) ? 3 : 1;
  // with one state copy per replica only the first replica of every group aggregates; the others receive the result
  const uint32_t R = p->R_state;
  fa.n_extra = G * (R - 1);
  for (int arr = 0; arr < n_arrays; ++arr) {
    const std::vector<float*>& src = arr == 0 ? p->master : (arr == 1 ? p->m : p->v);
    for (uint32_t g = 0; g < G; ++g) {
      fa.x[g] = src[g * R];
      fa.pbf16[g] = p->pbf16[g * R];
      for (uint32_t r = 1; r < R; ++r) {
        fa.x_extra[g * (R - 1) + r - 1] = src[g * R + r];
        fa.pbf16_extra[g * (R - 1) + r - 1] = p->pbf16[g * R + r];
      }
    }
    fa.write_bf16 = arr == 0 ? 1 : 0;
    const bool use_outer = outer && arr == 0;       // the outer optimizer acts on the parameters only
    fa.x_global = use_outer ? outer->x_global : nullptr;
    fa.outer_buf = use_outer ? outer->buf : nullptr;
    fa.outer_lr = use_outer ? float(outer->lr) : 0.f;
    fa.momentum = use_outer ? float(outer->momentum) : 0.f;
    fa.nesterov = use_outer ? outer->nesterov : 0;
    const bool overlap = p->overlap && !p->profiling && arr > 0;
    cudaError_t e = timed_launch(p, FLS_KERNEL_FEDAVG, st, [&] { return launch_fedavg(fa, p->grid_for(FLS_KERNEL_FEDAVG), st, overlap); });
    if (e != cudaSuccess) return cuda_fail(e, "fedavg kernel launch");
  }
  return FLS_OK;
}
}  // namespace

int fls_fedavg(fls_plan* p, const uint64_t* sample_counts, void* cuda_stream) {
  if (!p) return fail(FLS_EINVAL, "fls_fedavg: null plan");
  if (!p->bound) return fail(FLS_ESTATE, "fls_fedavg: plan has no buffers bound");
  return fedavg_impl(p, sample_counts, cuda_stream, nullptr, "fls_fedavg");
}

int fls_fedavg_outer(fls_plan* p, const uint64_t* sample_counts, double outer_lr, double momentum, int nesterov,
                     float* global_params, float* outer_momentum, void* cuda_stream) {
  if (!p) return fail(FLS_EINVAL, "fls_fedavg_outer: null plan");
  if (!p->bound) return fail(FLS_ESTATE, "fls_fedavg_outer: plan has no buffers bound");
  if (!global_params || !outer_momentum) return fail(FLS_EPTR, "fls_fedavg_outer: null buffer");
  if (reinterpret_cast<uintptr_t>(global_params) % FLS_BUFFER_ALIGN || reinterpret_cast<uintptr_t>(outer_momentum) % FLS_BUFFER_ALIGN)
    return fail(FLS_EALIGN, "fls_fedavg_outer: buffers must be %d-byte aligned", FLS_BUFFER_ALIGN);
  if (global_params == outer_momentum) return fail(FLS_EPTR, "fls_fedavg_outer: the two buffers are the same");
  if (!std::isfinite(outer_lr) || !std::isfinite(momentum)) return fail(FLS_EINVAL, "fls_fedavg_outer: outer_lr and momentum must be finite");
  const OuterOpt o{global_params, outer_momentum, outer_lr, momentum, nesterov ? 1 : 0};
  return fedavg_impl(p, sample_counts, cuda_stream, &o, "fls_fedavg_outer");
}

int fls_sync_step_fedavg(fls_plan* p, double lr, const uint64_t* sample_counts, void* cuda_stream) {
  if (!p) return fail(FLS_EINVAL, "fls_sync_step_fedavg: null plan");
  if (!p->bound) return fail(FLS_ESTATE, "fls_sync_step_fedavg: plan has no buffers bound");
  const uint32_t G = p->desc.groups;
  if (!p->fused_plan || p->resident()) {   // not planned for fusion, or the step runs as one resident kernel: the two calls in sequence give the same result
    const int rc = fls_sync_step(p, lr, cuda_stream, nullptr);
    return rc != FLS_OK ? rc : fls_fedavg(p, sample_counts, cuda_stream);
  }
  if (!step_preamble(p, &lr)) return fail(FLS_EINVAL, "fls_sync_step_fedavg: lr must be finite and >= 0");
  long double total = 0;
  for (uint32_t g = 0; g < G; ++g) total += sample_counts ? (long double)sample_counts[g] : 1.0L;
  if (!(total > 0)) return fail(FLS_EINVAL, "fls_sync_step_fedavg: all sample counts are zero");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const uint64_t t_new = p->step + 1;
  if (p->batching()) {
    const int rc = run_groups_batched(p, lr, t_new, st, false);
    if (rc != FLS_OK) return rc;
  } else {
    for (uint32_t g = 0; g < G; ++g) {
      const int rc = run_group(p, g, lr, t_new, st, g > 0, g, false);
      if (rc != FLS_OK) return rc;
    }
  }
  const AdamScalars sc = adam_scalars(p->desc, lr, t_new);
  FusedArgs fa{};
  const uint32_t R = p->R_state;
  fa.replicas = R;
  for (uint32_t g = 0; g < G; ++g) {
    fa.gbar[g] = p->d_gbar(g);
    fa.theta[g] = p->master[g * R];
    fa.m[g] = p->m[g * R];
    fa.v[g] = p->v[g * R];
    fa.pbf16[g] = p->pbf16[g * R];
    fa.w[g] = float((sample_counts ? double(sample_counts[g]) : 1.0) / double(total));
    for (uint32_t r = 1; r < R; ++r) {
      const uint32_t i = g * (R - 1) + r - 1;
      fa.theta_extra[i] = p->master[g * R + r];
      fa.m_extra[i] = p->m[g * R + r];
      fa.v_extra[i] = p->v[g * R + r];
      fa.pbf16_extra[i] = p->pbf16[g * R + r];
    }
  }
  fa.coefs = p->d_coefs();
  fa.idx = p->seg_index();
  fa.G = G;
  fa.avg_opt_state = (p->desc.fedavg_what & FLS_AVG_OPT_STATE) ? 1 : 0;
  fa.descending = p->descending[FLS_KERNEL_ADAMW_FEDAVG];
  fa.decay = sc.decay; fa.beta1 = sc.beta1; fa.omb1 = sc.omb1; fa.beta2 = sc.beta2; fa.omb2 = sc.omb2;
  fa.step_size = sc.step_size; fa.inv_sqrt_bc2 = sc.inv_sqrt_bc2; fa.eps = sc.eps;
  const bool overlap = p->overlap && !p->profiling;
  cudaError_t e = timed_launch(p, FLS_KERNEL_ADAMW_FEDAVG, st,
                               [&] { return launch_adamw_fedavg(fa, p->grid_for(FLS_KERNEL_ADAMW_FEDAVG), st, overlap); });
  if (e != cudaSuccess) return cuda_fail(e, "fused adamw+fedavg kernel launch");
  p->step = t_new;
  return FLS_OK;
}

int fls_get_norms(const fls_plan* p, const float** dev_norms, const float** dev_coefs) {
  if (!p) return fail(FLS_EINVAL, "fls_get_norms: null plan");
  if (!p->bound) return fail(FLS_ESTATE, "fls_get_norms: plan has no buffers bound");
  if (dev_norms) *dev_norms = p->d_norms();
  if (dev_coefs) *dev_coefs = p->d_coefs();
  return FLS_OK;
}

int fls_get_reduced_grad(const fls_plan* p, const float** dev_gbar) {
  if (!p || !dev_gbar) return fail(FLS_EINVAL, "fls_get_reduced_grad: null argument");
  if (!p->bound) return fail(FLS_ESTATE, "fls_get_reduced_grad: plan has no buffers bound");
  if (!p->gbar_valid) return fail(FLS_ESTATE, "fls_get_reduced_grad: the last step did not store the reduced gradient (recompute or single-pass plan)");
  *dev_gbar = p->d_gbar(p->last_slot);
  return FLS_OK;
}

int fls_get_status(const fls_plan* p, const uint32_t** dev_status) {
  if (!p || !dev_status) return fail(FLS_EINVAL, "fls_get_status: null argument");
  if (!p->bound) return fail(FLS_ESTATE, "fls_get_status: plan has no buffers bound");
  *dev_status = p->d_status();
  return FLS_OK;
}

int fls_get_step(const fls_plan* p, uint64_t* t) {
  if (!p || !t) return fail(FLS_EINVAL, "fls_get_step: null argument");
  *t = p->step;
  return FLS_OK;
}

int fls_set_step(fls_plan* p, uint64_t t) {
  if (!p) return fail(FLS_EINVAL, "fls_set_step: null plan");
  p->step = t;
  return FLS_OK;
}

int fls_comm_report(const fls_plan* p, const double* bw, fls_comm_costs* out) {
  if (!p || !out) return fail(FLS_EINVAL, "fls_comm_report: null argument");
  if (bw)
    for (int i = 0; i < 3; ++i)
      if (!(bw[i] > 0.0)) return fail(FLS_EINVAL, "fls_comm_report: bandwidths must be positive");
  comm_report(p->lay, p->desc, p->route(), bw, out);
  return FLS_OK;
}

int fls_plan_tune(fls_plan* p, uint32_t kernel, int ctas_per_sm, int descending) {
  if (!p || kernel >= FLS_KERNEL_COUNT) return fail(FLS_EINVAL, "fls_plan_tune: bad argument");
  if (ctas_per_sm > 0) p->ctas_per_sm[kernel] = std::min(ctas_per_sm, 1 << 16);
  if (ctas_per_sm == -2) p->ctas_per_sm[kernel] = 0;   // back to the default: one pass, the grid covers every tile
  if (descending >= 0) p->descending[kernel] = descending ? 1 : 0;
  return FLS_OK;
}

int fls_plan_set_recompute(fls_plan* p, int mode) {
  if (!p) return fail(FLS_EINVAL, "fls_plan_set_recompute: null plan");
  const fls_plan_desc& d = p->desc;
  const bool small = uint64_t(p->K) * (d.grad_dtype == FLS_GRAD_F32 ? 4 : 2) < 8;
  if (mode > 0 && (!small || !p->plain_reduce()))
    return fail(FLS_ESTATE, "fls_plan_set_recompute: only for K*e_g < 8 bytes, fp32 partial sums in ascending order and one state copy per group");
  p->recompute = mode > 0 || (mode < 0 && small && p->plain_reduce());
  return FLS_OK;
}

int fls_plan_set_single_pass(fls_plan* p, int mode) {
  if (!p) return fail(FLS_EINVAL, "fls_plan_set_single_pass: null plan");
  const bool can = p->plain_reduce() && !(p->desc.max_grad_norm > 0.0);
  if (mode > 0 && !can)
    return fail(FLS_ESTATE, "fls_plan_set_single_pass: only for plans without clipping, with fp32 partial sums in ascending order and one state copy per group");
  p->single_pass = mode > 0 || (mode < 0 && can);
  return FLS_OK;
}

int fls_plan_bind_shadow(fls_plan* p, float* const* master, float* const* m, float* const* v) {
  if (!p || !master || !m || !v) return fail(FLS_EINVAL, "fls_plan_bind_shadow: null argument");
  if (!p->bound) return fail(FLS_ESTATE, "fls_plan_bind_shadow: bind the plan's buffers first");
  if (p->R_state != 1) return fail(FLS_ESTATE, "fls_plan_bind_shadow: not for plans with one state copy per replica");
  const uint32_t G = p->desc.groups;
  const uint64_t N = p->lay.n_padded;
  std::vector<Range> ranges = p->ranges;
  for (uint32_t g = 0; g < G; ++g) {
    const float* ptrs[3] = {master[g], m[g], v[g]};
    const char* names[3] = {"shadow master", "shadow m", "shadow v"};
    for (int i = 0; i < 3; ++i)
      ranges.push_back(Range{reinterpret_cast<uintptr_t>(ptrs[i]), reinterpret_cast<uintptr_t>(ptrs[i]) + N * 4, names[i], int(g), true});
  }
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
  if (dev != p->device) return fail(FLS_ESTATE, "fls_plan_bind_shadow: the plan was bound on device %d, current device is %d", p->device, dev);
  const int rc = check_ranges(ranges, dev);
  if (rc != FLS_OK) return rc;
  p->master2.assign(master, master + G);
  p->m2.assign(m, m + G);
  p->v2.assign(v, v + G);
  return FLS_OK;
}

int fls_plan_set_speculative(fls_plan* p, int enabled) {
  if (!p) return fail(FLS_EINVAL, "fls_plan_set_speculative: null plan");
  if (enabled) {
    if (!p->bound || p->master2.empty()) return fail(FLS_ESTATE, "fls_plan_set_speculative: needs fls_plan_bind_shadow first");
    if (!(p->desc.max_grad_norm > 0.0)) return fail(FLS_ESTATE, "fls_plan_set_speculative: the plan does not clip (it already runs a single pass)");
    if (!p->plain_reduce())
      return fail(FLS_ESTATE, "fls_plan_set_speculative: only with fp32 partial sums in ascending order and one state copy per group");
  }
  p->speculative = enabled != 0;
  return FLS_OK;
}

int fls_get_spec_stats(const fls_plan* p, const uint32_t** dev_counts) {
  if (!p || !dev_counts) return fail(FLS_EINVAL, "fls_get_spec_stats: null argument");
  if (!p->bound) return fail(FLS_ESTATE, "fls_get_spec_stats: plan has no buffers bound");
  *dev_counts = p->d_spec_counts();
  return FLS_OK;
}

int fls_get_state(const fls_plan* p, uint32_t copy, float** master, float** m, float** v) {
  if (!p) return fail(FLS_EINVAL, "fls_get_state: null plan");
  if (!p->bound) return fail(FLS_ESTATE, "fls_get_state: plan has no buffers bound");
  if (copy >= p->n_copies) return fail(FLS_EINVAL, "fls_get_state: copy %u of %u", copy, p->n_copies);
  if (master) *master = p->master[copy];
  if (m) *m = p->m[copy];
  if (v) *v = p->v[copy];
  return FLS_OK;
}

int fls_plan_set_batching(fls_plan* p, int mode) {
  if (!p) return fail(FLS_EINVAL, "fls_plan_set_batching: null plan");
  if (mode > 0 && !p->can_batch() && !p->can_norm_first())
    return fail(FLS_ESTATE, "fls_plan_set_batching: needs G > 1, G*K <= 64, K = 4 or 8 in a flat or 1/2/4-wide two-level order, the default "
                            "two-pass route, one state copy per group and a reduced-gradient slot per group (FLS_AVG_FUSED, or a small plan); "
                            "or a recompute plan with G > 1 and K = 1 or 2");
  p->batch_mode = mode < 0 ? -1 : (mode > 0 ? 1 : 0);
  return FLS_OK;
}

int fls_plan_get_batching(const fls_plan* p, int* active) {
  if (!p || !active) return fail(FLS_EINVAL, "fls_plan_get_batching: null argument");
  *active = (p->batching() || p->norm_first()) && !p->resident() ? 1 : 0;     // the resident step, where it applies, comes first
  return FLS_OK;
}

int fls_plan_set_resident(fls_plan* p, int mode, uint32_t wait_limit) {
  if (!p) return fail(FLS_EINVAL, "fls_plan_set_resident: null plan");
  if (mode > 0 && !p->can_resident())
    return fail(FLS_ESTATE, "fls_plan_set_resident: needs a bound plan whose G * ceil(tiles / T) CTAs fit the device at once, K in {1, 2, 4, 8} "
                            "in a flat or 1/2/4-wide two-level order, G*K <= 64, fp32 partial sums in ascending order, one state copy per "
                            "group, clipping on and no speculation");
  p->resident_mode = mode < 0 ? -1 : (mode > 0 ? 1 : 0);
  if (wait_limit) p->res_wait_limit = wait_limit;
  return FLS_OK;
}

int fls_plan_get_resident(const fls_plan* p, int* active) {
  if (!p || !active) return fail(FLS_EINVAL, "fls_plan_get_resident: null argument");
  *active = p->resident() ? 1 : 0;
  return FLS_OK;
}

int fls_debug_expire_next_wait(fls_plan* p) {
  if (!p) return fail(FLS_EINVAL, "fls_debug_expire_next_wait: null plan");
  p->res_hold_back = true;
  return FLS_OK;
}

int fls_plan_set_l2_keep(fls_plan* p, uint64_t bytes) {
  if (!p) return fail(FLS_EINVAL, "fls_plan_set_l2_keep: null plan");
  p->l2_keep_bytes = bytes;
  return FLS_OK;
}

int fls_plan_set_overlap(fls_plan* p, int enabled) {
  if (!p) return fail(FLS_EINVAL, "fls_plan_set_overlap: null plan");
  p->overlap = enabled != 0;
  return FLS_OK;
}

int fls_set_profiling(fls_plan* p, int enabled) {
  if (!p) return fail(FLS_EINVAL, "fls_set_profiling: null plan");
  p->profiling = enabled != 0;
  return FLS_OK;
}

int fls_get_kernel_ms(fls_plan* p, double* ms, uint64_t* launches) {
  if (!p || !ms || !launches) return fail(FLS_EINVAL, "fls_get_kernel_ms: null argument");
  for (int k = 0; k < FLS_KERNEL_COUNT; ++k) {
    ms[k] = 0.0;
    launches[k] = 0;
  }
  int rc = FLS_OK;
  for (const TimedLaunch& t : p->timed) {
    cudaError_t e = cudaEventSynchronize(t.end);
    float f = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&f, t.begin, t.end);
    if (e != cudaSuccess) {
      rc = cuda_fail(e, "cudaEventElapsedTime");
    } else {
      ms[t.kernel] += double(f);
      launches[t.kernel] += 1;
    }
    p->event_pool.push_back(t.begin);
    p->event_pool.push_back(t.end);
  }
  p->timed.clear();
  return rc;
}

int fls_get_launch_count(const fls_plan* p, uint64_t* launches) {
  if (!p || !launches) return fail(FLS_EINVAL, "fls_get_launch_count: null argument");
  *launches = p->launches;
  return FLS_OK;
}

int fls_plan_destroy(fls_plan* p) {
  if (!p) return FLS_OK;
  for (const TimedLaunch& t : p->timed) {
    cudaEventDestroy(t.begin);
    cudaEventDestroy(t.end);
  }
  for (cudaEvent_t e : p->event_pool) cudaEventDestroy(e);
  for (cudaEvent_t e : p->ev_copied)
    if (e) cudaEventDestroy(e);
  if (p->ev_begin) cudaEventDestroy(p->ev_begin);
  if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
  delete p;
  return FLS_OK;
}

}  // extern "C"
