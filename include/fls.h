/*
 * fls.h -- C ABI of libfls: the data-parallel arithmetic of FL+FSDP / FL+HSDP on one B200.
 *
 * What the library computes (paper: "Accelerating Sharded Data Parallelism at Scale with
 * Federated Learning"):
 *   - F federation groups apply the same sharding policy and train independently
 *     (Section "Augmenting Sharded DP Through FL").  Here: G groups, one layout for all.
 *   - Inside a group, FSDP reduce-scatters the gradients of every layer over the S ranks
 *     (Background, FSDP); HSDP does so inside each of R sharding groups and then
 *     all-reduces corresponding gradient shards across the R replicas (Background, HSDP;
 *     Section "HSDP", Eq. 2).  Here: K = S*R gradient buffers per group are read from
 *     HBM and reduced in that order; the result feeds a global-norm clip and AdamW on the
 *     group's fp32 master/m/v shards, and a bf16 parameter copy is written.
 *   - Every A steps the corresponding shards of all groups are replaced by their weighted
 *     average (FedAvg; Background "Federated Learning", Sections FL+FSDP and FL+HSDP).
 *   - Eq. 1-5 and the table of collective costs give the communication cost of each
 *     scheme; fls_comm_report evaluates them for a plan.
 * Symbols: G = paper F (groups), H = paper A (aggregation period), S = shards,
 * R_rep = paper R (replicas; 1 for FSDP), L units = the paper's L sharded layers.
 *
 * Conventions
 *   - Every function returns 0 (FLS_OK) or an error code > 0 and never throws, aborts or
 *     prints.  fls_last_error() gives the calling thread's last message.
 *   - "host" / "device" beside a pointer says where the memory it points to lives.
 *   - The caller owns every device buffer and the stream.  The library owns the plan, its
 *     host tables, a few CUDA events and one internal copy stream; on the device it uses
 *     only the caller's workspace.  It allocates no bulk device memory.
 *   - Nothing synchronises the device except where stated (fls_plan_bind,
 *     fls_sync_step_host, fls_get_kernel_ms).
 *   - A plan is not thread-safe; use one plan per host thread or lock around it.
 */
#ifndef FLS_H_
#define FLS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fls_plan fls_plan; /* opaque, created by fls_plan_create, freed by fls_plan_destroy */

enum { FLS_OK = 0, FLS_EINVAL = 1, FLS_EALIGN = 2, FLS_EPTR = 3, FLS_ESIZE = 4, FLS_ECUDA = 5, FLS_ESTATE = 6 };
enum { FLS_GRAD_BF16 = 0, FLS_GRAD_F32 = 1 };
enum { FLS_WIRE_F32 = 0, FLS_WIRE_BF16 = 1 };          /* reduce_wire */
enum { FLS_ORDER_ASCENDING = 0, FLS_ORDER_RING = 1 };  /* reduce_order */
enum { FLS_STATE_PER_GROUP = 0, FLS_STATE_PER_REPLICA = 1 }; /* state_copies */
enum { FLS_AVG_PARAMS = 1, FLS_AVG_OPT_STATE = 2, FLS_AVG_FUSED = 4 }; /* fedavg_what bit mask */
enum { FLS_KERNEL_REDUCE = 0, FLS_KERNEL_ADAMW = 1, FLS_KERNEL_FEDAVG = 2, FLS_KERNEL_ADAMW_FEDAVG = 3, FLS_KERNEL_COUNT = 4 };
enum { FLS_STATUS_NONFINITE_NORM = 1,   /* sticky bits of the device status word */
       FLS_STATUS_WAIT_EXPIRED = 2 };   /* a CTA of the resident step gave up waiting for its group's norm; the step is incomplete */

#define FLS_MAX_GROUPS 64        /* G <= 64 */
#define FLS_MAX_GRAD_BUFFERS 64  /* K = shard_dim * replicate_dim <= 64 */
#define FLS_MAX_FUSED_GROUPS 16  /* fls_sync_step_fedavg fuses the aggregation for G up to this */
#define FLS_MAX_STATE_COPIES 64  /* G * R_rep <= 64 with FLS_STATE_PER_REPLICA */
#define FLS_BUFFER_ALIGN 32      /* every device buffer must start on a 32-byte boundary */
#define FLS_NOALLOC_MAX_ELEMS 536870912ull /* 2^29: largest n_elems fls_reduce_norm_noalloc accepts */

/* Problem statement.  One layout is shared by all groups (the paper's alignment constraint:
 * shards of different federation groups must correspond one to one). */
typedef struct {
  uint64_t n_params;          /* logical parameter count P = sum of unit_numel                          */
  uint32_t n_units;           /* L; 0 with unit_numel == NULL means one unit of n_params                */
  const uint64_t* unit_numel; /* host, L entries, copied: the bucket / FSDP-unit ("layer") table        */
  uint32_t groups;            /* G >= 1                                                                 */
  uint32_t shard_dim;         /* S >= 1                                                                 */
  uint32_t replicate_dim;     /* R_rep >= 1; 1 = FL+FSDP, > 1 = FL+HSDP (shard level reduced first)     */
  uint32_t sync_period;       /* H >= 1: FedAvg is due after every H-th step                            */
  uint32_t grad_dtype;        /* FLS_GRAD_BF16 or FLS_GRAD_F32                                          */
  uint32_t align_elems;       /* Q >= 1: every unit's shard length is rounded up to a multiple of Q.
                                 Q = 1 pads a unit to a multiple of S exactly; multiples of 8 keep every
                                 shard on the vector path (otherwise element-wise loads are used)      */
  uint32_t fedavg_what;       /* FLS_AVG_PARAMS, optionally | FLS_AVG_OPT_STATE (m and v averaged too),
                                 optionally | FLS_AVG_FUSED (workspace holds one reduced gradient per group
                                 so that fls_sync_step_fedavg can fuse the aggregation into the step)      */
  uint32_t reduce_wire;       /* FLS_WIRE_F32 (default): partial sums of bf16 gradients in fp32 (exact unless the
                                 addends span more than 16 binades), of fp32 gradients in double with one rounding
                                 to fp32 after the scaling by 1/K.  FLS_WIRE_BF16 (bf16 gradients only):
                                 every partial sum of both reduction levels and the final mean are rounded
                                 to bf16, emulating collectives that run in bf16 -- the setting in which the
                                 paper observes that the FSDP and HSDP orders give different numbers.  Slower
                                 (generic kernel); meant for numerical experiments                         */
  uint32_t reduce_order;      /* FLS_ORDER_ASCENDING (default): buffers are added in ascending index at both levels.
                                 FLS_ORDER_RING: in the order ring collectives produce.  The elements rank s owns
                                 after the reduce-scatter are summed sigma = s+1, s+2, ..., s (mod S): the chunk
                                 starts on the next rank and its owner adds last.  The all-reduce across replicas
                                 is a ring reduce-scatter + all-gather over R_rep equal sub-chunks of every
                                 rank's slice of a unit (ceil(M_u/R_rep) elements each): sub-chunk c is summed
                                 rho = c+1, ..., c (mod R_rep).  Same sums, other rounding order: visible with
                                 FLS_WIRE_BF16, within rounding otherwise.  Generic kernel (slower)           */
  uint32_t state_copies;      /* FLS_STATE_PER_GROUP (default): one master/m/v/bf16 copy per group.
                                 FLS_STATE_PER_REPLICA: one per replica, G*R_rep in all (FL+HSDP as it runs: every
                                 replica of a group applies the same mean gradient to its own copy; only one replica
                                 per group takes part in FedAvg and then broadcasts the result inside its group, the
                                 C_BC term of Eq. 5).  Needs G*R_rep <= FLS_MAX_STATE_COPIES                       */
  double lr, beta1, beta2, eps, weight_decay;
  double max_grad_norm;       /* <= 0 disables clipping (the norm is still computed)                    */
} fls_plan_desc;

/* Layout computed by the planner.  Arrays are owned by the plan and live as long as it does.
 *   unit u is zero-padded to S*M_u elements, M_u = roundup(ceil(n_u/S), Q);
 *   UNSHARDED order (gradient buffers, bf16 parameter copy): element i of unit u at unit_offset[u] + i;
 *   SHARD order (master, m, v): rank s = i / M_u holds it at s*shard_numel + unit_shard_offset[u] + i % M_u.
 * Padding elements must be zero in every buffer the caller fills; the library keeps them zero. */
typedef struct {
  uint64_t n_padded;                 /* N_pad = sum S*M_u: element count of EVERY buffer below          */
  uint64_t shard_numel;              /* N_pad / S                                                       */
  uint32_t n_units;
  uint32_t grad_buffers;             /* K = S*R_rep per group                                           */
  const uint64_t* unit_offset;       /* host, L entries                                                 */
  const uint64_t* unit_shard_numel;  /* host, L entries: M_u                                            */
  const uint64_t* unit_shard_offset; /* host, L entries                                                 */
  uint64_t workspace_bytes;          /* size the caller must provide in fls_buffers.workspace           */
  uint32_t n_segments;               /* contiguous (unit, shard) runs the kernels walk                  */
  uint32_t vector_path;              /* 1 if every segment is 8-element aligned in both orders          */
  uint32_t n_state_copies;           /* entries of fls_buffers.master / m / v / param_bf16: G, or G*R_rep with
                                        FLS_STATE_PER_REPLICA                                            */
  uint32_t reserved;
} fls_layout;

/* Device buffers, all caller-owned, each N_pad elements, FLS_BUFFER_ALIGN-aligned, non-overlapping.
 * The pointer ARRAYS are host memory and are copied by fls_plan_bind. */
typedef struct {
  const void* const* grads; /* host array of G*K device pointers, index g*K + rho*S + sigma; bf16 or fp32;
                               unsharded order; read-only to the library, never cleared by it            */
  float* const* master;     /* host array of n_state_copies device pointers (G; with FLS_STATE_PER_REPLICA G*R_rep,
                               index g*R_rep + rho): fp32 parameters, shard order, in/out                   */
  float* const* m;          /* same: first moment                                                        */
  float* const* v;          /* same: second moment                                                       */
  void* const* param_bf16;  /* host array of n_state_copies device pointers: bf16 copy, unsharded order, output */
  void* workspace;          /* device, >= workspace_bytes; holds the reduced gradient, the norm partials,
                               per-group norm / clip coefficient, the status word and the segment table  */
  uint64_t workspace_bytes;
} fls_buffers;

/* Communication cost of one training step, one value per equation of the paper. */
typedef struct { double fsdp, hsdp, fl, fl_fsdp, fl_hsdp; } fls_cost5; /* Eq. 1, 2, 3, 4, 5 */
typedef struct {
  fls_cost5 paper_bytes; /* Eq. 1-5 as printed with the bandwidths taken out: message size D = M_u, the unit's
                            shard in bytes of the gradient dtype, summed over units instead of M*L            */
  fls_cost5 wire_bytes;  /* bytes one rank sends per step when D of all-gather / reduce-scatter is the whole
                            unit (S*M_u), the convention of the NCCL performance notes the paper cites        */
  fls_cost5 seconds;     /* Eq. 1-5 with B_S, B_R, B_F; NaN when no bandwidths were given                     */
  double hbm_bytes_sync_step; /* bytes one fls_sync_step must move on the route the plan is set to at the time of the
                                 call: G*N_pad*(K*e_g + 34) (store and reread), G*N_pad*(2*K*e_g + 26) (recompute,
                                 the default when K*e_g < 8), G*N_pad*(K*e_g + 26) (single pass: no clipping, a
                                 speculative step that is kept, or the resident step of a small plan).  With FLS_STATE_PER_REPLICA: G*N_pad*(K*e_g + 4 +
                                 30*R_rep)                                                                     */
  double hbm_bytes_fedavg;    /* bytes one fls_fedavg must move: G*N_pad*10, or *26 with optimizer state; with
                                 FLS_STATE_PER_REPLICA the broadcast adds 6 (14) per extra copy: G*N_pad*(4 + 6*R_rep),
                                 or G*N_pad*(12 + 14*R_rep)                                                    */
} fls_comm_costs;

/* Layout planner + validation (flat-buffer layout: padding to the shard multiple, per-unit offsets).
 * Host only: touches no GPU.  Errors: FLS_EINVAL for a null argument, G, S, R_rep, H or Q = 0, G or K
 * above the maxima, sum(unit_numel) != n_params, a zero-length unit, beta outside [0,1), eps <= 0, lr < 0,
 * an unknown dtype, order or state_copies value, FLS_WIRE_BF16 with fp32 gradients, G*R_rep above
 * FLS_MAX_STATE_COPIES with FLS_STATE_PER_REPLICA, or fedavg_what without FLS_AVG_PARAMS.  On error *out is NULL. */
int fls_plan_create(const fls_plan_desc* desc, fls_plan** out);

/* Copies the layout summary into *out (host). */
int fls_plan_query(const fls_plan* plan, fls_layout* out);

/* Validates and records the caller's buffers, uploads the segment table into the workspace and clears
 * the status word.  Uses the current CUDA device; synchronises it.  May be called again to rebind.
 * Errors: FLS_EPTR (null, host or overlapping buffers), FLS_EALIGN, FLS_ESIZE (workspace too small),
 * FLS_ECUDA. */
int fls_plan_bind(fls_plan* plan, const fls_buffers* buffers);

/* One local training step of all G groups (the groups train without waiting for one another), enqueued
 * on `cuda_stream` (a cudaStream_t; NULL = default stream).  Per group: mean of the K gradient buffers,
 * stored as fp32: ascending buffer order inside a sharding group, then ascending replica order (reduce-scatter
 * over S, then all-reduce over R: Background FSDP/HSDP, Eq. 2; reduce_wire and reduce_order change the
 * precision of the partial sums and the order), one scaling by 1/K; L2 norm of the mean
 * gradient over the whole group; c = min(1, max_grad_norm/(norm + 1e-6)); AdamW with decoupled weight
 * decay and bias correction on master/m/v in place (on every state copy of the group; speculative plans
 * write the other buffer set, see fls_plan_set_speculative); bf16 copy of the new parameters (round to
 * nearest even).  `lr` overrides the plan's learning rate for this step; pass NaN to use the plan's.  The step
 * counter t is incremented; *fedavg_due (host, may be NULL) is set to (t % H == 0).
 * Errors: FLS_ESTATE if not bound, FLS_ECUDA on a launch failure (state is then undefined). */
int fls_sync_step(fls_plan* plan, double lr, void* cuda_stream, int* fedavg_due);

/* Same step with the gradients in HOST memory: host_grads is a host array of G*K host pointers (same
 * order and size as fls_buffers.grads; pinned memory for full speed).  Each group's gradients are copied
 * into the bound device gradient buffers on an internal stream while the previous group computes; after
 * the last group the G norms are copied to host_norms (host, G floats, may be NULL) and the call waits
 * for `cuda_stream`.  This is the end-to-end form of fls_sync_step. */
int fls_sync_step_host(fls_plan* plan, const void* const* host_grads, double lr, void* cuda_stream,
                       float* host_norms, int* fedavg_due);

/* FedAvg: every group's parameters become sum_g w_g x_g, w_g = n_g / sum n (the weighted mean of the
 * locally trained models of Background "Federated Learning", taken shard by shard across the federation
 * groups, Section FL+FSDP).  fp32 accumulation in ascending group order; all G master copies and
 * all G bf16 copies are rewritten; m and v too if the plan has FLS_AVG_OPT_STATE.  With
 * FLS_STATE_PER_REPLICA replica 0 of every group is read and all G*R_rep copies are rewritten (the
 * broadcast inside each group, Section FL+HSDP).  sample_counts: host,
 * G entries, NULL = equal weights.  The step counter is unchanged.
 * Errors: FLS_EINVAL if all counts are zero, FLS_ESTATE, FLS_ECUDA. */
int fls_fedavg(fls_plan* plan, const uint64_t* sample_counts, void* cuda_stream);

/* Aggregation with an outer optimizer (the FedOpt family of the paper's related work: AdamW inside the groups,
 * SGD with optional Nesterov momentum across them; the paper presents FedAvg as the base strategy that others
 * can replace).  With xbar = sum_g w_g x_g as in fls_fedavg:
 *   delta = x_global - xbar;  buf = momentum*buf + delta;  d = nesterov ? delta + momentum*buf : buf;
 *   x_global -= outer_lr * d;  every group's master = x_global, every bf16 copy = bf16(x_global).
 * outer_lr = 1, momentum = 0 is plain FedAvg (up to fp32 rounding of x - (x - xbar)).  global_params and
 * outer_momentum: device, N_pad floats each, shard order, FLS_BUFFER_ALIGN-aligned, caller-owned, in/out (start
 * them as a copy of the initial parameters and as zeros).  m and v are averaged as in fls_fedavg when the plan has
 * FLS_AVG_OPT_STATE.  fp32 arithmetic, fma accumulation of xbar in ascending g.
 * Errors: FLS_EPTR / FLS_EALIGN for the two buffers, FLS_EINVAL (non-finite outer_lr or momentum, all counts zero),
 * FLS_ESTATE, FLS_ECUDA. */
int fls_fedavg_outer(fls_plan* plan, const uint64_t* sample_counts, double outer_lr, double momentum, int nesterov,
                     float* global_params, float* outer_momentum, void* cuda_stream);

/* One local step of all groups immediately followed by FedAvg, i.e. exactly fls_sync_step then fls_fedavg
 * (same results bit for bit), for the steps on which aggregation is due (every A-th step, after
 * its optimizer update).  With FLS_AVG_FUSED in the plan and G <= FLS_MAX_FUSED_GROUPS the aggregation is fused
 * into the optimizer kernel: after the G reductions one kernel applies AdamW to every group's element,
 * averages the G results in registers and writes the average to all G copies, which saves FedAvg's own
 * read and write of the parameters (10*G bytes per parameter).  Otherwise (and with more than 32 extra replica
 * copies) it runs the two calls one after the other.  sample_counts: host, G entries, NULL = equal weights.  Errors: as fls_sync_step and fls_fedavg. */
int fls_sync_step_fedavg(fls_plan* plan, double lr, const uint64_t* sample_counts, void* cuda_stream);

/* Device pointers (inside the workspace) to G floats each: the gradient norm and the clip coefficient of
 * the last step, valid once that step has completed on its stream.  Either output may be NULL. */
int fls_get_norms(const fls_plan* plan, const float** dev_norms, const float** dev_coefs);

/* Device pointer to the reduced (mean) gradient of the LAST group processed: N_pad floats, shard order.
 * FLS_ESTATE if the last step stored none (plans with K*e_g < 8 bytes recompute it, see fls_plan_set_recompute;
 * plans without clipping run a single pass, see fls_plan_set_single_pass). */
int fls_get_reduced_grad(const fls_plan* plan, const float** dev_gbar);

/* Device pointer to the sticky status word (FLS_STATUS_* bits).  Non-finite values are not errors:
 * they propagate by IEEE rules and set a bit here. */
int fls_get_status(const fls_plan* plan, const uint32_t** dev_status);

/* Step counter t (starts at 0; the first step uses exponent 1 in the bias corrections).  fls_set_step
 * resumes from a checkpoint: master/m/v are the caller's, t is the only other state. */
int fls_get_step(const fls_plan* plan, uint64_t* t);
int fls_set_step(fls_plan* plan, uint64_t t);

/* Eq. 1-5 for this plan (L units, M_u, S, R = R_rep, F = G, A = H).  bw_bytes_per_s: host, {B_S, B_R, B_F}
 * or NULL.  With R_rep = 1 the FL+HSDP entry equals the FL+FSDP one (the paper's fallback).  Host only. */
int fls_comm_report(const fls_plan* plan, const double* bw_bytes_per_s, fls_comm_costs* out);

/* Launch shape of one kernel (FLS_KERNEL_*).  By default the grid covers every tile once.  For the AdamW and
 * FedAvg kernels ctas_per_sm > 0 switches to a persistent grid of ctas_per_sm * (number of SMs) CTAs that
 * stride over the tiles; -2 restores the default; 0 and -1 keep the current value.  descending: 1 / 0 sets
 * the direction in which those two kernels walk the tiles, negative keeps it.  The reduce kernel has one
 * launch shape and ignores both. */
int fls_plan_tune(fls_plan* plan, uint32_t kernel, int ctas_per_sm, int descending);

/* How fls_sync_step gets the mean gradient into AdamW.  With fewer than 8 gradient bytes per element (bf16 and
 * K <= 3, fp32 and K = 1) reading the gradients twice (a norm pass, then AdamW forming the mean itself: 2*K*e_g +
 * 26 bytes per element) is cheaper than storing the fp32 mean and reading it back (K*e_g + 34); such plans do
 * that by default.  mode 0 forces store-and-reread, 1 forces recomputation (FLS_ESTATE if the plan does not
 * qualify), -1 restores the default.  The results are identical either way. */
int fls_plan_set_recompute(fls_plan* plan, int mode);

/* Plans without clipping (max_grad_norm <= 0) need no second pass: the clip coefficient is 1 before the norm is
 * known, so by default one kernel per group reduces the gradients, applies AdamW and accumulates the norm (which
 * is still reported): K*e_g + 26 bytes per element.  mode 0 forces the two-pass route, 1 forces the single pass
 * (FLS_ESTATE if the plan clips or uses FLS_WIRE_BF16), -1 restores the default.  master, m, v and the bf16 copy
 * are identical either way; after a single-pass step fls_get_reduced_grad has nothing to offer (FLS_ESTATE). */
int fls_plan_set_single_pass(fls_plan* plan, int mode);

/* Speculative single pass for plans that clip.  When the norm usually stays below max_grad_norm, the two passes
 * of a step (norm first, then AdamW) can be replaced by one that guesses "clip coefficient = 1": one kernel per
 * group forms the mean gradient, applies AdamW with coefficient 1 and computes the norm; a second, normally empty
 * kernel looks at the coefficient and, only if it is not 1, redoes the step with it.  K*e_g + 26 bytes per element
 * when the guess holds, twice that when it does not (the default route costs K*e_g + 34 either way), so it pays
 * only on workloads that rarely clip; it is never on by default.  Results are bit-identical to the default route.
 * The first kernel must not overwrite its own input, so the plan needs a second set of state buffers:
 * fls_plan_bind_shadow gives it G device pointers each for master, m and v (host arrays; N_pad floats each,
 * FLS_BUFFER_ALIGN-aligned, caller-owned, overlapping nothing bound).  Every speculative step reads the current set
 * and writes the other one, which then becomes current: after each fls_sync_step ask fls_get_state where group g's
 * state is now.  fls_plan_set_speculative(plan, 1) turns it on: FLS_ESTATE without shadow buffers, for plans that do
 * not clip, for FLS_WIRE_BF16, FLS_ORDER_RING or FLS_STATE_PER_REPLICA plans; 0 turns it off (the state stays where
 * it is).  The fused aggregation of fls_sync_step_fedavg steps in place and does not speculate.
 * fls_get_spec_stats: device pointer to two uint32 counters, [0] group-steps whose guess held, [1] group-steps that
 * were redone; valid once the steps have completed on their stream. */
int fls_plan_bind_shadow(fls_plan* plan, float* const* master, float* const* m, float* const* v);
int fls_plan_set_speculative(fls_plan* plan, int enabled);
int fls_get_spec_stats(const fls_plan* plan, const uint32_t** dev_counts);

/* Current device pointers of state copy `copy` (0 .. n_state_copies-1): what was bound, except on speculative
 * plans, where every step moves the state to the other buffer set.  Any output may be NULL. */
int fls_get_state(const fls_plan* plan, uint32_t copy, float** master, float** m, float** v);

/* Small plans are launch-bound when every group gets its own two kernels.  When the plan allows it (G > 1, G*K <= 64,
 * K = 4 or 8 in a flat or 1/2/4-wide two-level order, the default two-pass route, one state copy per group, and a
 * reduced-gradient slot per group in the workspace: FLS_AVG_FUSED plans and plans whose G reduced gradients need at
 * most 24 MiB) fls_sync_step can run all groups in ONE reduce grid and ONE AdamW grid, with the group in the grid's y
 * dimension; fls_sync_step_fedavg then uses the one reduce grid as well.  mode -1 (default): automatically, only while
 * the G reduced gradients fit in 24 MiB (beyond that the per-group sequence is faster: its reduced gradient is still in
 * L2 when AdamW reads it); 0: never; 1: whenever the plan allows it (FLS_ESTATE otherwise).  Results do not change.
 * Recompute plans (K*e_g < 8, which store no mean gradient) with G > 1 and K = 1 or 2 have their own form of it, at any
 * size unless mode is 0: ONE grid computes the norms of all groups, then one AdamW kernel per group forms the mean
 * gradient again (G + 1 launches instead of 2 G).
 * fls_plan_get_batching: whether the next fls_sync_step would run that way. */
int fls_plan_set_batching(fls_plan* plan, int mode);
int fls_plan_get_batching(const fls_plan* plan, int* active);

/* Resident step.  When all G groups together are small enough for every CTA of one grid to be resident on the device
 * at once (each CTA keeping the mean gradient of up to a few tiles in shared memory: about 8 million elements in all on
 * 148 SMs), fls_sync_step can run as ONE cooperative kernel: reduce, norm, a wait inside the kernel until the group's
 * clip coefficient is known, AdamW.  K*e_g + 26 bytes per element and one launch instead of two or 2*G.  Needs K in
 * {1, 2, 4, 8} in a flat or 1/2/4-wide two-level order, G*K <= 64, fp32 partial sums in ascending order, one state copy
 * per group, clipping on, no speculation.  mode -1 (default): automatically, when the plan fits and the G mean
 * gradients would take at most 16 MiB (about four million elements; measured: a clear gain up to two million, even at four); 0: never; 1: whenever the plan fits (FLS_ESTATE otherwise; the fit depends on
 * the device, so the plan must be bound).  The reduced gradient is not stored (fls_get_reduced_grad: FLS_ESTATE) and
 * fls_sync_step_fedavg runs the resident step followed by fls_fedavg.  Mean gradient and AdamW arithmetic are those of
 * the other routes; the norm is summed over another tree (several tiles per CTA), so it can differ from theirs in the
 * last bits of a double.  The wait is bounded: a CTA that polls `wait_limit` times in vain (0 keeps the default,
 * about a second) sets FLS_STATUS_WAIT_EXPIRED in the status word and leaves its part of the state untouched.
 * fls_plan_get_resident: whether the next fls_sync_step would run that way. */
int fls_plan_set_resident(fls_plan* plan, int mode, uint32_t wait_limit);
int fls_plan_get_resident(const fls_plan* plan, int* active);

/* For tests of the bounded wait: the next resident step (one launch) is started so that its CTAs wait for a value
 * that nobody publishes.  Every CTA gives up after `wait_limit` polls, FLS_STATUS_WAIT_EXPIRED appears in the status
 * word, master/m/v/bf16 stay as they were, and the device stays usable.  Set a small wait_limit first. */
int fls_debug_expire_next_wait(fls_plan* plan);

/* How many bytes at the end of the reduced gradient the reduce kernel stores with the "evict last" L2 policy (the
 * AdamW kernel walks the reduced gradient backwards, so it reads that part first and finds it in L2); the rest is
 * stored "evict first" like every other stream.  Default 64 MiB.  Scheduling only: results do not change. */
int fls_plan_set_l2_keep(fls_plan* plan, uint64_t bytes);

/* enabled != 0 (the default): inside one call every kernel but the first is launched so that its first CTAs may
 * start during the tail of the kernel before it (programmatic dependent launch); they fetch what that kernel does
 * not write and wait for its completion before touching anything else, so the results are identical.  0: plain
 * launches, each kernel starts when the previous one has finished. */
int fls_plan_set_overlap(fls_plan* plan, int enabled);

/* Per-kernel timing with CUDA events recorded on the caller's stream around every launch.
 * fls_set_profiling(plan, 1) turns it on; fls_get_kernel_ms waits for the recorded events, adds their
 * durations into ms[FLS_KERNEL_COUNT] / launches[FLS_KERNEL_COUNT] (host, indexed by FLS_KERNEL_*) and clears
 * the record. */
int fls_set_profiling(fls_plan* plan, int enabled);
int fls_get_kernel_ms(fls_plan* plan, double* ms, uint64_t* launches);

/* Number of kernels this plan has launched so far. */
int fls_get_launch_count(const fls_plan* plan, uint64_t* launches);

/* (No counterpart in the paper: this call exists for users of the library who are not allowed to allocate.)
 * Gradient reduction + global norm of ONE group without a plan, a workspace or any allocation, for callers
 * that must not call cudaMalloc: a plug-in inside an application whose pool already owns the device, a
 * service that forbids allocation after start-up, a loop that cannot afford the device-wide stall an
 * allocation can cause.  It computes what the first kernel of fls_sync_step computes for one group:
 *   gbar_out[j] = mean over the K = shard_dim*replicate_dim buffers (same order: ascending inside a
 *   sharding group, then ascending replicas; fp32), norm_coef_out[0] = L2 norm of gbar,
 *   norm_coef_out[1] = min(1, max_grad_norm/(norm + 1e-6)) (1 if max_grad_norm <= 0).
 * grads: host array of K device pointers (bf16 or fp32 per grad_dtype, n_elems each, 32-byte aligned);
 * gbar_out: device, n_elems floats, 32-byte aligned; norm_coef_out: device, 2 floats, 8-byte aligned;
 * all caller-owned.  The work is enqueued on cuda_stream; nothing is synchronised.
 * Scratch (one double per 16384 elements and a counter) lives in a static device array of about 256 KiB
 * that every GPU using the library holds until the process exits; hence n_elems <= FLS_NOALLOC_MAX_ELEMS,
 * larger sizes are rejected with FLS_ESIZE and a message.  The first call on each device looks up the
 * array's device address; make that first call outside any stream capture.  All calls share the array:
 * calls that overlap on the same GPU (other streams or threads) race and must be serialised by the caller.
 * No cudaMalloc/cudaFree or other allocating routine is called.
 * Errors: FLS_EPTR, FLS_EALIGN, FLS_EINVAL (K > 64, n_elems = 0, bad dtype), FLS_ESIZE, FLS_ECUDA. */
int fls_reduce_norm_noalloc(const void* const* grads, uint32_t shard_dim, uint32_t replicate_dim, uint32_t grad_dtype,
                            uint64_t n_elems, double max_grad_norm, float* gbar_out, float* norm_coef_out,
                            void* cuda_stream);

/* Frees the plan and its events/stream.  Device buffers are the caller's and are not touched. */
int fls_plan_destroy(fls_plan* plan);

/* Message of the last error on the calling thread ("" if none).  Host string owned by the library. */
const char* fls_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FLS_H_ */
