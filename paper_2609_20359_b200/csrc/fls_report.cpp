// Communication-cost reporter: the paper's Table of symbols (cost of all-gather, reduce-scatter,
// all-reduce, broadcast) and Eq. 1-5, evaluated for a plan.  Host only.
//
//   C_AG(D, n) = C_RS(D, n) = D (n-1)/(n B_n),   C_AR(D, n) = 2 D (n-1)/(n B_n),   C_BC(D, n) = D / B_n
//   Eq. 1  C_FSDP    = 2 C_AG(M,S) L + C_RS(M,S) L
//   Eq. 2  C_HSDP    = C_FSDP + C_AR(M,R) L
//   Eq. 3  C_FL      = (1/A) C_AR(M,F) L
//   Eq. 4  C_FL+FSDP = C_FSDP + (1/A) C_AR(M,F) L
//   Eq. 5  C_FL+HSDP = C_HSDP + (1/A) C_AR(M,F) L + (1/A) C_BC(M,R) L,  and the FL+FSDP cost when R = 1
// The paper's uniform M*L becomes a sum over the plan's units of their shard size in bytes.
#include <cmath>
#include <limits>

#include "fls_internal.h"

namespace fls {
namespace {

double c_ag(double D, double n, double B) { return D * (n - 1.0) / (n * B); }
double c_rs(double D, double n, double B) { return D * (n - 1.0) / (n * B); }
double c_ar(double D, double n, double B) { return 2.0 * D * (n - 1.0) / (n * B); }
double c_bc(double D, double /*n*/, double B) { return D / B; }

// whole_unit: take D of all-gather / reduce-scatter as the whole unit (S*M), so that the result with
// B = 1 is the byte count one rank puts on the wire.
fls_cost5 eval(const Layout& lay, double elem_bytes, double S, double R, double F, double A, double BS, double BR,
               double BF, bool whole_unit) {
  double fsdp = 0, ar_r = 0, ar_f = 0, bc = 0;
  for (uint64_t m : lay.unit_shard_numel) {
    const double M = double(m) * elem_bytes;
    const double D = whole_unit ? M * S : M;
    fsdp += 2.0 * c_ag(D, S, BS) + c_rs(D, S, BS);
    ar_r += c_ar(M, R, BR);
    ar_f += c_ar(M, F, BF) / A;
    bc += c_bc(M, R, BR) / A;
  }
  fls_cost5 c;
  c.fsdp = fsdp;
  c.hsdp = fsdp + ar_r;
  c.fl = ar_f;
  c.fl_fsdp = fsdp + ar_f;
  c.fl_hsdp = (R > 1.0) ? fsdp + ar_r + ar_f + bc : c.fl_fsdp;
  return c;
}

}  // namespace

void comm_report(const Layout& lay, const fls_plan_desc& d, int route, const double* bw, fls_comm_costs* out) {
  const double e = d.grad_dtype == FLS_GRAD_F32 ? 4.0 : 2.0;
  const double S = d.shard_dim, R = d.replicate_dim, F = d.groups, A = d.sync_period;
  out->paper_bytes = eval(lay, e, S, R, F, A, 1, 1, 1, false);
  out->wire_bytes = eval(lay, e, S, R, F, A, 1, 1, 1, true);
  if (bw) {
    out->seconds = eval(lay, e, S, R, F, A, bw[0], bw[1], bw[2], false);
  } else {
    const double nan = std::numeric_limits<double>::quiet_NaN();
    out->seconds = fls_cost5{nan, nan, nan, nan, nan};
  }
  const double K = S * R;
  // HBM bytes per element of one group's step.  Store and reread: K*e_g read + 4 written by the reduction, then per
  // state copy 16 read (mean gradient, theta, m, v) + 14 written (theta, m, v, bf16).  Recompute: the gradients are
  // read twice and nothing is stored.  Single pass: one kernel, the gradients read once.
  const double copies = d.state_copies == FLS_STATE_PER_REPLICA ? R : 1.0;
  const double per_elem = route == 2 ? K * e + 26.0 : route == 1 ? 2.0 * K * e + 26.0 : K * e + 4.0 + 30.0 * copies;
  out->hbm_bytes_sync_step = F * double(lay.n_padded) * per_elem;
  // FedAvg reads one copy per group and writes every copy (4 + 2 bytes for the parameters and their bf16 copy,
  // 4 + 4 for m and v when they are averaged too)
  const bool opt = (d.fedavg_what & FLS_AVG_OPT_STATE) != 0;
  out->hbm_bytes_fedavg = F * double(lay.n_padded) * ((opt ? 12.0 : 4.0) + (opt ? 14.0 : 6.0) * copies);
}

}  // namespace fls
