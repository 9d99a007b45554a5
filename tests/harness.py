"""Shared test helper: runs the same seeded inputs through the CPU oracle and the CUDA library and
compares them buffer by buffer.  The oracle's planner places the logical vectors in the physical
buffers, so the library's own planner and kernels are checked against it."""
from __future__ import annotations

import numpy as np
import torch

import synthetic as sy
from oracle import fls_oracle as orc

TOL_STATE = 1e-6          # |d| <= 1e-6 * max(1, |x|) on fp32 master / m / v
# m and v are small (1e-4, 1e-8), so the official absolute gate says little about them.  Extra gate:
# |d| <= 1e-5 |x| + 1e-6 max(rms(x), 0.1 * largest |x| any element has had so far).  The second term covers elements that
# cancelled towards zero, whose fp32 store error scales with the magnitude they had before, not with what is left; the
# history term matters only for plans of a handful of parameters, where the rms of the one array says nothing (a
# one-parameter plan whose m went from -1.7e-5 to -2.0e-7 in one step was 1.2e-12 off: 6e-6 of what was left).
REL_M = REL_V = 1e-5
ABS_M = ABS_V = "rms"


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bf16_ordinal(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns on a monotone integer line (+0 and -0 coincide)."""
    b = bits.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b)


def assert_state_close(got: np.ndarray, want: np.ndarray, what: str, rel=None, abs_=None, seen_max=0.0):
    got = got.astype(np.float64); want = want.astype(np.float64)
    d = np.abs(got - want)
    lim = TOL_STATE * np.maximum(1.0, np.abs(want))
    bad = ~(d <= lim)
    assert not bad.any(), f"{what}: {bad.sum()} elements beyond 1e-6*max(1,|x|); worst {d[bad].max() if bad.any() else 0}"
    if rel is not None:
        if abs_ == "rms":
            abs_ = 1e-6 * max(float(np.sqrt(np.mean(want * want))), 0.1 * seen_max) + 1e-30
        bad = ~(d <= rel * np.abs(want) + abs_)
        assert not bad.any(), f"{what}: {bad.sum()} elements beyond rel {rel}; worst idx {np.argmax(d - rel * np.abs(want))}"


def bf16_value(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def assert_bf16_close(got_bits: np.ndarray, want_bits: np.ndarray, what: str):
    """Within 1 bf16 ulp.  The bf16 copy is the rounding of an fp32 value that may itself differ from
    the oracle's by the state tolerance, so for values near zero (where a bf16 ulp is smaller than that
    tolerance) the allowance is one ulp plus the fp32 tolerance: |d| <= ulp_bf16(x) + 1e-6*max(1,|x|)."""
    got, want = bf16_value(got_bits), bf16_value(want_bits)
    fin = np.isfinite(want)
    assert np.array_equal(np.isfinite(got), fin), f"{what}: finiteness differs"
    mag = np.maximum(np.abs(want[fin]), 2.0 ** -126)
    ulp = 2.0 ** (np.floor(np.log2(mag)) - 7)
    d = np.abs(got[fin] - want[fin])
    bad = ~(d <= ulp + TOL_STATE * np.maximum(1.0, mag))
    assert not bad.any(), f"{what}: {bad.sum()} bf16 elements beyond 1 ulp; worst {d[bad].max() if bad.any() else 0}"
    ordinal = np.abs(bf16_ordinal(got_bits) - bf16_ordinal(want_bits))
    assert np.mean(ordinal <= 1) > 0.999, f"{what}: only {np.mean(ordinal <= 1):.5f} of the bf16 copies are within one code"


class Case:
    """One problem instance held twice: logical oracle state and a bound GPU Session."""

    def __init__(self, units, G, S, R_rep=1, H=1, Q=8, grad_dtype="bf16", opt_state=False, seed=1234,
                 grad_sigma=1e-3, master_sigma=0.02, per_buffer_scale=False, hp: orc.Hyper = None, guard=4096,
                 same_grads_all_groups=False, fused=False, state_per_replica=False, speculative=False, resident=-1):
        from paper_2609_20359_b200.session import Session
        self.units, self.G, self.S, self.R_rep, self.H, self.Q = list(units), G, S, R_rep, H, Q
        self.K = S * R_rep
        self.P = int(sum(units))
        self.grad_dtype, self.opt_state, self.seed = grad_dtype, opt_state, seed
        self.grad_sigma, self.per_buffer_scale = grad_sigma, per_buffer_scale
        self.same_grads = same_grads_all_groups
        self.hp = hp or orc.Hyper()
        self.L = orc.plan(units, S, Q)
        th0 = sy.normal_fill_(torch.empty(self.P), sy.stream_key(seed, sy.KIND_MASTER), master_sigma).numpy()
        z = np.zeros(self.P, np.float32)
        # state copies per group: one, or one per replica (FL+HSDP as it runs); states[g] is the first copy of group g
        self.R_state = R_rep if state_per_replica else 1
        self.copies = [[orc.GroupState(th0.copy(), z.copy(), z.copy(), orc.f32_to_bf16_bits(th0)) for _ in range(self.R_state)]
                       for _ in range(G)]
        self.states = [c[0] for c in self.copies]
        self.ring = orc.ring_positions(self.L, R_rep) if self.hp.ring else None
        self.sess = Session(self.P, units, G, S, R_rep, H, grad_dtype, Q, opt_state, self.hp.lr, self.hp.beta1,
                            self.hp.beta2, self.hp.eps, self.hp.weight_decay, self.hp.max_grad_norm, guard_bytes=guard, fused=fused,
                            wire_bf16=self.hp.wire_bf16, ring=self.hp.ring, state_per_replica=state_per_replica, speculative=speculative)
        self.fused = fused
        if resident != -1:            # -1: the library's default (small plans run the step as one resident kernel)
            import paper_2609_20359_b200._binding as _b
            _b.fls_plan_set_resident(self.sess.plan, resident)
        lay = self.sess.layout
        assert lay["n_padded"] == self.L.n_padded and lay["shard_numel"] == self.L.shard_numel
        assert lay["n_state_copies"] == G * self.R_state
        for g in range(G * self.R_state):
            self.sess.master[g].copy_(torch.from_numpy(orc.pack_sharded(self.L, th0)))
            self.sess.param_bf16[g].copy_(torch.from_numpy(orc.pack_unsharded(self.L, th0)).to(torch.bfloat16))
        self.t = 0
        self.norms = []
        self.seen_m = self.seen_v = 0.0          # largest |m|, |v| any element of the oracle state has had

    # gradients of (step, group, buffer) as a logical torch tensor in the gradient dtype
    def grad_logical(self, t, g, k) -> torch.Tensor:
        gg = 0 if self.same_grads else g
        scale = sy.uniform_scale(self.seed, gg, k) if self.per_buffer_scale else 1.0
        dt = torch.float32 if self.grad_dtype == "f32" else torch.bfloat16
        return sy.normal_fill_(torch.empty(self.P, dtype=dt), sy.stream_key(self.seed, sy.KIND_GRAD, t, gg, k), self.grad_sigma, scale)

    def _as_f64(self, x: torch.Tensor) -> np.ndarray:
        if x.dtype == torch.bfloat16:
            return orc.bf16_bits_to_f64(bf16_bits(x))
        return x.numpy().astype(np.float64)

    def load_grads(self, t, override=None):
        """Writes step t's gradients into the GPU buffers and returns the oracle's float64 copies."""
        out = []
        for g in range(self.G):
            row = []
            for k in range(self.K):
                x = override(t, g, k) if override else self.grad_logical(t, g, k)
                row.append(self._as_f64(x))
                if x.dtype == torch.bfloat16:
                    packed = torch.from_numpy(orc.pack_unsharded(self.L, bf16_bits(x).view(np.int16))).view(torch.bfloat16)
                else:
                    packed = torch.from_numpy(orc.pack_unsharded(self.L, x.numpy()))
                self.sess.grads[g][k].copy_(packed)
            out.append(row)
        return out

    def step(self, counts=None, override=None, lr=None, fedavg=True):
        self.t += 1
        grads = self.load_grads(self.t, override)
        row = []
        for g in range(self.G):
            if self.R_state > 1:
                nrm, c, _ = orc.sync_step_replicated(self.copies[g], grads[g], self.S, self.R_rep, self.t, self.hp, lr, self.ring)
            else:
                nrm, c, _ = orc.sync_step_group(self.states[g], grads[g], self.S, self.R_rep, self.t, self.hp, lr, self.ring)
            row.append((nrm, c))
        for st in (c for grp in self.copies for c in grp):
            self.seen_m = max(self.seen_m, float(np.abs(st.m).max()))
            self.seen_v = max(self.seen_v, float(np.abs(st.v).max()))
        self.norms.append(row)
        due = self.t % self.H == 0
        if due and fedavg and self.fused:
            # the single call that does the step and the aggregation
            self.oracle_fedavg(counts)
            self.sess.step_fedavg(counts, float("nan") if lr is None else lr)
        else:
            assert self.sess.step(float("nan") if lr is None else lr) == due
            if due and fedavg:
                self.oracle_fedavg(counts)
                self.sess.fedavg(counts)
        torch.cuda.synchronize()
        return row

    def oracle_fedavg(self, counts):
        if self.R_state > 1:
            orc.fedavg_replicated(self.copies, counts, self.opt_state)
        else:
            orc.fedavg(self.states, counts, self.opt_state)

    def compare(self, check_norms=True):
        torch.cuda.synchronize()
        assert self.sess.guards_intact(), "a kernel wrote outside its buffers"
        if check_norms and self.norms:
            got_n = self.sess.norms().cpu().numpy().astype(np.float64)
            got_c = self.sess.coefs().cpu().numpy().astype(np.float64)
            for g, (nrm, c) in enumerate(self.norms[-1]):
                assert abs(got_n[g] - nrm) <= 1e-6 * max(nrm, 1e-30), (g, got_n[g], nrm)
                assert abs(got_c[g] - c) <= 1e-6 * c, (g, got_c[g], c)
        master, m, v = self.sess.master, self.sess.m, self.sess.v
        for g, st in enumerate(c for grp in self.copies for c in grp):       # copy index g*R_state + rho
            assert_state_close(master[g].cpu().numpy(), orc.pack_sharded(self.L, st.theta), f"master[{g}]")
            assert_state_close(m[g].cpu().numpy(), orc.pack_sharded(self.L, st.m), f"m[{g}]", REL_M, ABS_M, self.seen_m)
            assert_state_close(v[g].cpu().numpy(), orc.pack_sharded(self.L, st.v), f"v[{g}]", REL_V, ABS_V, self.seen_v)
            assert_bf16_close(bf16_bits(self.sess.param_bf16[g]), orc.pack_unsharded(self.L, st.param_bf16), f"param_bf16[{g}]")
            # and the copy is exactly the nearest-even rounding of the GPU's own fp32 master
            own = orc.unpack_sharded(self.L, bf16_bits(master[g].to(torch.bfloat16)))
            assert np.array_equal(orc.unpack_unsharded(self.L, bf16_bits(self.sess.param_bf16[g])), own), f"bf16 copy {g} is not RNE(master)"

    def close(self):
        self.sess.close()
