"""CPU oracle for the FL+FSDP / FL+HSDP sync step and FedAvg.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain definition that the CUDA library is checked against.
It is numpy in float64, shares no code with the CUDA path and must never be
imported by it: only the tests, the smoke check and the benchmark's CPU-baseline
leg may call it.

What the paper fixes and what it leaves open
--------------------------------------------
The paper defines the communication pattern, not the arithmetic:
  * FSDP: every layer is split equally in S shards; the backward pass
    reduce-scatters the gradients over the S ranks (Background, "Fully Sharded
    Data Parallelism").
  * HSDP: R x S mesh; reduce-scatter inside each sharding group, then an
    all-reduce of corresponding gradient shards across the R replicas
    (Background, "Hybrid Sharded Data Parallelism"; Section "HSDP" before Eq. 2).
  * FL+FSDP / FL+HSDP: F federation groups with the same sharding policy train
    independently and every A steps each shard is replaced by the (weighted)
    average of the corresponding shards of all groups (Section "Augmenting
    Sharded DP Through FL"; FedAvg as described in Background, "Federated
    Learning").
  * Optimiser: AdamW with learning rate 3e-4, training in bf16 (Experimental Setup).
  * Cost model: Table of symbols and Eq. 1-5.
Everything numeric that the paper does not state (mean vs sum, order, clipping
rule, AdamW variant, rounding) follows the readings listed beside each function.

Coordinates.  The oracle works on LOGICAL vectors: the P parameters of all units
concatenated, unit after unit.  `plan()` and `pack_*`/`unpack_*` translate
between logical vectors and the two physical orders of the flat buffers.
Symbols: G groups (paper F), S shards, R_rep replicas (paper R), K = S*R_rep
gradient buffers per group, H sync period (paper A).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

CLIP_EPS = 1e-6  # added to the norm in the clip coefficient (reading: the common global-norm convention)


# --------------------------------------------------------------------------- bf16 <-> values
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of bf16 bit patterns (uint16): a bf16 is the top half of an fp32."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round stored fp32 values to bf16, nearest-even on the 16 dropped bits; NaN stays NaN."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    keep_lsb = (u >> np.uint64(16)) & np.uint64(1)
    rounded = (u + np.uint64(0x7FFF) + keep_lsb) >> np.uint64(16)
    out = rounded.astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out = np.where(nan, ((u >> np.uint64(16)) | np.uint64(0x0040)).astype(np.uint16), out)
    return out


# --------------------------------------------------------------------------- layout planner
@dataclass
class Layout:
    """Flat-buffer layout of one group (identical for every group: the paper's
    alignment constraint, Section "Augmenting Sharded DP Through FL")."""
    unit_numel: List[int]          # n_u
    S: int
    Q: int
    unit_shard_numel: List[int]    # M_u
    unit_padded: List[int]         # n'_u = S*M_u
    unit_offset: List[int]         # off_u  in the unsharded order (gradients, bf16 copy)
    unit_shard_offset: List[int]   # soff_u inside one rank's shard buffer
    n_params: int
    n_padded: int
    shard_numel: int
    _addr_unsharded: Optional[np.ndarray] = field(default=None, repr=False)
    _addr_sharded: Optional[np.ndarray] = field(default=None, repr=False)


def plan(unit_numel: Sequence[int], S: int, Q: int = 1) -> Layout:
    """Each unit ("layer") is split equally over S ranks in shards of size M_u
    (Background, FSDP).  Reading for indivisible sizes: zero-pad the unit to
    S*M_u with M_u = roundup(ceil(n_u/S), Q)."""
    assert S >= 1 and Q >= 1 and len(unit_numel) >= 1
    M, padded, off, soff = [], [], [], []
    o = so = 0
    for n in unit_numel:
        assert n >= 1
        per = -(-n // S)
        m = -(-per // Q) * Q
        M.append(m); padded.append(S * m); off.append(o); soff.append(so)
        o += S * m; so += m
    return Layout(list(unit_numel), S, Q, M, padded, off, soff, int(sum(unit_numel)), o, so)


def addresses_of(L: Layout, logical_index) -> tuple:
    """For logical elements (index into the concatenation of all units): their index in the unsharded
    order and their address in the rank-major shard order [S][shard_numel]."""
    p = np.asarray(logical_index, dtype=np.int64)
    starts = np.concatenate([[0], np.cumsum(L.unit_numel)]).astype(np.int64)
    u = np.searchsorted(starts, p, side="right") - 1                 # unit of each element
    i = p - starts[u]                                                # index inside the unit
    M = np.asarray(L.unit_shard_numel, dtype=np.int64)[u]
    j = np.asarray(L.unit_offset, dtype=np.int64)[u] + i
    a = (i // M) * L.shard_numel + np.asarray(L.unit_shard_offset, dtype=np.int64)[u] + i % M
    return j, a


def _addresses(L: Layout):
    """addresses_of every logical element, cached."""
    if L._addr_unsharded is None:
        L._addr_unsharded, L._addr_sharded = addresses_of(L, np.arange(L.n_params, dtype=np.int64))
    return L._addr_unsharded, L._addr_sharded


def pack_unsharded(L: Layout, logical: np.ndarray) -> np.ndarray:
    """Logical vector -> padded buffer in unsharded order (what backward produces /
    the all-gather result).  Padding is zero."""
    out = np.zeros(L.n_padded, dtype=logical.dtype)
    out[_addresses(L)[0]] = logical
    return out


def pack_sharded(L: Layout, logical: np.ndarray) -> np.ndarray:
    """Logical vector -> padded buffer in shard order: rank s holds, for every unit
    in turn, elements [s*M_u, (s+1)*M_u) of that unit."""
    out = np.zeros(L.n_padded, dtype=logical.dtype)
    out[_addresses(L)[1]] = logical
    return out


def unpack_unsharded(L: Layout, buf: np.ndarray) -> np.ndarray:
    return np.asarray(buf)[_addresses(L)[0]]


def unpack_sharded(L: Layout, buf: np.ndarray) -> np.ndarray:
    return np.asarray(buf)[_addresses(L)[1]]


# --------------------------------------------------------------------------- one local step
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Values rounded to bf16 (via the stored-fp32 rounding above), returned as float64."""
    return bf16_bits_to_f64(f32_to_bf16_bits(np.asarray(x, dtype=np.float64).astype(np.float32)))


def ring_positions(L: Layout, R_rep: int):
    """For every logical element: (s, c) = the rank that ends up owning it after the reduce-scatter over the S
    ranks of a sharding group, and the sub-chunk of that rank's slice it falls in when the slice is cut into
    R_rep equal parts for the ring all-reduce across the replicas.  Element i of unit u: s = i div M_u; its
    position inside the slice is p = i mod M_u and c = p div ceil(M_u / R_rep)."""
    s_all, c_all = [], []
    for n, M in zip(L.unit_numel, L.unit_shard_numel):
        i = np.arange(n, dtype=np.int64)
        sub = -(-M // R_rep)
        s_all.append(i // M)
        c_all.append((i % M) // sub)
    return np.concatenate(s_all), np.concatenate(c_all)


def ring_order(owner: int, n: int) -> List[int]:
    """Order in which a ring reduce-scatter over n ranks adds the contributions to the chunk that rank `owner`
    ends up with: the chunk starts on the next rank and travels once around the ring, every rank adding its own
    part, so the owner's part is added last: owner+1, owner+2, ..., n-1, 0, ..., owner."""
    return [(owner + 1 + q) % n for q in range(n)]


def _sum_levels(grads, S: int, R_rep: int, sigma_order, rho_order, wire_bf16: bool) -> np.ndarray:
    """Two-level sum in the given visiting orders, then one division by K; fp32 result."""
    K = S * R_rep
    if wire_bf16:
        outer = np.zeros_like(np.asarray(grads[0], dtype=np.float64))
        for rho in rho_order:
            inner = np.zeros_like(outer)
            for sigma in sigma_order:
                inner = round_to_bf16((inner + np.asarray(grads[rho * S + sigma], dtype=np.float64)).astype(np.float32))
            outer = round_to_bf16((outer + inner).astype(np.float32))
        return round_to_bf16((outer / K).astype(np.float32)).astype(np.float32)
    outer = None
    for rho in rho_order:
        inner = None
        for sigma in sigma_order:
            x = np.asarray(grads[rho * S + sigma], dtype=np.float64)
            inner = x.copy() if inner is None else inner + x
        outer = inner if outer is None else outer + inner
    return (outer / K).astype(np.float32)


def reduce_mean(grads: Sequence[np.ndarray], S: int, R_rep: int = 1, wire_bf16: bool = False, ring=None) -> np.ndarray:
    """Mean gradient of one group, stored as fp32.

    grads: K = R_rep*S float64 arrays (exact input values), buffer rho*S+sigma.
    FSDP (R_rep = 1): the reduce-scatter sums the S rank gradients.
    HSDP: first the reduce-scatter inside each sharding group (over sigma), then
    the all-reduce across the R_rep replicas (over rho) -- shard level first,
    replicate level second.  Reading: the reduction is a mean (sum, then one
    division by K after the last level), kept in fp32 afterwards.

    wire_bf16: emulation of collectives that run in bf16 (the paper's runs are in
    bfloat16 and it attributes HSDP's different result to the order of floating-point
    operations): every partial sum and the final mean are rounded to bf16, so the
    two orders give different numbers.  Both levels start from zero, as on the GPU.

    ring: None visits the buffers in ascending index at both levels.  Otherwise the pair of integer arrays
    `ring_positions` returns (owner rank s and all-reduce sub-chunk c of every element): the order a ring
    produces.  The shard level adds sigma = s+1, s+2, ..., s (mod S); the replicate level, a ring all-reduce
    (reduce-scatter of R_rep sub-chunks, then all-gather), adds rho = c+1, ..., c (mod R_rep).  The sums are the
    same mathematically; with bf16 partial sums the start of the ring changes the rounding.
    """
    K = len(grads)
    assert K == S * R_rep and K >= 1
    if ring is None:
        return _sum_levels(grads, S, R_rep, range(S), range(R_rep), wire_bf16)
    s_idx, c_idx = ring
    out = np.zeros(np.asarray(grads[0]).shape, np.float32)
    for s in range(S):
        for c in range(R_rep):
            sel = (s_idx == s) & (c_idx == c)
            if sel.any():
                out[sel] = _sum_levels([np.asarray(g)[sel] for g in grads], S, R_rep, ring_order(s, S), ring_order(c, R_rep), wire_bf16)
    return out


def grad_norm(gbar: np.ndarray) -> float:
    """L2 norm of the whole group's mean gradient (all units together), in double."""
    total = 0.0
    g = np.asarray(gbar, dtype=np.float32)
    for lo in range(0, g.size, 1 << 20):
        c = g[lo:lo + (1 << 20)].astype(np.float64)
        total += float(np.dot(c, c))
    return math.sqrt(total)


def clip_coef(norm: float, max_grad_norm: float) -> float:
    """Global-norm clipping (the paper never mentions clipping; reading: scale the
    mean gradient by min(1, clip/(norm+1e-6)); clip <= 0 disables it)."""
    if not (max_grad_norm > 0.0):
        return 1.0
    c = max_grad_norm / (norm + CLIP_EPS)
    if math.isnan(c):
        return c                     # non-finite norms propagate, nothing is special-cased
    return c if c < 1.0 else 1.0


def adamw(theta, m, v, gbar, coef, t_new, lr, beta1, beta2, eps, weight_decay):
    """AdamW on stored fp32 state, double arithmetic, fp32 stores (Experimental
    Setup names only "AdamW"; reading: decoupled weight decay applied to theta
    first, bias-corrected moments, eps added outside the square root)."""
    th = np.asarray(theta, dtype=np.float32).astype(np.float64)
    m_ = np.asarray(m, dtype=np.float32).astype(np.float64)
    v_ = np.asarray(v, dtype=np.float32).astype(np.float64)
    g = coef * np.asarray(gbar, dtype=np.float32).astype(np.float64)
    th = th * (1.0 - lr * weight_decay)
    m_ = beta1 * m_ + (1.0 - beta1) * g
    v_ = beta2 * v_ + (1.0 - beta2) * g * g
    mhat = m_ / (1.0 - beta1 ** t_new)
    vhat = v_ / (1.0 - beta2 ** t_new)
    th = th - lr * mhat / (np.sqrt(vhat) + eps)
    th32 = th.astype(np.float32)
    return th32, m_.astype(np.float32), v_.astype(np.float32), f32_to_bf16_bits(th32)


@dataclass
class GroupState:
    """Logical fp32 state of one federation group plus its bf16 parameter copy."""
    theta: np.ndarray
    m: np.ndarray
    v: np.ndarray
    param_bf16: np.ndarray      # uint16 bit patterns


@dataclass
class Hyper:
    lr: float = 3e-4
    beta1: float = 0.9
    beta2: float = 0.95
    eps: float = 1e-8
    weight_decay: float = 0.1
    max_grad_norm: float = 1.0
    wire_bf16: bool = False        # bf16 emulation of the two reduction levels (see reduce_mean)
    ring: bool = False             # visit the buffers in the order a ring produces (see reduce_mean)


def sync_step_group(st: GroupState, grads: Sequence[np.ndarray], S: int, R_rep: int, t_new: int,
                    hp: Hyper, lr: Optional[float] = None, ring=None):
    """One local step of one group: reduce -> norm -> clip -> AdamW.  Returns
    (norm, coef, gbar).  Every federation group runs its steps on its own, without
    waiting for the others (Section FL+FSDP).  `ring`: see reduce_mean (needed when hp.ring)."""
    assert (ring is not None) == bool(hp.ring)
    gbar = reduce_mean(grads, S, R_rep, hp.wire_bf16, ring)
    nrm = grad_norm(gbar)
    c = clip_coef(nrm, hp.max_grad_norm)
    st.theta, st.m, st.v, st.param_bf16 = adamw(
        st.theta, st.m, st.v, gbar, c, t_new, hp.lr if lr is None else lr,
        hp.beta1, hp.beta2, hp.eps, hp.weight_decay)
    return nrm, c, gbar


# --------------------------------------------------------------------------- FedAvg
def fedavg_weights(sample_counts: Optional[Sequence[int]], G: int) -> np.ndarray:
    if sample_counts is None:
        sample_counts = [1] * G
    n = np.asarray(sample_counts, dtype=np.float64)
    assert n.size == G and (n >= 0).all() and n.sum() > 0
    return n / n.sum()


def fedavg_array(copies: Sequence[np.ndarray], w: np.ndarray) -> np.ndarray:
    """Weighted average of G corresponding copies, double accumulate in ascending
    group order, stored as fp32 (FedAvg combines the locally trained models into one by a
    weighted mean, Background "Federated Learning"; here shard by shard over the F groups)."""
    acc = None
    for g, x in enumerate(copies):
        term = w[g] * np.asarray(x, dtype=np.float32).astype(np.float64)
        acc = term if acc is None else acc + term
    return acc.astype(np.float32)


def fedavg(states: Sequence[GroupState], sample_counts: Optional[Sequence[int]] = None,
           opt_state: bool = False) -> None:
    """After the aggregation each shard holds the mean of the shards it corresponds to in
    the other federation groups (Section FL+FSDP): every group receives the same
    averaged parameters (and the bf16 copy of them).  Reading: w_g = n_g / sum n;
    m and v are averaged the same way only when `opt_state` is set."""
    G = len(states)
    w = fedavg_weights(sample_counts, G)
    th = fedavg_array([s.theta for s in states], w)
    bits = f32_to_bf16_bits(th)
    if opt_state:
        m = fedavg_array([s.m for s in states], w)
        v = fedavg_array([s.v for s in states], w)
    for s in states:
        s.theta = th.copy(); s.param_bf16 = bits.copy()
        if opt_state:
            s.m = m.copy(); s.v = v.copy()


def sync_step_replicated(replicas: Sequence[GroupState], grads: Sequence[np.ndarray], S: int, R_rep: int, t_new: int,
                         hp: Hyper, lr: Optional[float] = None, ring=None):
    """FL+HSDP with one state copy per replica: after the shard-level reduce-scatter and the all-reduce across
    the replicas every replica of the group holds the same mean gradient, and each applies the optimizer to its
    own copy of the shard (Background, HSDP).  `replicas`: the R_rep state copies of one group."""
    assert len(replicas) == R_rep
    out = None
    for st in replicas:
        out = sync_step_group(st, grads, S, R_rep, t_new, hp, lr, ring)
    return out


def fedavg_replicated(groups: Sequence[Sequence[GroupState]], sample_counts: Optional[Sequence[int]] = None,
                      opt_state: bool = False) -> None:
    """FedAvg of FL+HSDP (Section FL+HSDP): only one replica of every federation group takes part in the
    aggregation across the groups, after which it broadcasts the new parameters to the other replicas of its
    group.  groups[g][rho]; replica 0 of each group is the one that aggregates.  The broadcast copies the
    aggregated replica's parameters (and, with `opt_state`, its averaged m and v); without `opt_state` every
    replica keeps the moments of its own optimizer."""
    firsts = [reps[0] for reps in groups]
    fedavg(firsts, sample_counts, opt_state)
    for reps in groups:
        src = reps[0]
        for st in reps[1:]:
            st.theta = src.theta.copy(); st.param_bf16 = src.param_bf16.copy()
            if opt_state:
                st.m = src.m.copy(); st.v = src.v.copy()


def fedavg_outer(states: Sequence[GroupState], x_global: np.ndarray, buf: np.ndarray, sample_counts=None,
                 outer_lr: float = 1.0, momentum: float = 0.0, nesterov: bool = False):
    """Aggregation with an outer optimizer (the FedOpt family the paper's related work describes: AdamW inside
    the groups, SGD with (Nesterov) momentum outside; plain FedAvg is the case outer_lr = 1, momentum = 0).
    The weighted average of the groups is turned into a pseudo-gradient against the global copy:
        xbar = sum_g w_g x_g ;  delta = x_global - xbar ;  buf = momentum*buf + delta
        d = delta + momentum*buf  (Nesterov)  or  buf ;  x_global = x_global - outer_lr*d
    and every group restarts from x_global.  Double arithmetic, fp32 stores.  Returns (x_global, buf)."""
    G = len(states)
    w = fedavg_weights(sample_counts, G)
    xbar = np.zeros(np.asarray(x_global).shape, np.float64)
    for g, st in enumerate(states):
        xbar = xbar + w[g] * np.asarray(st.theta, dtype=np.float32).astype(np.float64)
    xg = np.asarray(x_global, dtype=np.float32).astype(np.float64)
    delta = xg - xbar
    b = momentum * np.asarray(buf, dtype=np.float32).astype(np.float64) + delta
    d = delta + momentum * b if nesterov else b
    xg = (xg - outer_lr * d).astype(np.float32)
    bits = f32_to_bf16_bits(xg)
    for st in states:
        st.theta = xg.copy(); st.param_bf16 = bits.copy()
    return xg, b.astype(np.float32)


# --------------------------------------------------------------------------- driver loop
def run(states: List[GroupState], grads_for_step, S: int, R_rep: int, H: int, n_steps: int, hp: Hyper,
        sample_counts=None, opt_state: bool = False, t0: int = 0):
    """for step: every group takes one local step; after every H-th step FedAvg (the
    aggregation period A of Section FL+FSDP; it follows that step's optimizer update).  grads_for_step(step, g)
    returns that group's K float64 gradient arrays (logical).  The step counter
    is global and is not reset by FedAvg.  Returns the per-step list of norms."""
    norms = []
    t = t0
    for _ in range(n_steps):
        t += 1
        row = []
        for g, st in enumerate(states):
            nrm, _, _ = sync_step_group(st, grads_for_step(t, g), S, R_rep, t, hp)
            row.append(nrm)
        norms.append(row)
        if t % H == 0:
            fedavg(states, sample_counts, opt_state)
    return norms


# --------------------------------------------------------------------------- communication-cost model
def cost_all_gather(D, n, B=1.0):
    return D * (n - 1) / (n * B)


def cost_reduce_scatter(D, n, B=1.0):
    return D * (n - 1) / (n * B)


def cost_all_reduce(D, n, B=1.0):
    return 2.0 * D * (n - 1) / (n * B)


def cost_broadcast(D, n, B=1.0):
    return D / B


def comm_costs(unit_shard_bytes: Sequence[float], S: int, R: int, F: int, A: int,
               B_S: float = 1.0, B_R: float = 1.0, B_F: float = 1.0) -> dict:
    """Eq. 1-5 written as the sums of collectives they are defined by (the left-hand
    forms), with the uniform M*L replaced by a sum over units.  With all
    bandwidths 1 the values are bytes per step; with real bandwidths, seconds.
    FL+HSDP with R = 1 costs what FL+FSDP costs (the fallback stated in Section FL+HSDP)."""
    fsdp = hsdp = fl = bc = 0.0
    for M in unit_shard_bytes:
        f = 2 * cost_all_gather(M, S, B_S) + cost_reduce_scatter(M, S, B_S)
        fsdp += f
        hsdp += f + cost_all_reduce(M, R, B_R)
        fl += cost_all_reduce(M, F, B_F) / A
        bc += cost_broadcast(M, R, B_R) / A
    fl_hsdp = hsdp + fl + bc if R > 1 else fsdp + fl
    return dict(fsdp=fsdp, hsdp=hsdp, fl=fl, fl_fsdp=fsdp + fl, fl_hsdp=fl_hsdp)
