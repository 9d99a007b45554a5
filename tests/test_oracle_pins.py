"""Pins for the CPU oracle: each test checks it against something other than itself --
exact rational brute force on tiny inputs, closed forms, a library routine for a
special case, invariants the method must satisfy, or the paper's printed closed
forms (cost model).  No GPU is used here."""
import json
import math
import os
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import fls_oracle as orc

HP = orc.Hyper()  # lr 3e-4, betas (0.9, 0.95), eps 1e-8, wd 0.1, clip 1.0
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng_bf16_bits(rng, n, sigma=1e-3):
    """Random bf16 bit patterns (uint16) built with torch's own RNE cast."""
    x = torch.from_numpy(rng.normal(0.0, sigma, n).astype(np.float32)).to(torch.bfloat16)
    return x.view(torch.int16).numpy().view(np.uint16).copy()


def frac_of_bf16(bits):
    """Exact rational value of one bf16 bit pattern, decoded field by field."""
    bits = int(bits)
    sign = -1 if bits >> 15 else 1
    e = (bits >> 7) & 0xFF
    f = bits & 0x7F
    assert e != 0xFF
    if e == 0:
        return sign * Fraction(f, 1 << 7) * Fraction(2) ** (-126)
    return sign * (1 + Fraction(f, 1 << 7)) * Fraction(2) ** (e - 127)


def f32_of_fraction(q):
    # Fraction -> nearest double -> nearest fp32 (the values used here are exact in double)
    return np.float32(float(q))


# ----------------------------------------------------------------------------- bf16 conversions
def test_bf16_decode_matches_field_decoding_and_torch():
    rng = np.random.default_rng(1)
    bits = rng.integers(0, 1 << 16, 4096, dtype=np.uint16)
    bits = bits[((bits >> 7) & 0xFF) != 0xFF]           # finite only
    got = orc.bf16_bits_to_f64(bits)
    want = np.array([float(frac_of_bf16(b)) for b in bits])
    assert np.array_equal(got, want)
    t = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(got, t)


def test_bf16_rounding_matches_torch_rne_including_ties_and_specials():
    rng = np.random.default_rng(2)
    x = rng.normal(0, 1, 20000).astype(np.float32)
    u = rng.integers(0, 1 << 32, 20000, dtype=np.uint64).astype(np.uint32).view(np.float32)
    ties = (rng.integers(0, 1 << 16, 5000, dtype=np.uint64).astype(np.uint32) << np.uint32(16) | np.uint32(0x8000)).view(np.float32)
    special = np.array([0.0, -0.0, np.inf, -np.inf, 3.3895314e38, 1e-45, -1e-45, 1.0, 1.00390625, 1.01171875], np.float32)
    allx = np.concatenate([x, u, ties, special])
    allx = allx[~np.isnan(allx)]
    got = orc.f32_to_bf16_bits(allx)
    want = torch.from_numpy(allx).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, want)
    nan_bits = orc.f32_to_bf16_bits(np.array([np.nan], np.float32))
    assert (int(nan_bits[0]) & 0x7F80) == 0x7F80 and (int(nan_bits[0]) & 0x7F) != 0


# ----------------------------------------------------------------------------- planner
@pytest.mark.parametrize("units,S,Q", [([17], 4, 1), ([17], 4, 8), ([5, 1, 12], 3, 1), ([5, 1, 12], 3, 4),
                                       ([1000003], 4, 1), ([7, 9, 64, 3], 8, 8), ([33], 1, 1)])
def test_planner_brute_force(units, S, Q):
    L = orc.plan(units, S, Q)
    # definition, enumerated element by element
    seen_u, seen_a = set(), set()
    for u, n in enumerate(units):
        M = L.unit_shard_numel[u]
        assert M % Q == 0 and M * S >= n and (M - Q) * S < n          # smallest multiple of Q that covers n
        for i in range(n):
            s, k = divmod(i, M)
            j = sum(L.unit_padded[:u]) + i
            a = s * L.shard_numel + sum(L.unit_shard_numel[:u]) + k
            seen_u.add(j); seen_a.add(a)
    assert len(seen_u) == L.n_params == len(seen_a)
    assert L.n_padded == sum(L.unit_padded) == S * L.shard_numel and L.n_padded % (S * Q) == 0
    logical = np.arange(1, L.n_params + 1, dtype=np.float32)
    pu, ps = orc.pack_unsharded(L, logical), orc.pack_sharded(L, logical)
    assert sorted(np.flatnonzero(pu)) == sorted(seen_u) and sorted(np.flatnonzero(ps)) == sorted(seen_a)
    assert np.array_equal(orc.unpack_unsharded(L, pu), logical) and np.array_equal(orc.unpack_sharded(L, ps), logical)
    # a rank's slice of a unit is contiguous in both orders
    p = 0
    for u, n in enumerate(units):
        M = L.unit_shard_numel[u]
        for s in range(S):
            lo, hi = s * M, min(n, (s + 1) * M)
            if lo < hi:
                seg = logical[p + lo:p + hi]
                j0 = L.unit_offset[u] + lo
                a0 = s * L.shard_numel + L.unit_shard_offset[u]
                assert np.array_equal(pu[j0:j0 + hi - lo], seg) and np.array_equal(ps[a0:a0 + hi - lo], seg)
        p += n


def test_addresses_of_matches_elementwise_definition():
    units, S, Q = [5, 1, 12, 7], 3, 4
    L = orc.plan(units, S, Q)
    j, a = orc.addresses_of(L, np.arange(sum(units)))
    p = 0
    for u, n in enumerate(units):
        for i in range(n):
            s_, k = divmod(i, L.unit_shard_numel[u])
            assert j[p] == sum(L.unit_padded[:u]) + i
            assert a[p] == s_ * L.shard_numel + sum(L.unit_shard_numel[:u]) + k
            p += 1
    jj, aa = orc.addresses_of(L, [24, 0, 17])
    assert list(jj) == [j[24], j[0], j[17]] and list(aa) == [a[24], a[0], a[17]]


def test_planner_p17_numbers():
    L = orc.plan([17], 4, 1)
    assert (L.n_padded, L.shard_numel, L.unit_shard_numel) == (20, 5, [5])
    L = orc.plan([1000003], 4, 1)
    assert (L.n_padded, L.shard_numel) == (1000004, 250001)
    L = orc.plan([1000003], 4, 8)
    assert (L.n_padded, L.shard_numel) == (1000032, 250008)
    # single unit: both physical orders coincide
    x = np.arange(17, dtype=np.float32)
    L = orc.plan([17], 4, 1)
    assert np.array_equal(orc.pack_sharded(L, x), orc.pack_unsharded(L, x))


# ----------------------------------------------------------------------------- reduce (FSDP and HSDP), P = 17
@pytest.mark.parametrize("S,R_rep", [(4, 1), (2, 2), (4, 2), (3, 1), (1, 1), (1, 3), (8, 8)])
def test_reduce_mean_brute_force_p17(S, R_rep):
    rng = np.random.default_rng(100 + S * 10 + R_rep)
    K = S * R_rep
    bits = [rng_bf16_bits(rng, 17) for _ in range(K)]
    got = orc.reduce_mean([orc.bf16_bits_to_f64(b) for b in bits], S, R_rep)
    for j in range(17):
        exact = sum(frac_of_bf16(bits[k][j]) for k in range(K)) / K     # the plain definition: the mean
        assert got[j] == f32_of_fraction(exact), (j, got[j], float(exact))
    assert got.dtype == np.float32


@pytest.mark.parametrize("S,R_rep", [(4, 1), (2, 2), (4, 2), (3, 1), (1, 3)])
def test_reduce_mean_bf16_wire_brute_force_p17(S, R_rep):
    """bf16-wire mode: every partial sum and the mean rounded to bf16, exact rationals + an independent
    nearest-even rounding (the one of the worked-case generator)."""
    from tests.golden.make_worked_cases import _round_to_bits
    r32 = lambda q: _round_to_bits(q, 23, -126)
    rb = lambda q: _round_to_bits(r32(q), 7, -126)       # an fp32 add/divide, then the bf16 store
    rng = np.random.default_rng(300 + S * 10 + R_rep)
    K = S * R_rep
    bits = [rng_bf16_bits(rng, 17, 1.0) for _ in range(K)]
    got = orc.reduce_mean([orc.bf16_bits_to_f64(b) for b in bits], S, R_rep, wire_bf16=True)
    for j in range(17):
        outer = Fraction(0)
        for rho in range(R_rep):
            inner = Fraction(0)
            for sigma in range(S):
                inner = rb(inner + frac_of_bf16(bits[rho * S + sigma][j]))
            outer = rb(outer + inner)
        assert Fraction(float(got[j])) == rb(outer / K), j
    # the values are bf16-representable, and close to (but in general not equal to) the fp32-accumulated mean
    assert np.array_equal(orc.round_to_bf16(got), got.astype(np.float64))
    plain = orc.reduce_mean([orc.bf16_bits_to_f64(b) for b in bits], S, R_rep)
    assert np.allclose(got, plain, rtol=2 ** -6, atol=0.03)       # a bf16 ulp of the O(1) partial sums


def test_bf16_wire_makes_the_two_orders_differ():
    """The paper's remark: FSDP's single reduction and HSDP's two-tier reduction are the same mathematically
    but not numerically in bf16.  In fp32 accumulation the two orders agree on these inputs; with bf16
    partial sums they do not."""
    rng = np.random.default_rng(77)
    g = [orc.bf16_bits_to_f64(rng_bf16_bits(rng, 4000, 1e-3)) for _ in range(8)]
    assert np.array_equal(orc.reduce_mean(g, 8, 1), orc.reduce_mean(g, 4, 2))
    a, b = orc.reduce_mean(g, 8, 1, wire_bf16=True), orc.reduce_mean(g, 4, 2, wire_bf16=True)
    assert 0.02 < np.mean(a != b) < 0.9
    assert np.allclose(a, b, rtol=2 ** -5, atol=1e-5)


def _ring_token_sum(values, owner, add):
    """A ring reduce-scatter written as message passing: the chunk that rank `owner` will hold starts as the
    value of the next rank, is handed from rank to rank once around the ring, and every rank it reaches adds its
    own value with `add`; the owner is reached last."""
    n = len(values)
    rank = (owner + 1) % n
    token = add(Fraction(0), values[rank])
    while rank != owner:
        rank = (rank + 1) % n
        token = add(token, values[rank])
    return token


@pytest.mark.parametrize("S,R_rep", [(2, 1), (3, 1), (4, 1), (2, 2), (3, 2), (4, 2)])
@pytest.mark.parametrize("wire", [True, False])
def test_reduce_mean_ring_order_brute_force_p17(S, R_rep, wire):
    """Ring order on P = 17 (padded shards of ceil(17/S) elements): element j belongs to rank s = j div M; inside
    that rank's slice it lies in sub-chunk c of R_rep for the all-reduce across replicas.  The expected value is
    the message-passing ring above in exact rationals, with the nearest-even rounding of the worked-case
    generator after every add when the wire is bf16; with fp32 partial sums it is the exactly rounded mean."""
    from tests.golden.make_worked_cases import _round_to_bits
    r32 = lambda q: _round_to_bits(q, 23, -126)
    rb = lambda q: _round_to_bits(r32(q), 7, -126)
    rng = np.random.default_rng(500 + S * 10 + R_rep)
    K = S * R_rep
    bits = [rng_bf16_bits(rng, 17, 1.0) for _ in range(K)]
    L = orc.plan([17], S, 1)
    ring = orc.ring_positions(L, R_rep)
    M = -(-17 // S)
    sub = -(-M // R_rep)
    got = orc.reduce_mean([orc.bf16_bits_to_f64(b) for b in bits], S, R_rep, wire_bf16=wire, ring=ring)
    add = (lambda a, b: rb(a + b)) if wire else (lambda a, b: a + b)
    for j in range(17):
        s, c = j // M, (j % M) // sub
        assert (ring[0][j], ring[1][j]) == (s, c)
        per_replica = [_ring_token_sum([frac_of_bf16(bits[rho * S + sigma][j]) for sigma in range(S)], s, add) for rho in range(R_rep)]
        total = _ring_token_sum(per_replica, c, add)
        want = rb(total / K) if wire else total / K
        assert (Fraction(float(got[j])) == want) if wire else (got[j] == f32_of_fraction(want)), (j, s, c)
    if wire:
        asc = orc.reduce_mean([orc.bf16_bits_to_f64(b) for b in bits], S, R_rep, wire_bf16=True)
        assert np.allclose(got, asc, rtol=2 ** -6, atol=0.03)           # same sum, other rounding


def test_ring_order_changes_bf16_sums_but_not_fp32_sums():
    rng = np.random.default_rng(78)
    g = [orc.bf16_bits_to_f64(rng_bf16_bits(rng, 4096, 1e-3)) for _ in range(8)]
    for S, R_rep in ((8, 1), (4, 2)):
        ring = orc.ring_positions(orc.plan([4096], S, 8), R_rep)
        assert np.array_equal(orc.reduce_mean(g, S, R_rep, ring=ring), orc.reduce_mean(g, S, R_rep))
        a, b = orc.reduce_mean(g, S, R_rep, True, ring), orc.reduce_mean(g, S, R_rep, True)
        # rank S-1 of the shard level (and sub-chunk R_rep-1) visits the buffers in ascending order anyway
        last = (ring[0] == S - 1) & (ring[1] == R_rep - 1)
        assert np.array_equal(a[last], b[last]) and 0.02 < np.mean(a[~last] != b[~last]) < 0.9
    assert orc.ring_order(2, 4) == [3, 0, 1, 2] and orc.ring_order(0, 1) == [0] and orc.ring_order(3, 4) == [0, 1, 2, 3]


def test_ring_positions_on_several_units():
    L = orc.plan([10, 3, 8], 2, 1)          # shard lengths 5, 2, 4
    s, c = orc.ring_positions(L, 2)
    want_s, want_c = [], []
    for n, M in zip([10, 3, 8], [5, 2, 4]):
        for i in range(n):
            want_s.append(i // M)
            want_c.append((i % M) // (-(-M // 2)))
    assert s.tolist() == want_s and c.tolist() == want_c
    assert max(want_c) == 1 and c[:10].tolist() == [0, 0, 0, 1, 1, 0, 0, 0, 1, 1]


def test_reduce_special_cases():
    rng = np.random.default_rng(7)
    g = [orc.bf16_bits_to_f64(rng_bf16_bits(rng, 1000)) for _ in range(8)]
    assert np.array_equal(orc.reduce_mean(g[:1], 1, 1), g[0].astype(np.float32))            # K = 1: identity
    flat = orc.reduce_mean(g, 8, 1)
    assert np.array_equal(flat, orc.reduce_mean(g, 8, 1))
    two = orc.reduce_mean(g, 4, 2)
    # two-level and flat orders are the same mean: equal to rounding (here bf16 inputs: exactly)
    assert np.allclose(two, flat, rtol=1e-7, atol=0)
    perm = [g[i] for i in rng.permutation(8)]
    assert np.allclose(orc.reduce_mean(perm, 8, 1), flat, rtol=1e-7, atol=0)
    # a dropped buffer or a sum instead of a mean must show
    assert not np.allclose(orc.reduce_mean(g[:7] + [np.zeros(1000)], 8, 1), flat, rtol=1e-3, atol=0)
    assert np.allclose(flat.astype(np.float64) * 8, np.sum(g, axis=0), rtol=1e-6)
    # HSDP indexing: buffer rho*S+sigma; with fp64-exact inputs where order matters the
    # level structure is visible: (a + b) + (c + d) with a = 1, b = 2^-60, c = -1, d = 2^-60
    a, b = np.array([1.0]), np.array([2.0 ** -60])
    lvl = orc.reduce_mean([a, b, -a, b], 2, 2)     # (1 + 2^-60) + (-1 + 2^-60) -> both inner sums lose the 2^-60 -> 0
    flt = orc.reduce_mean([a, b, -a, b], 4, 1)     # ((1 + 2^-60) - 1) + 2^-60 = 2^-60
    assert lvl[0] == 0.0 and flt[0] == np.float32(2.0 ** -60 / 4)


def test_reduce_mean_of_fp32_inputs_that_cancel_is_the_exactly_rounded_mean():
    """fp32 inputs around 1e-3 whose mean is around 1e-8: the result is the exact rational mean rounded once to fp32
    (an fp32 running sum is off by a large fraction of such a mean, which AdamW's division by sqrt(v)+eps would amplify)."""
    rng = np.random.default_rng(41)
    for S, R_rep in ((2, 3), (8, 1), (5, 1)):
        K = S * R_rep
        x = [rng.normal(0, 1e-3, 64).astype(np.float32) for _ in range(K - 1)]
        x.append((rng.normal(0, 1e-8, 64) * K - np.sum([a.astype(np.float64) for a in x], axis=0)).astype(np.float32))
        got = orc.reduce_mean([a.astype(np.float64) for a in x], S, R_rep)
        running = np.zeros(64, np.float32)
        for a in x:
            running = running + a
        running = running / np.float32(K)
        for j in range(64):
            exact = sum(Fraction(float(a[j])) for a in x) / K
            assert got[j] == f32_of_fraction(exact), (S, R_rep, j)
        assert np.median(np.abs(got)) < 1e-7 and np.mean(running != got) > 0.5


# ----------------------------------------------------------------------------- norm and clip
def test_norm_closed_forms():
    a = np.float32(0.00390625)                                     # 2^-8, exact
    assert orc.grad_norm(np.full(1 << 22, a, np.float32)) == float(a) * 2048.0          # |a| sqrt(N), N = 2^22
    one_hot = np.zeros(3_000_001, np.float32); one_hot[2_999_999] = -3.5
    assert orc.grad_norm(one_hot) == 3.5
    assert orc.grad_norm(np.array([3, 4], np.float32)) == 5.0
    rng = np.random.default_rng(3)
    x = rng.normal(0, 1e-3, 2_500_000).astype(np.float32)
    assert math.isclose(orc.grad_norm(x), math.sqrt(math.fsum(float(v) ** 2 for v in x[:200000]) +
                                                    float(np.sum(x[200000:].astype(np.float64) ** 2))), rel_tol=1e-12)
    assert math.isclose(orc.grad_norm(x), float(np.linalg.norm(x.astype(np.float64))), rel_tol=1e-12)


def test_clip_coef_cases():
    assert orc.clip_coef(0.5, 1.0) == 1.0                          # below the threshold: inactive
    assert orc.clip_coef(5.0, 1.0) == 1.0 / (5.0 + 1e-6)
    assert orc.clip_coef(5.0, 0.0) == 1.0 and orc.clip_coef(5.0, -1.0) == 1.0
    assert orc.clip_coef(1.0, 1.0) == 1.0 / (1.0 + 1e-6)           # at the threshold the 1e-6 term already bites
    assert orc.clip_coef(float("inf"), 1.0) == 0.0
    assert math.isnan(orc.clip_coef(float("nan"), 1.0))
    # agrees with the library's rule on a real tensor
    g = torch.tensor([3.0, 4.0], dtype=torch.float64)
    p = torch.nn.Parameter(torch.zeros(2, dtype=torch.float64)); p.grad = g.clone()
    torch.nn.utils.clip_grad_norm_([p], 1.0)
    assert torch.allclose(p.grad, g * orc.clip_coef(5.0, 1.0), rtol=1e-15, atol=0)


# ----------------------------------------------------------------------------- AdamW
def test_adamw_first_step_closed_form():
    """From m = v = 0 the first step has a closed form: m1 = (1-b1) g, v1 = (1-b2) g^2,
    theta1 = theta0 (1 - lr wd) - lr g / (|g| + eps)."""
    rng = np.random.default_rng(11)
    n = 5000
    th0 = rng.normal(0, 0.02, n).astype(np.float32)
    g = rng.normal(0, 1e-3, n).astype(np.float32)
    g[:5] = [0.0, 1e-12, -1e-12, 1e-8, -3.0]                       # |g| << eps, |g| = eps, large
    c = 0.37
    z = np.zeros(n, np.float32)
    th1, m1, v1, bits = orc.adamw(th0, z, z, g, c, 1, HP.lr, HP.beta1, HP.beta2, HP.eps, HP.weight_decay)
    gd = c * g.astype(np.float64)
    want_th = th0.astype(np.float64) * (1 - HP.lr * HP.weight_decay) - HP.lr * gd / (np.abs(gd) + HP.eps)
    ulp = np.spacing(np.abs(want_th).astype(np.float32)).astype(np.float64)
    assert np.all(np.abs(th1.astype(np.float64) - want_th) <= 0.5000001 * ulp)
    assert np.allclose(m1, (1 - HP.beta1) * gd, rtol=1e-7, atol=0) and np.allclose(v1, (1 - HP.beta2) * gd * gd, rtol=1e-7, atol=1e-45)
    assert np.array_equal(bits, torch.from_numpy(th1).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))
    # eps sits outside the square root: for |g| = eps the update is lr/2, not lr/sqrt(2)
    k = 3
    assert math.isclose(float(th0[k]) * (1 - HP.lr * HP.weight_decay) - float(th1[k]), HP.lr * (c * 1e-8) / (c * 1e-8 + 1e-8), rel_tol=1e-4)


@pytest.mark.parametrize("eps,gs", [(1e-8, 1e-3), (1e-4, 1e-4)])
def test_adamw_and_clip_match_torch_library_over_steps(eps, gs):
    """K = 1, G = 1 reduces to torch.optim.AdamW + clip_grad_norm_ (run in float64 so that
    only the oracle's fp32 stores separate the two)."""
    rng = np.random.default_rng(12)
    n, steps = 4096, 6
    th0 = rng.normal(0, 0.02, n).astype(np.float32)
    hp = orc.Hyper(eps=eps, max_grad_norm=50 * gs)   # norms alternate between ~192 gs and ~19 gs
    st = orc.GroupState(th0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32), None)
    p = torch.nn.Parameter(torch.from_numpy(th0.astype(np.float64)))
    opt = torch.optim.AdamW([p], lr=hp.lr, betas=(hp.beta1, hp.beta2), eps=hp.eps, weight_decay=hp.weight_decay)
    active = []
    for t in range(1, steps + 1):
        bits = rng_bf16_bits(rng, n, gs * (3.0 if t % 2 else 0.3))
        g = orc.bf16_bits_to_f64(bits)
        nrm, c, _ = orc.sync_step_group(st, [g], 1, 1, t, hp)
        active.append(c < 1.0)
        p.grad = torch.from_numpy(g.copy())
        tn = torch.nn.utils.clip_grad_norm_([p], hp.max_grad_norm)
        assert math.isclose(float(tn), nrm, rel_tol=1e-12)
        opt.step()
        state = opt.state[p]
        # the fp32 stores cost half an ulp of the value held at that step; a value that has since
        # moved towards zero keeps the older, larger error, hence the floor on the ulp's argument
        for got, want, floor in ((st.theta, p.detach().numpy(), hp.lr * t),
                                 (st.m, state["exp_avg"].numpy(), float(np.median(np.abs(st.m)))),
                                 (st.v, state["exp_avg_sq"].numpy(), float(np.median(st.v)))):
            ulp = np.spacing(np.maximum(np.abs(want), floor).astype(np.float32)).astype(np.float64)
            assert np.all(np.abs(got.astype(np.float64) - want) <= 2 * t * ulp), t
    assert any(active) and not all(active)      # both branches of the clamp were taken


def test_worked_cases_exact_rational():
    """Small cases worked out with exact rational arithmetic by tests/golden/make_worked_cases.py
    (which uses neither the oracle nor the CUDA path)."""
    cases = json.load(open(os.path.join(GOLDEN, "worked_cases.json")))
    from tests.golden import make_worked_cases
    assert make_worked_cases.build() == cases, "golden file is stale: rerun tests/golden/make_worked_cases.py"
    hexf = lambda a: [float(x).hex() for x in np.asarray(a, np.float32)]
    for c in cases["sync"]:
        theta = np.array([float.fromhex(h) for h in c["theta0"]], np.float32)
        st = orc.GroupState(theta, np.zeros_like(theta), np.zeros_like(theta), None)
        for step in c["steps"]:
            grads = [orc.bf16_bits_to_f64(np.array(b, np.uint16)) for b in c["grad_bits"]]
            nrm, coef, _ = orc.sync_step_group(st, grads, c["S"], c["R_rep"], step["t"], HP)
            assert hexf(st.theta) == step["theta"] and hexf(st.m) == step["m"] and hexf(st.v) == step["v"]
            assert [int(b) for b in st.param_bf16] == step["bf16"]
            assert math.isclose(nrm, step["norm"], rel_tol=1e-15) and math.isclose(coef, step["coef"], rel_tol=1e-15)
    for c in cases["fedavg"]:
        sts = [orc.GroupState(np.array([float.fromhex(h) for h in col], np.float32), None, None, None) for col in c["copies"]]
        orc.fedavg(sts, c["counts"])
        for s in sts:
            assert hexf(s.theta) == c["avg"] and [int(b) for b in s.param_bf16] == c["bf16"]


# ----------------------------------------------------------------------------- FedAvg
def test_fedavg_brute_force_p17_and_invariants():
    rng = np.random.default_rng(21)
    G, n = 5, 17
    copies = [rng.normal(0, 0.02, n).astype(np.float32) for _ in range(G)]
    counts = [int(c) for c in rng.integers(1, 1001, G)]
    sts = [orc.GroupState(c.copy(), c.copy() * 2, np.abs(c), None) for c in copies]
    orc.fedavg(sts, counts, opt_state=True)
    tot = sum(counts)
    for j in range(n):
        exact = sum(Fraction(counts[g], tot) * Fraction(float(copies[g][j])) for g in range(G))
        # weights are rounded to double first, so allow one ulp of fp32 around the exact weighted mean
        assert abs(Fraction(float(sts[0].theta[j])) - exact) <= Fraction(float(np.spacing(np.float32(abs(float(exact)))))), j
        lo, hi = min(c[j] for c in copies), max(c[j] for c in copies)
        assert lo <= sts[0].theta[j] <= hi
    for s in sts[1:]:
        assert np.array_equal(s.theta, sts[0].theta) and np.array_equal(s.m, sts[0].m) and np.array_equal(s.v, sts[0].v)
        assert np.array_equal(s.param_bf16, sts[0].param_bf16)
    assert np.allclose(sts[0].m, 2 * sts[0].theta.astype(np.float64), rtol=1e-6)      # linear in the input
    before = sts[0].theta.copy()
    orc.fedavg(sts, counts, opt_state=True)                                              # idempotent up to rounding
    assert np.allclose(sts[0].theta, before, rtol=2e-7, atol=0)


def test_fedavg_identity_cases():
    rng = np.random.default_rng(22)
    x = rng.normal(0, 0.02, 1000).astype(np.float32)
    one = [orc.GroupState(x.copy(), x.copy(), x.copy(), None)]
    orc.fedavg(one, [123])
    assert np.array_equal(one[0].theta, x)                                               # G = 1: bit-exact identity
    same = [orc.GroupState(x.copy(), x.copy(), x.copy(), None) for _ in range(4)]
    orc.fedavg(same, [1, 2, 3, 4])
    assert np.allclose(same[0].theta, x, rtol=1.2e-7, atol=0)                            # identical copies: identity
    eq = [orc.GroupState(x.copy(), x.copy(), x.copy(), None) for _ in range(4)]
    orc.fedavg(eq, None)
    assert np.array_equal(eq[0].theta, x)                                                # weights 1/4: exact
    # params only: m and v are left alone
    a = [orc.GroupState(x.copy(), x * g, x * g, None) for g in range(1, 4)]
    orc.fedavg(a, None, opt_state=False)
    assert all(np.array_equal(a[g - 1].m, x * g) for g in range(1, 4))
    # equal weights: invariant under a permutation of the groups
    ys = [rng.normal(0, 0.02, 500).astype(np.float32) for _ in range(4)]
    s1 = [orc.GroupState(y.copy(), None, None, None) for y in ys]
    s2 = [orc.GroupState(y.copy(), None, None, None) for y in ys[::-1]]
    orc.fedavg(s1); orc.fedavg(s2)
    assert np.allclose(s1[0].theta, s2[0].theta, rtol=2e-7, atol=0)


def test_replicated_state_copies_stay_identical_and_match_the_single_copy():
    """FL+HSDP with one state copy per replica: every replica of a group applies the same mean gradient, so the
    copies stay bit-identical; the aggregation reads one replica per group and its broadcast makes all R_rep
    copies of every group equal to what plain FedAvg over one copy per group gives."""
    rng = np.random.default_rng(41)
    G, S, R_rep, n = 3, 2, 2, 300
    hp = orc.Hyper(max_grad_norm=0.01)
    th0 = rng.normal(0, 0.02, n).astype(np.float32)
    z = np.zeros(n, np.float32)
    single = [orc.GroupState(th0.copy(), z.copy(), z.copy(), None) for _ in range(G)]
    repl = [[orc.GroupState(th0.copy(), z.copy(), z.copy(), None) for _ in range(R_rep)] for _ in range(G)]
    counts = [3, 1, 5]
    for opt_state in (False, True):
        for t in (1, 2):
            for g in range(G):
                grads = [orc.bf16_bits_to_f64(rng_bf16_bits(rng, n)) for _ in range(S * R_rep)]
                a = orc.sync_step_group(single[g], grads, S, R_rep, t, hp)
                b = orc.sync_step_replicated(repl[g], grads, S, R_rep, t, hp)
                assert a[0] == b[0] and a[1] == b[1]
                for st in repl[g]:
                    assert np.array_equal(st.theta, single[g].theta) and np.array_equal(st.v, single[g].v)
        assert not np.array_equal(repl[0][1].theta, repl[1][1].theta)      # groups have diverged
        orc.fedavg(single, counts, opt_state)
        orc.fedavg_replicated(repl, counts, opt_state)
        for g in range(G):
            for st in repl[g]:
                assert np.array_equal(st.theta, single[g].theta) and np.array_equal(st.param_bf16, single[g].param_bf16)
                assert np.array_equal(st.m, single[g].m) and np.array_equal(st.v, single[g].v)
        assert np.array_equal(repl[0][1].theta, repl[2][0].theta)
        assert np.array_equal(repl[0][1].m, repl[2][0].m) == opt_state     # moments are shared only when averaged
    # a replica that did not take part must still receive the broadcast: corrupt one, aggregate, all equal again
    repl[1][1].theta = repl[1][1].theta + 1.0
    orc.fedavg_replicated(repl, counts, False)
    assert all(np.array_equal(st.theta, repl[0][0].theta) for reps in repl for st in reps)


def test_fedavg_outer_special_case_and_torch_sgd():
    """Outer optimizer: lr 1 / momentum 0 is plain FedAvg; in general it is torch.optim.SGD (momentum, Nesterov)
    on the pseudo-gradient x_global - xbar, followed over several rounds."""
    rng = np.random.default_rng(23)
    n, G = 3000, 4
    counts = [int(c) for c in rng.integers(1, 1001, G)]
    xg0 = rng.normal(0, 0.02, n).astype(np.float32)
    def groups(r):
        return [orc.GroupState((xg0 + rng.normal(0, 1e-3, n)).astype(np.float32), None, None, None) for _ in range(G)]
    # special case
    sts = groups(0)
    plain = [orc.GroupState(s.theta.copy(), None, None, None) for s in sts]
    orc.fedavg(plain, counts)
    xg, buf = orc.fedavg_outer(sts, xg0, np.zeros(n, np.float32), counts, outer_lr=1.0, momentum=0.0)
    assert np.allclose(xg, plain[0].theta, rtol=0, atol=4e-9) and all(np.array_equal(s.theta, xg) for s in sts)
    # against the library optimizer, three rounds
    for nesterov in (False, True):
        p = torch.nn.Parameter(torch.from_numpy(xg0.astype(np.float64)))
        opt = torch.optim.SGD([p], lr=0.7, momentum=0.9, nesterov=nesterov)
        xg, buf = xg0.copy(), np.zeros(n, np.float32)
        for r in range(3):
            sts = [orc.GroupState((xg + rng.normal(0, 1e-3, n)).astype(np.float32), None, None, None) for _ in range(G)]
            w = np.asarray(counts, np.float64) / sum(counts)
            xbar = sum(w[g] * sts[g].theta.astype(np.float64) for g in range(G))
            p.grad = p.detach() - torch.from_numpy(xbar)
            opt.step()
            xg, buf = orc.fedavg_outer(sts, xg, buf, counts, outer_lr=0.7, momentum=0.9, nesterov=nesterov)
            assert np.allclose(xg, p.detach().numpy(), rtol=0, atol=2e-8 * (r + 1))
            assert np.array_equal(sts[2].param_bf16, orc.f32_to_bf16_bits(xg))


# ----------------------------------------------------------------------------- whole loop
def _make_states(rng, G, n):
    th = rng.normal(0, 0.02, n).astype(np.float32)
    return [orc.GroupState(th.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32), orc.f32_to_bf16_bits(th)) for _ in range(G)]


def test_g1_is_plain_fsdp():
    """One federation group: FedAvg is the identity, so the loop is plain FSDP."""
    n, K = 3000, 4
    grads = {t: [orc.bf16_bits_to_f64(rng_bf16_bits(np.random.default_rng(1000 + t * 10 + k), n, 2e-2)) for k in range(K)] for t in range(1, 7)}
    a = _make_states(np.random.default_rng(5), 1, n)
    b = _make_states(np.random.default_rng(5), 1, n)
    orc.run(a, lambda t, g: grads[t], K, 1, 2, 6, HP, sample_counts=[17])
    orc.run(b, lambda t, g: grads[t], K, 1, 10 ** 9, 6, HP)          # FedAvg never fires
    assert np.array_equal(a[0].theta, b[0].theta) and np.array_equal(a[0].m, b[0].m) and np.array_equal(a[0].v, b[0].v)
    assert np.array_equal(a[0].param_bf16, b[0].param_bf16)


def test_h1_equal_weights_equals_fsdp_over_all_replicas():
    """H = 1 with equal weights equals FSDP over R*G replicas when every group sees the same
    mean gradient (group g's buffer r is group 0's buffer (r+g) mod R): then all groups take the
    same step and averaging them changes nothing.  With different group gradients the two
    differ, because AdamW and clipping are not linear in the gradient (checked as well)."""
    n, R, G, steps = 2000, 4, 3, 5
    base = {t: [orc.bf16_bits_to_f64(rng_bf16_bits(np.random.default_rng(2000 + t * 10 + k), n, 2e-2)) for k in range(R)] for t in range(1, steps + 1)}
    fl = _make_states(np.random.default_rng(6), G, n)
    orc.run(fl, lambda t, g: [base[t][(r + g) % R] for r in range(R)], R, 1, 1, steps, HP, None, opt_state=True)
    big = _make_states(np.random.default_rng(6), 1, n)
    orc.run(big, lambda t, g: [base[t][k % R] for k in range(R * G)], R * G, 1, 10 ** 9, steps, HP)
    for s in fl:
        assert np.allclose(s.theta, big[0].theta, rtol=0, atol=1e-8)
        assert np.allclose(s.m, big[0].m, rtol=1e-5, atol=1e-12) and np.allclose(s.v, big[0].v, rtol=1e-5, atol=1e-18)
    # negative example: independent group gradients -> parameter averaging != gradient averaging
    other = {t: [[orc.bf16_bits_to_f64(rng_bf16_bits(np.random.default_rng(3000 + t * 100 + g * 10 + k), n, 2e-2)) for k in range(R)]
                 for g in range(G)] for t in range(1, steps + 1)}
    fl2 = _make_states(np.random.default_rng(6), G, n)
    orc.run(fl2, lambda t, g: other[t][g], R, 1, 1, steps, HP, None, opt_state=True)
    big2 = _make_states(np.random.default_rng(6), 1, n)
    orc.run(big2, lambda t, g: [other[t][k // R][k % R] for k in range(R * G)], R * G, 1, 10 ** 9, steps, HP)
    assert np.max(np.abs(fl2[0].theta - big2[0].theta)) > 1e-5


def test_padding_and_alignment_quantum_do_not_change_logical_results():
    rng = np.random.default_rng(31)
    units = [5, 1, 12]
    logical = rng.normal(0, 1, 18).astype(np.float32)
    for S, Q in [(3, 1), (3, 4), (2, 8)]:
        L = orc.plan(units, S, Q)
        assert np.array_equal(orc.unpack_sharded(L, orc.pack_sharded(L, logical)), logical)
        assert np.count_nonzero(orc.pack_sharded(L, logical)) == np.count_nonzero(logical)
    # zero padding is inert: zero gradient on zero state stays zero under AdamW (weight decay included)
    z = np.zeros(4, np.float32)
    th, m, v, bits = orc.adamw(z, z, z, z, 0.3, 5, HP.lr, HP.beta1, HP.beta2, HP.eps, HP.weight_decay)
    assert not th.any() and not m.any() and not v.any() and not bits.any()


def test_step_counter_and_resume():
    n, K = 500, 2
    grads = {t: [orc.bf16_bits_to_f64(rng_bf16_bits(np.random.default_rng(4000 + t * 10 + k), n)) for k in range(K)] for t in range(1, 5)}
    a = _make_states(np.random.default_rng(8), 2, n)
    orc.run(a, lambda t, g: grads[t], K, 1, 2, 4, HP)
    b = _make_states(np.random.default_rng(8), 2, n)
    orc.run(b, lambda t, g: grads[t], K, 1, 2, 2, HP)
    orc.run(b, lambda t, g: grads[t], K, 1, 2, 2, HP, t0=2)
    assert np.array_equal(a[0].theta, b[0].theta) and np.array_equal(a[1].v, b[1].v)


# ----------------------------------------------------------------------------- cost model (Eq. 1-5, Table 2)
def test_comm_costs_match_printed_closed_forms():
    """The right-hand sides printed in Eq. 1-5 / the 2x2 cost table, typed from the paper,
    against the oracle's sums of collectives."""
    rng = np.random.default_rng(41)
    for _ in range(50):
        S, R, F, A = (int(x) for x in rng.integers(2, 65, 4))
        L_ = int(rng.integers(1, 40)); M = float(rng.integers(1, 10 ** 9))
        BS, BR, BF = (float(x) for x in rng.uniform(1e9, 1e12, 3))
        got = orc.comm_costs([M] * L_, S, R, F, A, BS, BR, BF)
        ML = M * L_
        want = dict(
            fsdp=ML * (3 * (S - 1) / (S * BS)),
            hsdp=ML * (3 * (S - 1) / (S * BS) + 2 * (R - 1) / (R * BR)),
            fl=ML * ((1 / A) * (2 * (F - 1) / (F * BF))),
            fl_fsdp=ML * (3 * (S - 1) / (S * BS) + (1 / A) * (2 * (F - 1) / (F * BF))),
            fl_hsdp=ML * (3 * (S - 1) / (S * BS) + 2 * (R - 1) / (R * BR) + (1 / A) * (2 * (F - 1) / (F * BF) + 1 / BR)),
        )
        for k in want:
            assert math.isclose(got[k], want[k], rel_tol=1e-12), k


def test_comm_costs_degenerate_cases():
    M = [1000.0, 24.0]
    c = orc.comm_costs(M, 8, 1, 4, 8)
    assert c["fl_hsdp"] == c["fl_fsdp"] and c["hsdp"] == c["fsdp"]            # R = 1: FL+HSDP falls back to FL+FSDP
    c = orc.comm_costs(M, 8, 2, 1, 1)
    assert c["fl"] == 0.0 and c["fl_fsdp"] == c["fsdp"]                        # F = 1, A = 1: not federated
    assert orc.comm_costs(M, 1, 1, 1, 1)["fsdp"] == 0.0                         # S = 1: not sharded
    big = orc.comm_costs(M, 8, 2, 4, 10 ** 12)
    assert math.isclose(big["fl_hsdp"], big["hsdp"], rel_tol=1e-9)              # A -> infinity
    assert orc.cost_all_reduce(10.0, 4) == 2 * orc.cost_reduce_scatter(10.0, 4) == 15.0
    assert orc.cost_all_gather(10.0, 4) == 7.5 and orc.cost_broadcast(10.0, 4, 2.0) == 5.0
