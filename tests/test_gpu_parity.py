"""GPU parity: the CUDA library against the CPU oracle, element by element, on the same seeded
inputs, through the C ABI.  Tolerances: |d| <= 1e-6*max(1,|x|) on fp32 master/m/v (plus a relative
gate on m and v, whose magnitudes make the absolute gate weak); the bf16 copy within 1 bf16 ulp (plus
the fp32 tolerance where a bf16 ulp is smaller than it) and bit-exactly the rounding of the GPU's own
fp32 master."""
import math
import os

import numpy as np
import pytest
import torch

import synthetic as sy
from oracle import fls_oracle as orc
from tests.harness import Case, assert_bf16_close, assert_state_close, bf16_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fls():
    from paper_2609_20359_b200 import build
    build.build()
    import paper_2609_20359_b200._binding as b
    return b


def test_generator_is_bit_identical_on_cpu_and_gpu():
    key = sy.stream_key(77, sy.KIND_GRAD, 3, 1, 2)
    for dt in (torch.float32, torch.bfloat16):
        a = sy.normal_fill_(torch.empty(300_001, dtype=dt), key, 1e-3, 1.37, start=12345)
        b = sy.normal_fill_(torch.empty(300_001, dtype=dt, device="cuda"), key, 1e-3, 1.37, start=12345)
        assert torch.equal(a.view(torch.int16 if dt == torch.bfloat16 else torch.int32),
                           b.cpu().view(torch.int16 if dt == torch.bfloat16 else torch.int32))
    idx = torch.tensor([0, 1, 299_999, 12, 7_000_000_000], dtype=torch.int64)
    assert torch.equal(sy.normal_at(idx, key, 1e-3), sy.normal_at(idx.cuda(), key, 1e-3).cpu())


# ------------------------------------------------------------------ the tiny FL+FSDP workload
@pytest.mark.parametrize("Q,clip,resident", [(1, 1.0, -1), (8, 1.0, -1), (8, 0.1, -1), (1, 1.0, 0), (8, 0.1, 0)])
def test_tiny_fl_fsdp_8_steps(fls, Q, clip, resident):
    """P = 1,000,003, G = 2, K = S = 4, H = 4, 8 steps, equal weights.  Q = 1 pads to a multiple of
    S only (shard length 250,001: the buffer tail leaves the vector path); clip 1.0 is inactive
    (norm ~ 0.5), clip 0.1 is active.  resident -1: the library's default for a plan of this size (one cooperative
    kernel per step); 0: the reduce and AdamW kernels."""
    cfg = sy.CONFIGS[0]
    hp = orc.Hyper(max_grad_norm=clip)
    c = Case(cfg["unit_numel"], cfg["groups"], cfg["shard_dim"], 1, cfg["sync_period"], Q, seed=cfg["seed"], hp=hp, resident=resident)
    assert fls.fls_plan_get_resident(c.sess.plan) == (resident == -1)
    active = []
    for _ in range(cfg["steps"]):
        row = c.step()
        active += [co < 1.0 for _, co in row]
        c.compare()
    assert all(active) if clip < 0.5 else not any(active)
    # after the last FedAvg (step 8) all groups hold the same parameters, bit for bit
    assert torch.equal(c.sess.master[0], c.sess.master[1]) and torch.equal(c.sess.param_bf16[0], c.sess.param_bf16[1])
    assert c.sess.status() == 0
    c.close()


# ------------------------------------------------------------------ layouts, reduction orders, dtypes
@pytest.mark.parametrize("units,G,S,R_rep,Q,dtype", [
    ([17], 2, 4, 1, 1, "bf16"),                         # the brute-force size
    ([1], 1, 1, 1, 1, "bf16"),                          # a single parameter
    ([5000, 1, 12345, 2048, 77], 2, 4, 1, 8, "bf16"),   # several units, aligned shards, ragged tiles
    ([5000, 1, 12345, 2048, 77], 2, 3, 1, 1, "bf16"),   # unaligned shards: element-wise path
    ([40000, 30011], 2, 4, 2, 8, "bf16"),               # two-level order, K = 8
    ([40000, 30011], 1, 8, 8, 8, "bf16"),               # K = 64
    ([40000, 30011], 2, 3, 1, 8, "bf16"),               # K = 3: mean is not a power-of-two scale
    ([40000, 30011], 2, 5, 2, 8, "f32"),                # fp32 gradients, K = 10 (two load batches)
    ([70001], 3, 2, 2, 1, "f32"),                       # fp32 gradients, unaligned tail
    ([300000], 1, 1, 1, 8, "bf16"),                     # K = 1: plain AdamW on the gradient itself
])
@pytest.mark.parametrize("resident", [-1, 0])
def test_layouts_and_orders(fls, units, G, S, R_rep, Q, dtype, resident):
    """resident -1: the default route (the shapes with K in {1, 2, 4, 8} and a static order run as one cooperative kernel);
    0: the reduce and AdamW kernels for all of them."""
    hp = orc.Hyper(max_grad_norm=0.05)
    c = Case(units, G, S, R_rep, H=2, Q=Q, grad_dtype=dtype, opt_state=True, hp=hp, per_buffer_scale=True, resident=resident)
    counts = [sy.sample_count(5, g) for g in range(G)]
    for _ in range(3):
        c.step(counts)
        c.compare()
    c.close()


def test_large_segment_table_uses_global_lookup(fls):
    """200 units x 4 shards = 800 segments: above the 512 that travel in the kernel parameters, so the kernels
    bisect the table in global memory."""
    rng = np.random.default_rng(8)
    units = [int(x) for x in rng.integers(1, 3000, 200)]
    c = Case(units, 2, 4, 2, H=1, Q=8, opt_state=True, hp=orc.Hyper(max_grad_norm=0.05))
    assert c.sess.layout["n_segments"] == 800
    for _ in range(2):
        c.step([3, 1])
        c.compare()
    c.close()


@pytest.mark.parametrize("ctas,descending,overlap", [(1, 0, True), (3, 1, False), (0, 1, False), (64, 0, True)])
def test_tuned_launch_shapes_give_identical_results(fls, ctas, descending, overlap):
    """Persistent / descending launch shapes of the AdamW and FedAvg kernels and plain instead of overlapped
    launches change scheduling only: the results are bit-identical to the defaults."""
    def run(tune):
        c = Case([40000, 30011, 5000], 3, 4, 1, H=1, Q=8, opt_state=True, hp=orc.Hyper(max_grad_norm=0.05))
        if tune:
            for kern in (fls.FLS_KERNEL_REDUCE, fls.FLS_KERNEL_ADAMW, fls.FLS_KERNEL_FEDAVG, fls.FLS_KERNEL_ADAMW_FEDAVG):
                fls.fls_plan_tune(c.sess.plan, kern, ctas, descending)
            fls.fls_plan_set_overlap(c.sess.plan, overlap)
        for _ in range(2):
            c.step([1, 2, 3])
        c.compare()
        out = [x.clone() for x in c.sess.master + c.sess.m + c.sess.v + c.sess.param_bf16]
        c.close()
        return out
    assert all(torch.equal(x, y) for x, y in zip(run(False), run(True)))


@pytest.mark.parametrize("units,G,S,R_rep,Q,dtype,fused", [
    ([40000, 30011, 5000], 3, 4, 1, 8, "bf16", False),     # K = 4 flat
    ([40000, 30011, 5000], 4, 8, 1, 8, "bf16", True),      # K = 8 flat, fused aggregation on the one reduce grid
    ([40000, 30011], 2, 4, 2, 8, "bf16", True),            # two-level 4 x 2
    ([70001], 8, 2, 2, 1, "f32", False),                   # fp32 gradients, unaligned shards, G*K = 32
    ([1000003], 2, 4, 1, 1, "bf16", True),                 # the tiny workload's shape
    ([17], 2, 2, 2, 1, "bf16", False),
])
def test_groups_in_one_grid_give_identical_results(fls, units, G, S, R_rep, Q, dtype, fused):
    """Small plans run all groups in one reduce grid and one AdamW grid (the group is the grid's y coordinate).
    Against the oracle, and bit for bit against one launch per group; the launch count shows which way it ran."""
    outs, launches = [], []
    counts = [sy.sample_count(29, g) for g in range(G)]
    for mode in (-1, 0):
        c = Case(units, G, S, R_rep, H=2, Q=Q, grad_dtype=dtype, opt_state=True, hp=orc.Hyper(max_grad_norm=0.05), fused=fused,
                 per_buffer_scale=True, resident=0)
        fls.fls_plan_set_batching(c.sess.plan, mode)
        assert fls.fls_plan_get_batching(c.sess.plan) == (mode == -1)      # these plans are small: automatic means on
        for _ in range(4):
            c.step(counts)
            c.compare()
        outs.append([x.clone() for x in c.sess.master + c.sess.m + c.sess.v + c.sess.param_bf16] + [c.sess.norms().clone(), c.sess.coefs().clone()])
        launches.append(fls.fls_get_launch_count(c.sess.plan))
        assert c.sess.status() == 0
        c.close()
    assert all(torch.equal(x, y) for x, y in zip(*outs))
    n_avg = 3                                                             # opt_state: FedAvg launches per call (parameters, m, v)
    if fused and G <= 16:
        assert launches == [2 * 2 + 2 * 2, 2 * 2 * G + 2 * (G + 1)]       # plain steps: 2 | 2G; aggregation steps: 2 | G + 1
    else:
        assert launches == [4 * 2 + 2 * n_avg, 4 * 2 * G + 2 * n_avg]


@pytest.mark.parametrize("units,G,S,R_rep,Q,dtype", [([40000, 30011], 2, 1, 1, 8, "bf16"), ([70001], 3, 2, 1, 1, "bf16"),
                                                     ([40000, 30011], 4, 1, 2, 8, "bf16"), ([300000], 2, 1, 1, 8, "f32")])
def test_norm_passes_of_all_groups_in_one_grid(fls, units, G, S, R_rep, Q, dtype):
    """Recompute plans (fewer than 8 gradient bytes per element) with several groups: one grid computes all groups' norms,
    then one AdamW kernel per group forms the mean gradient again.  Against the oracle, bit for bit against one norm pass
    and one AdamW kernel per group, and the launch count shows which way it ran."""
    outs, launches = [], []
    for mode in (-1, 0):
        c = Case(units, G, S, R_rep, H=2, Q=Q, grad_dtype=dtype, hp=orc.Hyper(max_grad_norm=0.05), per_buffer_scale=True, resident=0)
        fls.fls_plan_set_batching(c.sess.plan, mode)
        assert fls.fls_plan_get_batching(c.sess.plan) == (mode == -1)
        for _ in range(3):
            c.step(fedavg=False)
            c.compare()
        outs.append([x.clone() for x in c.sess.master + c.sess.m + c.sess.v + c.sess.param_bf16] + [c.sess.norms().clone(), c.sess.coefs().clone()])
        launches.append(fls.fls_get_launch_count(c.sess.plan))
        assert c.sess.status() == 0
        c.close()
    assert all(torch.equal(x, y) for x, y in zip(*outs))
    assert launches == [3 * (G + 1), 3 * 2 * G]


def test_batching_is_automatic_only_for_small_plans(fls):
    from paper_2609_20359_b200.session import Session
    big = Session(6_000_000, None, groups=2, shard_dim=4, fused=True)      # 2 x 24 MB of reduced gradients: above 24 MiB
    assert not fls.fls_plan_get_batching(big.plan)
    fls.fls_plan_set_batching(big.plan, 1)                                  # the fused plan has a slot per group: may be forced
    assert fls.fls_plan_get_batching(big.plan)
    big.close()
    unfused = Session(6_000_000, None, groups=2, shard_dim=4)
    with pytest.raises(fls.FlsError) as e:
        fls.fls_plan_set_batching(unfused.plan, 1)                          # one slot only
    assert e.value.code == fls.FLS_ESTATE
    unfused.close()
    odd = Session(4096, None, groups=2, shard_dim=3)                        # K = 3: no batched kernel
    assert not fls.fls_plan_get_batching(odd.plan)
    odd.close()


@pytest.mark.parametrize("units,G,S,R_rep,Q,dtype", [([40000, 30011], 2, 1, 1, 8, "bf16"), ([40000, 30011], 2, 2, 1, 8, "bf16"),
                                                     ([40000, 30011], 2, 1, 2, 8, "bf16"), ([70001], 2, 3, 1, 1, "bf16"),
                                                     ([70001], 2, 1, 3, 8, "bf16"), ([40000, 30011], 2, 1, 1, 8, "f32")])
def test_recompute_plan_is_bit_identical_to_store_and_reread(fls, units, G, S, R_rep, Q, dtype):
    """K*e_g < 8 bytes: by default the mean gradient is recomputed inside AdamW instead of stored; forcing the
    stored path gives the same bits, both match the oracle, and the stored gradient is only offered when it exists."""
    outs = []
    for mode in (-1, 0):
        c = Case(units, G, S, R_rep, H=2, Q=Q, grad_dtype=dtype, hp=orc.Hyper(max_grad_norm=0.05), per_buffer_scale=True, resident=0)
        fls.fls_plan_set_recompute(c.sess.plan, mode)
        for _ in range(3):
            c.step()
            c.compare()
        if mode == -1:
            with pytest.raises(fls.FlsError) as e:
                c.sess.reduced_grad()
            assert e.value.code == fls.FLS_ESTATE
        else:
            assert c.sess.reduced_grad().numel() == c.L.n_padded
        outs.append([x.clone() for x in c.sess.master + c.sess.m + c.sess.v + c.sess.param_bf16] + [c.sess.norms().clone()])
        c.close()
    assert all(torch.equal(x, y) for x, y in zip(*outs))
    c = Case([4096], 1, 8, 1, H=2, Q=8)
    with pytest.raises(fls.FlsError):
        fls.fls_plan_set_recompute(c.sess.plan, 1)          # 16 gradient bytes per element: does not qualify
    c.close()


@pytest.mark.parametrize("units,G,S,R_rep,Q,dtype", [([40000, 30011], 2, 8, 1, 8, "bf16"), ([40000, 30011], 2, 4, 2, 8, "bf16"),
                                                     ([70001], 2, 3, 2, 1, "bf16"), ([40000, 30011], 2, 2, 1, 8, "f32"),
                                                     ([40000, 30011], 1, 1, 1, 8, "bf16"), ([17], 2, 4, 1, 1, "bf16")])
def test_single_pass_without_clipping(fls, units, G, S, R_rep, Q, dtype):
    """max_grad_norm = 0: one kernel per group does reduce + norm + AdamW.  Against the oracle, and bit for bit against
    the forced two-pass route (norms to rounding: the partial sums are grouped differently)."""
    outs, norms = [], []
    for mode in (-1, 0):
        c = Case(units, G, S, R_rep, H=2, Q=Q, grad_dtype=dtype, hp=orc.Hyper(max_grad_norm=0.0), per_buffer_scale=True, fused=(G > 1))
        fls.fls_plan_set_single_pass(c.sess.plan, mode)
        for _ in range(4):
            c.step([2, 1][:G])
            c.compare()
        assert c.sess.coefs().cpu().tolist() == [1.0] * G
        outs.append([x.clone() for x in c.sess.master + c.sess.m + c.sess.v + c.sess.param_bf16])
        norms.append(c.sess.norms().cpu())
        c.close()
    assert all(torch.equal(x, y) for x, y in zip(*outs))
    assert torch.allclose(norms[0], norms[1], rtol=1e-6, atol=0)
    c = Case([4096], 1, 8, 1, H=2, Q=8)                     # this plan clips
    with pytest.raises(fls.FlsError):
        fls.fls_plan_set_single_pass(c.sess.plan, 1)
    c.close()


def test_reduced_gradient_matches_oracle_exactly_for_bf16(fls):
    """With bf16 inputs of similar magnitude the fp32 running sum is exact, so the mean gradient is
    bit-identical to the oracle's (this case is small enough that no element loses bits)."""
    c = Case([40000, 30011], 1, 4, 2, H=10, Q=8, resident=0)       # two kernels, so that the mean gradient is stored
    grads = c.load_grads(1)
    c.sess.step()
    torch.cuda.synchronize()
    want = orc.pack_sharded(c.L, orc.reduce_mean(grads[0], 4, 2))
    assert np.array_equal(c.sess.reduced_grad().cpu().numpy(), want)
    c.close()


@pytest.mark.parametrize("units,G,S,R_rep,Q", [([40000, 30011], 2, 8, 1, 8), ([40000, 30011], 2, 4, 2, 8), ([70001], 1, 3, 2, 1), ([17], 2, 2, 2, 1)])
def test_bf16_wire_emulation(fls, units, G, S, R_rep, Q):
    """Partial sums and the mean rounded to bf16: the reduced gradient is bit-identical to the oracle's (every
    operation is an fp32 add or divide followed by a bf16 rounding on both sides), the step follows to tolerance."""
    hp = orc.Hyper(max_grad_norm=0.05, wire_bf16=True)
    c = Case(units, G, S, R_rep, H=2, Q=Q, hp=hp, per_buffer_scale=True)
    for t in range(1, 3):
        grads = c.load_grads(t)
        want = orc.pack_sharded(c.L, orc.reduce_mean(grads[G - 1], S, R_rep, wire_bf16=True))
        c.step()
        assert np.array_equal(c.sess.reduced_grad().cpu().numpy(), want)
        c.compare()
    c.close()


def test_bf16_wire_orders_differ_on_the_gpu_too(fls):
    """Same 8 buffers reduced flat (8 x 1) and two-level (4 x 2): with fp32 partial sums the two orders agree
    on all but a handful of elements (where a tiny addend loses bits), with bf16 partial sums they differ widely."""
    res = {}
    for wire in (False, True):
        for S, R_rep in ((8, 1), (4, 2)):
            c = Case([65536], 1, S, R_rep, H=10, Q=8, hp=orc.Hyper(max_grad_norm=0.0, wire_bf16=wire), resident=0)
            fls.fls_plan_set_single_pass(c.sess.plan, 0)      # two passes, so that the mean gradient is stored
            c.load_grads(1)
            c.sess.step()
            torch.cuda.synchronize()
            res[(wire, S)] = c.sess.reduced_grad().clone()
            c.close()
    assert (res[(False, 8)] != res[(False, 4)]).float().mean().item() < 1e-3
    assert 0.02 < (res[(True, 8)] != res[(True, 4)]).float().mean().item() < 0.9


@pytest.mark.parametrize("units,G,S,R_rep,Q,dtype,wire", [
    ([40000, 30011], 2, 8, 1, 8, "bf16", True),         # reduce-scatter ring only
    ([40000, 30011], 2, 4, 2, 8, "bf16", True),         # ring at both levels, sub-chunks of M/2
    ([70001, 33], 1, 3, 2, 1, "bf16", True),            # unaligned shards and sub-chunks: element-wise path
    ([17], 2, 2, 2, 1, "bf16", True),                   # the brute-force size
    ([40000, 30011], 2, 4, 3, 8, "bf16", True),         # K = 12, sub-chunk length not a multiple of 8
    ([40000, 30011], 2, 4, 2, 8, "bf16", False),        # ring order with fp32 partial sums
    ([40000, 30011], 1, 2, 2, 8, "f32", False),         # fp32 gradients
])
def test_ring_order_reduction(fls, units, G, S, R_rep, Q, dtype, wire):
    """reduce_order = FLS_ORDER_RING: every rank's slice is summed starting on the next rank, every all-reduce
    sub-chunk starting on the next replica.  With bf16 partial sums, and with fp32 gradients (double partial sums),
    the reduced gradient is bit-identical to the oracle's; with bf16 gradients and fp32 partial sums it equals the
    exactly rounded mean up to the rounding of the fp32 adds."""
    hp = orc.Hyper(max_grad_norm=0.05, wire_bf16=wire, ring=True)
    c = Case(units, G, S, R_rep, H=2, Q=Q, grad_dtype=dtype, hp=hp, per_buffer_scale=True)
    for t in range(1, 3):
        grads = c.load_grads(t)
        want = orc.pack_sharded(c.L, orc.reduce_mean(grads[G - 1], S, R_rep, wire_bf16=wire, ring=c.ring))
        c.step()
        got = c.sess.reduced_grad().cpu().numpy()
        if wire or dtype == "f32":
            assert np.array_equal(got, want)
        else:
            bound = orc.pack_sharded(c.L, 2.0 ** -24 * np.sum(np.abs(grads[G - 1]), axis=0))
            assert np.all(np.abs(got.astype(np.float64) - want) <= bound)
        c.compare()
    assert c.sess.status() == 0
    c.close()


def test_ring_start_changes_bf16_sums_and_not_fp32_sums(fls):
    """Same 8 buffers, ascending order against ring order, flat (8 x 1) and two-level (4 x 2): with bf16 partial
    sums a measurable share of the elements differs (all but those owned by the last rank / last sub-chunk, whose
    ring order is the ascending one); with fp32 partial sums of bf16 inputs the two orders agree."""
    res = {}
    for wire in (False, True):
        for S, R_rep in ((8, 1), (4, 2)):
            for ring in (False, True):
                c = Case([65536], 1, S, R_rep, H=10, Q=8, hp=orc.Hyper(max_grad_norm=10.0, wire_bf16=wire, ring=ring), resident=0)
                c.load_grads(1)
                c.sess.step()
                torch.cuda.synchronize()
                res[(wire, S, ring)] = c.sess.reduced_grad().clone()
                c.close()
    for S in (8, 4):
        assert (res[(False, S, False)] != res[(False, S, True)]).float().mean().item() < 1e-3
        assert 0.02 < (res[(True, S, False)] != res[(True, S, True)]).float().mean().item() < 0.9
    # the last rank's slice of the flat plan: ring order = ascending order, bit for bit
    M = 65536 // 8
    assert torch.equal(res[(True, 8, False)][7 * M:], res[(True, 8, True)][7 * M:])


def _fp32_running_mean(grads, S, R_rep):
    """What an fp32 accumulator would give (shard level, then replicate level, one division): NOT what the library does."""
    outer = np.zeros(grads[0].shape, np.float32)
    for rho in range(R_rep):
        inner = np.zeros(grads[0].shape, np.float32)
        for sigma in range(S):
            inner = inner + grads[rho * S + sigma].astype(np.float32)
        outer = outer + inner
    return outer / np.float32(S * R_rep)


@pytest.mark.parametrize("S,R_rep", [(8, 1), (4, 2), (3, 2), (1, 5)])
def test_fp32_gradients_are_summed_in_double(fls, S, R_rep):
    """fp32 gradients spanning many binades: the mean gradient is the oracle's bit for bit (double partial sums in
    the same order, one rounding to fp32), where an fp32 running sum would differ in many elements."""
    units, P = [4096, 7], 4103
    def big(t, g, k):
        x = sy.normal_fill_(torch.empty(P), sy.stream_key(9, sy.KIND_GRAD, t, g, k), 1.0)
        return x * (10.0 ** (k % 4 * 2))
    c = Case(units, 1, S, R_rep, H=10, Q=8, grad_dtype="f32", hp=orc.Hyper(max_grad_norm=0.0), resident=0)
    fls.fls_plan_set_single_pass(c.sess.plan, 0)          # two passes, so that the mean gradient is stored
    grads = c.load_grads(1, big)
    c.sess.step()
    torch.cuda.synchronize()
    got = orc.unpack_sharded(c.L, c.sess.reduced_grad().cpu().numpy())
    want = orc.reduce_mean(grads[0], S, R_rep)
    assert np.array_equal(got, want)
    assert np.mean(_fp32_running_mean(grads[0], S, R_rep) != want) > 0.1      # the inputs do tell the two apart
    c.close()


@pytest.mark.parametrize("S,R_rep,fused,spec,clip", [(2, 3, False, False, 0.0), (8, 1, True, False, 1e-7), (4, 1, False, True, 1e-7),
                                                     (5, 1, False, False, 1e-7), (4, 2, False, True, 1.0)])
def test_fp32_gradients_that_cancel(fls, S, R_rep, fused, spec, clip):
    """fp32 gradients whose mean nearly cancels (|mean| around AdamW's eps = 1e-8, addends around 1e-3).  The update
    divides by sqrt(v) + eps, so an error of 1e-10 in such a mean moves theta by 1e-6 and more: the state stays within
    the tolerance only because the partial sums are kept in double.  Three steps, with and without clipping."""
    K, P = S * R_rep, 2048 + 17
    def cancelling(t, g, k):
        if k < K - 1:
            return sy.normal_fill_(torch.empty(P), sy.stream_key(77, sy.KIND_GRAD, t, g, k), 1e-3)
        rest = sum(cancelling(t, g, i).double() for i in range(K - 1))
        tiny = sy.normal_fill_(torch.empty(P), sy.stream_key(78, sy.KIND_GRAD, t, g, k), 1e-8).double()
        return (tiny * K - rest).float()              # the fp32 rounding of this buffer leaves a mean of about 1e-8
    c = Case([17, 2048], 2, S, R_rep, H=3, Q=8, grad_dtype="f32", hp=orc.Hyper(max_grad_norm=clip), fused=fused, speculative=spec)
    grads = c.load_grads(1, cancelling)
    gbar = orc.reduce_mean(grads[0], S, R_rep)
    assert np.median(np.abs(gbar)) < 1e-7 and np.mean(_fp32_running_mean(grads[0], S, R_rep) != gbar) > 0.5
    for _ in range(3):
        c.step(override=cancelling)
        c.compare()
    c.close()


def _sweep_shapes():
    import bench
    seen = set()
    for pt in bench.sweep_points((17,)):
        key = (pt["G"], pt["S"], pt["R"], pt["dtype"])
        if key not in seen:
            seen.add(key)
            yield key


@pytest.mark.parametrize("G,S,R_rep,dtype", list(_sweep_shapes()))
def test_bandwidth_sweep_shapes(fls, G, S, R_rep, dtype):
    """Every (groups, buffers, order, gradient dtype) point of the bandwidth sweep, at P = 2^17 + a step and a FedAvg."""
    c = Case([1 << 17], G, S, R_rep, H=1, Q=8, grad_dtype=dtype, hp=orc.Hyper(max_grad_norm=0.05))
    c.step()
    c.compare()
    c.close()


# ------------------------------------------------------------------ FedAvg
@pytest.mark.parametrize("G,opt_state,counts", [(1, True, [9]), (3, False, [1, 2, 5]), (8, True, None), (9, True, "rand"), (64, False, "rand")])
def test_fedavg(fls, G, opt_state, counts):
    units = [3000, 517] if G < 64 else [999]
    c = Case(units, G, 2, 1, H=1, Q=8, opt_state=opt_state, hp=orc.Hyper(max_grad_norm=0.01))
    if counts == "rand":
        counts = [sy.sample_count(11, g) for g in range(G)]
    before = [m.clone() for m in c.sess.m]
    c.step(counts, fedavg=False)                 # groups diverge (different gradients)
    if G > 1:
        assert not torch.equal(c.sess.master[0], c.sess.master[1])
    m_after_step = [m.clone() for m in c.sess.m]
    orc.fedavg(c.states, counts, opt_state)
    c.sess.fedavg(counts)
    c.compare(check_norms=False)
    for g in range(1, G):                         # every copy equals the average, bit for bit
        assert torch.equal(c.sess.master[g], c.sess.master[0]) and torch.equal(c.sess.param_bf16[g], c.sess.param_bf16[0])
        if opt_state:
            assert torch.equal(c.sess.v[g], c.sess.v[0])
    if not opt_state:                             # params only: m and v untouched
        assert all(torch.equal(a, b) for a, b in zip(m_after_step, c.sess.m))
    del before
    c.close()


@pytest.mark.parametrize("units,G,S,R_rep,Q,dtype,opt_state", [
    ([50000, 1234, 4096], 2, 2, 2, 8, "bf16", False),
    ([50000, 1234, 4096], 4, 4, 1, 8, "bf16", True),
    ([70001], 3, 2, 1, 1, "f32", True),                 # unaligned tail, G = 3
    ([30000, 517], 16, 2, 1, 8, "bf16", False),         # the largest fused G
    ([30000, 517], 17, 2, 1, 8, "bf16", True),          # above it: the call falls back to the two-kernel sequence
    ([17], 2, 4, 1, 1, "bf16", False),
])
def test_fused_step_fedavg_matches_oracle_and_unfused(fls, units, G, S, R_rep, Q, dtype, opt_state):
    """fls_sync_step_fedavg = fls_sync_step + fls_fedavg: against the oracle, and bit for bit against the
    two separate calls on the same inputs (H = 2: steps 1 and 3 are plain, 2 and 4 aggregate)."""
    counts = [sy.sample_count(21, g) for g in range(G)]
    outs = []
    for fused in (True, False):
        c = Case(units, G, S, R_rep, H=2, Q=Q, grad_dtype=dtype, opt_state=opt_state, hp=orc.Hyper(max_grad_norm=0.05), fused=fused)
        for _ in range(4):
            c.step(counts)
            c.compare()
        assert c.sess.t == 4
        outs.append([x.clone() for x in c.sess.master + c.sess.m + c.sess.v + c.sess.param_bf16])
        c.close()
    assert all(torch.equal(x, y) for x, y in zip(*outs))


@pytest.mark.parametrize("units,G,S,R_rep,Q,dtype,opt_state,fused", [
    ([50000, 1234, 4096], 2, 2, 2, 8, "bf16", False, False),
    ([50000, 1234, 4096], 2, 2, 2, 8, "bf16", False, True),
    ([50000, 1234, 4096], 3, 4, 3, 8, "bf16", True, True),
    ([70001], 2, 2, 2, 1, "f32", True, False),           # unaligned tail
    ([70001], 2, 1, 2, 1, "bf16", False, True),          # K = 2: the recompute route is not taken with replica copies
    ([30000, 517], 16, 2, 3, 8, "bf16", False, True),    # 32 extra copies: the most the fused kernel serves
    ([30000, 517], 16, 2, 4, 8, "bf16", True, True),     # 48 extra copies: the fused call falls back to step + FedAvg
    ([17], 2, 2, 2, 1, "bf16", True, True),
    ([999, 40], 32, 1, 2, 8, "bf16", True, False),       # 64 state copies: the most a plan may hold
])
def test_state_copy_per_replica(fls, units, G, S, R_rep, Q, dtype, opt_state, fused):
    """FLS_STATE_PER_REPLICA: G*R_rep state copies.  Every replica of a group applies the group's mean gradient to
    its own copy; FedAvg reads one replica per group and its result is broadcast to all copies.  Against the
    oracle, copy by copy; all copies of a group stay bit-identical; after an aggregation all copies of all groups
    hold the same parameters."""
    counts = [sy.sample_count(23, g) for g in range(G)]
    c = Case(units, G, S, R_rep, H=2, Q=Q, grad_dtype=dtype, opt_state=opt_state, hp=orc.Hyper(max_grad_norm=0.05), fused=fused,
             state_per_replica=True)
    assert len(c.sess.master) == G * R_rep
    for t in range(1, 5):
        c.step(counts)
        c.compare()
        for g in range(G):
            for r in range(1, R_rep):
                a, b = g * R_rep, g * R_rep + r
                assert torch.equal(c.sess.master[a], c.sess.master[b]) and torch.equal(c.sess.m[a], c.sess.m[b])
                assert torch.equal(c.sess.v[a], c.sess.v[b]) and torch.equal(c.sess.param_bf16[a], c.sess.param_bf16[b])
        if t % 2 == 0:
            assert all(torch.equal(c.sess.master[0], x) for x in c.sess.master)
            assert all(torch.equal(c.sess.param_bf16[0], x) for x in c.sess.param_bf16)
            assert all(torch.equal(c.sess.m[0], x) for x in c.sess.m) == (opt_state or G == 1)
    rep = fls.fls_comm_report(c.sess.plan)
    N, K, eg = c.L.n_padded, S * R_rep, 4 if dtype == "f32" else 2
    assert rep["hbm_bytes_sync_step"] == G * N * (K * eg + 4 + 30 * R_rep)
    assert rep["hbm_bytes_fedavg"] == G * N * ((12 + 14 * R_rep) if opt_state else (4 + 6 * R_rep))
    c.close()


def test_state_copy_per_replica_equals_one_copy_per_group(fls):
    """The replica copies change where the numbers live, not the numbers: copy 0 of every group is bit-identical to
    the state of the same plan with one copy per group."""
    outs = []
    for per_replica in (False, True):
        c = Case([40000, 30011], 2, 4, 2, H=2, Q=8, opt_state=True, hp=orc.Hyper(max_grad_norm=0.05), fused=True,
                 state_per_replica=per_replica)
        for _ in range(4):
            c.step([5, 2])
        R = 2 if per_replica else 1
        outs.append([x.clone() for lst in (c.sess.master, c.sess.m, c.sess.v, c.sess.param_bf16) for x in lst[::R]])
        c.close()
    assert all(torch.equal(x, y) for x, y in zip(*outs))


@pytest.mark.parametrize("units,G,S,R_rep,Q,dtype,clip", [
    ([40000, 30011], 2, 8, 1, 8, "bf16", 10.0),          # never clips: every guess holds
    ([40000, 30011], 2, 4, 2, 8, "bf16", 0.02),          # always clips: every step is redone
    ([70001], 2, 3, 2, 1, "bf16", 10.0),                 # unaligned shards
    ([40000, 30011], 2, 2, 1, 8, "f32", 0.02),
    ([17], 1, 4, 1, 1, "bf16", 10.0),
])
def test_speculative_single_pass(fls, units, G, S, R_rep, Q, dtype, clip):
    """Speculative steps (guess: clip coefficient 1) against the oracle and, bit for bit, against the default
    two-pass route; the state moves to the other buffer set with every step; kept / redone counts are reported."""
    outs = []
    for spec in (True, False):
        c = Case(units, G, S, R_rep, H=2, Q=Q, grad_dtype=dtype, hp=orc.Hyper(max_grad_norm=clip), per_buffer_scale=True, speculative=spec)
        seen = set()
        for t in range(1, 5):
            c.step([2, 1][:G])
            c.compare()
            seen.add(c.sess.master[0].data_ptr())
        outs.append([x.clone() for x in c.sess.master + c.sess.m + c.sess.v + c.sess.param_bf16] + [c.sess.norms().clone(), c.sess.coefs().clone()])
        if spec:
            assert len(seen) == 2                              # the two buffer sets take turns
            kept, redone = c.sess.spec_stats()
            assert (kept, redone) == ((4 * G, 0) if clip > 1 else (0, 4 * G))
            rep = fls.fls_comm_report(c.sess.plan)
            assert rep["hbm_bytes_sync_step"] == G * c.L.n_padded * (S * R_rep * (4 if dtype == "f32" else 2) + 26)
        assert c.sess.status() == 0
        c.close()
    assert all(torch.equal(x, y) for x, y in zip(*outs[:1] + outs[1:]))


def test_speculative_mixed_hits_and_misses_and_errors(fls):
    """A threshold between the norms of the two groups: group 0's guess holds, group 1 is redone, in the same call."""
    c = Case([40000, 30011], 2, 4, 1, H=100, Q=8, hp=orc.Hyper(max_grad_norm=1.0), speculative=True)
    big = lambda t, g, k: c.grad_logical(t, g, k) * (1.0 if g == 0 else 16.0)       # norms about 0.13 and 2.1
    for _ in range(3):
        row = c.step(override=big)
        assert row[0][1] == 1.0 and row[1][1] < 1.0
        c.compare()
    assert c.sess.spec_stats() == (3, 3)
    fls.fls_plan_set_speculative(c.sess.plan, False)        # back to two passes, in place, wherever the state is now
    c.step(override=big)
    c.compare()
    assert c.sess.spec_stats() == (3, 3)
    c.close()
    plain = Case([4096], 1, 8, 1, H=2, Q=8)
    with pytest.raises(fls.FlsError) as e:
        fls.fls_plan_set_speculative(plain.sess.plan, True)                          # no second buffer set bound
    assert e.value.code == fls.FLS_ESTATE
    with pytest.raises(fls.FlsError) as e:
        fls.fls_plan_bind_shadow(plain.sess.plan, plain.sess.master, plain.sess.m, plain.sess.v)   # overlaps the bound state
    assert e.value.code == fls.FLS_EPTR
    plain.close()
    noclip = Case([4096], 1, 8, 1, H=2, Q=8, hp=orc.Hyper(max_grad_norm=0.0))
    extra = [torch.zeros(noclip.L.n_padded, device="cuda") for _ in range(3)]
    fls.fls_plan_bind_shadow(noclip.sess.plan, extra[:1], extra[1:2], extra[2:])
    with pytest.raises(fls.FlsError) as e:
        fls.fls_plan_set_speculative(noclip.sess.plan, True)                         # nothing to guess: the plan does not clip
    assert e.value.code == fls.FLS_ESTATE
    noclip.close()


@pytest.mark.parametrize("G,nesterov,opt_state,units,Q,R_rep", [(4, True, False, [30000, 517], 8, 1), (3, False, True, [70001], 1, 1),
                                                                 (9, True, False, [999], 8, 1), (3, True, True, [30000, 517], 8, 2)])
def test_fedavg_outer_optimizer(fls, G, nesterov, opt_state, units, Q, R_rep):
    """Aggregation through an outer SGD step with momentum on a global copy, three rounds, against the oracle (the last
    case with one state copy per replica: the new global parameters reach every copy)."""
    c = Case(units, G, 2, R_rep, H=1, Q=Q, opt_state=opt_state, hp=orc.Hyper(max_grad_norm=0.01), state_per_replica=R_rep > 1)
    counts = [sy.sample_count(31, g) for g in range(G)]
    xg = c.states[0].theta.copy()
    buf = np.zeros_like(xg)
    d_xg = c.sess.master[0].clone()
    d_buf = torch.zeros_like(d_xg)
    for r in range(3):
        c.step(counts, fedavg=False)
        xg, buf = orc.fedavg_outer(c.states, xg, buf, counts, outer_lr=0.7, momentum=0.9, nesterov=nesterov)
        if opt_state:       # m and v are averaged as in plain FedAvg
            w = orc.fedavg_weights(counts, G)
            mbar = orc.fedavg_array([st.m for st in c.states], w); vbar = orc.fedavg_array([st.v for st in c.states], w)
            for st in c.states:
                st.m = mbar.copy(); st.v = vbar.copy()
        for reps in c.copies:   # the broadcast inside every group
            for st in reps[1:]:
                st.theta = reps[0].theta.copy(); st.param_bf16 = reps[0].param_bf16.copy()
                if opt_state:
                    st.m = reps[0].m.copy(); st.v = reps[0].v.copy()
        fls.fls_fedavg_outer(c.sess.plan, counts, 0.7, 0.9, nesterov, d_xg, d_buf)
        c.compare(check_norms=False)
        assert_state_close(d_xg.cpu().numpy(), orc.pack_sharded(c.L, xg), "x_global")
        # the buffer accumulates x_global - xbar, a difference of nearly equal fp32 numbers: its error is a few
        # ulps of the parameters' magnitude (0.02 -> 2e-9), whatever the size of the difference itself
        assert np.allclose(d_buf.cpu().numpy(), orc.pack_sharded(c.L, buf), rtol=1e-5, atol=3e-8)
        assert all(torch.equal(x, d_xg) for x in c.sess.master)
    with pytest.raises(fls.FlsError) as e:
        fls.fls_fedavg_outer(c.sess.plan, counts, float("nan"), 0.9, True, d_xg, d_buf)
    assert e.value.code == fls.FLS_EINVAL
    with pytest.raises(fls.FlsError) as e:
        fls.fls_fedavg_outer(c.sess.plan, counts, 0.7, 0.9, True, d_xg, d_xg)
    assert e.value.code == fls.FLS_EPTR
    c.close()


def test_fedavg_g1_is_bit_exact_identity_and_idempotent(fls):
    c = Case([5000], 1, 2, 1, H=1, Q=8, opt_state=True)
    c.step(fedavg=False)
    snap = (c.sess.master[0].clone(), c.sess.m[0].clone(), c.sess.v[0].clone())
    c.sess.fedavg([123])
    torch.cuda.synchronize()
    assert torch.equal(snap[0], c.sess.master[0]) and torch.equal(snap[1], c.sess.m[0]) and torch.equal(snap[2], c.sess.v[0])
    c.close()
    c = Case([5000], 4, 2, 1, H=1, Q=8)
    c.step([3, 1, 4, 1])
    once = c.sess.master[0].clone()
    c.sess.fedavg([3, 1, 4, 1])                   # identical copies: identity up to the rounding of sum(w)
    torch.cuda.synchronize()
    assert torch.allclose(once, c.sess.master[0], rtol=2e-7, atol=0)
    c.close()


# ------------------------------------------------------------------ whole-loop properties
def test_h1_equal_weights_equals_fsdp_over_all_replicas(fls):
    """Same mean gradient in every group (group g reads group 0's buffers rotated by g): FL+FSDP with
    H = 1, equal weights and averaged optimizer state matches one FSDP group over all R*G buffers."""
    R, G, P = 4, 3, 20000
    fl = Case([P], G, R, 1, H=1, Q=8, opt_state=True, hp=orc.Hyper(max_grad_norm=0.02))
    big = Case([P], 1, R * G, 1, H=10 ** 6, Q=8, hp=orc.Hyper(max_grad_norm=0.02))
    base = lambda t, k: fl.grad_logical(t, 0, k)
    for _ in range(3):
        fl.step(None, override=lambda t, g, k: base(t, (k + g) % R))
        big.step(None, override=lambda t, g, k: base(t, k % R))
    a = orc.unpack_sharded(fl.L, fl.sess.master[0].cpu().numpy())
    b = orc.unpack_sharded(big.L, big.sess.master[0].cpu().numpy())
    assert_state_close(a, b, "fl vs fsdp master")
    assert_state_close(orc.unpack_sharded(fl.L, fl.sess.m[2].cpu().numpy()), orc.unpack_sharded(big.L, big.sess.m[0].cpu().numpy()), "m", 1e-5, "rms")
    fl.close(); big.close()


@pytest.mark.parametrize("speculative", [False, True])
def test_determinism_and_resume(fls, speculative):
    def run(split):
        c = Case([50000, 1234], 2, 4, 1, H=2, Q=8, opt_state=True, hp=orc.Hyper(max_grad_norm=0.02), speculative=speculative)
        for t in range(4 if not speculative else 5):
            if split and t == (2 if not speculative else 3):       # checkpoint: a new plan over the same tensors, step counter restored
                from paper_2609_20359_b200 import _binding as b
                old = c.sess.plan
                c.sess.plan = b.fls_plan_create(c.P, c.units, 2, 4, 1, 2, b.FLS_GRAD_BF16, 8, 3, c.hp.lr, c.hp.beta1, c.hp.beta2,
                                                c.hp.eps, c.hp.weight_decay, c.hp.max_grad_norm)
                b.fls_plan_destroy(old)
                c.sess.bind()          # binds the buffers that hold the state now (after an odd number of speculative steps: the second set)
                b.fls_set_step(c.sess.plan, 2 if not speculative else 3)
            c.step()
        out = [x.clone() for x in c.sess.master + c.sess.m + c.sess.v + c.sess.param_bf16]
        c.close()
        return out
    a, b, r = run(False), run(False), run(True)
    assert all(torch.equal(x, y) for x, y in zip(a, b)), "two identical runs differ"
    assert all(torch.equal(x, y) for x, y in zip(a, r)), "resume from a checkpoint differs"


def test_padding_stays_zero_and_q_does_not_change_logical_results(fls):
    outs = []
    for Q in (1, 8, 64):
        c = Case([1000, 37, 4001], 2, 4, 1, H=2, Q=Q, hp=orc.Hyper(max_grad_norm=0.02))
        for _ in range(2):
            c.step()
        c.compare()
        pad = np.ones(c.L.n_padded, bool); pad[orc._addresses(c.L)[1]] = False
        assert not c.sess.master[0].cpu().numpy()[pad].any() and not c.sess.v[1].cpu().numpy()[pad].any()
        outs.append(orc.unpack_sharded(c.L, c.sess.master[0].cpu().numpy()))
        c.close()
    # the vector and element-wise paths use the same fp32 operations: identical logical results
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[1], outs[2])


def test_lr_override_and_clip_disabled(fls):
    c = Case([30000], 1, 2, 1, H=100, Q=8, hp=orc.Hyper(max_grad_norm=0.0))
    c.step(lr=1e-3)
    c.step(lr=0.0)
    c.compare()
    assert c.sess.coefs().cpu().tolist() == [1.0]
    c.close()


def test_nonfinite_gradients_propagate_and_set_status(fls):
    c = Case([10000], 2, 2, 1, H=100, Q=8)
    def poisoned(t, g, k):
        x = c.grad_logical(t, g, k)
        if g == 1 and k == 0:
            x[77] = float("inf")
        return x
    with np.errstate(invalid="ignore"):
        c.step(override=poisoned)
    assert c.sess.status() & 1
    assert math.isinf(c.sess.norms()[1].item()) and c.sess.coefs()[1].item() == 0.0
    th1 = c.sess.master[1].cpu().numpy()
    assert np.isnan(th1[77]) and np.isfinite(np.delete(th1, 77)).all()      # 0 * inf = NaN only where the inf was
    assert np.isfinite(c.sess.master[0].cpu().numpy()).all()                 # the other group is untouched
    c.close()


def test_non_default_stream(fls):
    """Everything enqueued on a side stream (overlapped launches, fused aggregation, host-gradient step): same
    results as the oracle; the library never touches another stream's work."""
    side = torch.cuda.Stream()
    c = Case([50000, 1234, 4096], 3, 4, 2, H=2, Q=8, opt_state=True, hp=orc.Hyper(max_grad_norm=0.05), fused=True)
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for _ in range(4):
            c.step([3, 5, 1])
            c.compare()
        host = [[c.sess.grads[g][k].cpu().pin_memory() for k in range(c.K)] for g in range(c.G)]
        before = [x.clone() for x in c.sess.master]
        norms = torch.zeros(c.G, dtype=torch.float32)
        c.sess.step_host(host, host_norms=norms)            # step 5 on the same gradients, fed from the host
        side.synchronize()
        assert torch.equal(norms, c.sess.norms().cpu())
        assert all(not torch.equal(a, b) for a, b in zip(before, c.sess.master))
    c.close()


@pytest.mark.parametrize("kw", [{}, {"speculative": True}, {"state_per_replica": True}], ids=["plain", "speculative", "replica_copies"])
def test_step_from_host_buffers_matches_device_step(fls, kw):
    a = Case([50000, 777], 2, 2, 2, H=2, Q=8, hp=orc.Hyper(max_grad_norm=0.02), **kw)
    b = Case([50000, 777], 2, 2, 2, H=2, Q=8, hp=orc.Hyper(max_grad_norm=0.02), **kw)
    for t in range(1, 3):
        a.step()
        host = [[torch.from_numpy(orc.pack_unsharded(b.L, bf16_bits(b.grad_logical(t, g, k)).view(np.int16))).view(torch.bfloat16).pin_memory()
                 for k in range(b.K)] for g in range(b.G)]
        norms = torch.zeros(b.G, dtype=torch.float32)
        due = b.sess.step_host(host, host_norms=norms)
        if due:
            b.sess.fedavg(None)
        torch.cuda.synchronize()
        assert torch.equal(norms, a.sess.norms().cpu())
    for x, y in zip(a.sess.master + a.sess.v + a.sess.param_bf16, b.sess.master + b.sess.v + b.sess.param_bf16):
        assert torch.equal(x, y)
    a.close(); b.close()


# ------------------------------------------------------------------ argument errors that need a device
def test_bind_rejects_bad_buffers(fls):
    from paper_2609_20359_b200.session import Session
    s = Session(4096, None, groups=2, shard_dim=2, align_elems=8)
    flat = [t for row in s.grads for t in row]
    def bind(grads=flat, master=s.master, m=s.m, v=s.v, pb=s.param_bf16, ws=s.workspace, ws_bytes=None):
        fls.fls_plan_bind(s.plan, grads, master, m, v, pb, ws, ws_bytes)
    with pytest.raises(fls.FlsError) as e:
        bind(master=[s.master[0], torch.zeros(4096)])                       # host memory
    assert e.value.code == fls.FLS_EPTR
    with pytest.raises(fls.FlsError) as e:
        bind(m=[s.m[0], s.m[1].view(torch.uint8)[4:].view(torch.float32)])  # misaligned
    assert e.value.code == fls.FLS_EALIGN
    with pytest.raises(fls.FlsError) as e:
        bind(ws_bytes=1024)
    assert e.value.code == fls.FLS_ESIZE
    with pytest.raises(fls.FlsError) as e:
        bind(v=[s.v[0], s.v[0]])                                            # two outputs alias
    assert e.value.code == fls.FLS_EPTR
    with pytest.raises(fls.FlsError) as e:
        bind(grads=[s.master[0].view(torch.bfloat16)[:4096]] + flat[1:])    # a gradient aliases an output
    assert e.value.code == fls.FLS_EPTR
    with pytest.raises(fls.FlsError) as e:
        bind(master=[s.master[0], 0])
    assert e.value.code == fls.FLS_EPTR
    bind(grads=[flat[0]] * len(flat))                                       # inputs may be shared
    bind()
    s.step(); torch.cuda.synchronize()
    s.close()


# ------------------------------------------------------------------ randomized combinations
# ------------------------------------------------------------------ norm tree over several chunks of CTAs
@pytest.mark.parametrize("route", ["two_pass", "recompute", "single_pass", "speculative", "shared_grid"])
def test_norm_tree_with_several_chunks(fls, route):
    """2.7 million parameters per group: 1320 tiles, i.e. more than the 1024 CTAs a single chunk of the norm tree takes, so
    the grid closes six chunks of up to 256 partials and then adds the chunk sums.  All elements against the oracle, norm to
    1e-6, on every route that has its own kernel in front of the tree."""
    P = 2_700_011
    kw = dict(two_pass=dict(S=4), recompute=dict(S=2), single_pass=dict(S=4, clip=0.0), speculative=dict(S=4, spec=True),
              shared_grid=dict(S=4, G=2, fused=True))[route]
    G = kw.get("G", 1)
    c = Case([P], G, kw["S"], 1, H=2, Q=8, hp=orc.Hyper(max_grad_norm=kw.get("clip", 0.05)), fused=kw.get("fused", False),
             speculative=kw.get("spec", False), per_buffer_scale=True, resident=0)
    assert kw["S"] * -(-c.L.unit_shard_numel[0] // 2048) == 1320        # one 256-thread CTA per 2048-element tile
    if route == "shared_grid":
        fls.fls_plan_set_batching(c.sess.plan, 1)
        assert fls.fls_plan_get_batching(c.sess.plan)
    for _ in range(2):
        c.step()
        c.compare()
    assert c.sess.status() == 0
    c.close()


# ------------------------------------------------------------------ resident step (one cooperative kernel per step)
@pytest.mark.parametrize("units,G,S,R_rep,Q,dtype", [
    ([40000, 30011, 5000], 3, 4, 1, 8, "bf16"),         # K = 4 flat, one tile per CTA
    ([1000003], 2, 4, 1, 1, "bf16"),                    # the tiny workload's shape: 978 tiles, two per CTA
    ([1000003], 4, 8, 1, 8, "bf16"),                    # K = 8, four tiles per CTA
    ([300000, 17], 8, 2, 2, 8, "bf16"),                 # two-level 2 x 2, G*K = 32
    ([70001], 2, 1, 1, 1, "bf16"),                      # K = 1, unaligned
    ([70001, 2049], 2, 2, 1, 8, "f32"),                 # fp32 gradients, K = 2
    ([250000], 2, 4, 2, 8, "f32"),                      # fp32 gradients, two-level 4 x 2
    ([17], 1, 2, 2, 1, "bf16"),                         # one group, one ragged tile
])
def test_resident_step(fls, units, G, S, R_rep, Q, dtype):
    """Small plans run the whole step of all groups as one cooperative kernel.  Against the oracle, and against the
    two-kernel route: same state bit for bit, norms equal to the rounding of a double sum grouped differently; the launch
    count shows which way it ran and the stored mean gradient is only offered when it exists."""
    outs, launches = [], []
    counts = [sy.sample_count(31, g) for g in range(G)]
    for mode in (-1, 0):
        c = Case(units, G, S, R_rep, H=2, Q=Q, grad_dtype=dtype, hp=orc.Hyper(max_grad_norm=0.05), fused=(G > 1), per_buffer_scale=True,
                 resident=mode)
        assert fls.fls_plan_get_resident(c.sess.plan) == (mode == -1)        # these plans are small: automatic means on
        for _ in range(4):
            c.step(counts)
            c.compare()
        if mode == -1:
            with pytest.raises(fls.FlsError) as e:
                c.sess.reduced_grad()
            assert e.value.code == fls.FLS_ESTATE
            assert fls.fls_comm_report(c.sess.plan)["hbm_bytes_sync_step"] == G * c.L.n_padded * (S * R_rep * (4 if dtype == "f32" else 2) + 26)
        outs.append([x.clone() for x in c.sess.master + c.sess.m + c.sess.v + c.sess.param_bf16] + [c.sess.coefs().clone()])
        launches.append(fls.fls_get_launch_count(c.sess.plan))
        norms = c.sess.norms().double().cpu() if mode == -1 else norms
        assert torch.allclose(c.sess.norms().double().cpu(), norms, rtol=1e-6, atol=0)
        assert c.sess.status() == 0
        c.close()
    assert all(torch.equal(x, y) for x, y in zip(*outs))
    assert launches[0] == 4 + 2                                               # 4 resident steps, 2 FedAvg kernels


def test_resident_step_is_automatic_only_where_it_fits(fls):
    from paper_2609_20359_b200.session import Session
    big = Session(3_500_000, None, groups=2, shard_dim=4)                   # 2 x 14 MB of mean gradients: above 16 MiB
    assert not fls.fls_plan_get_resident(big.plan)
    fls.fls_plan_set_resident(big.plan, 1)                                  # 3418 tiles still fit the device: may be forced
    assert fls.fls_plan_get_resident(big.plan)
    big.close()
    huge = Session(40_000_000, None, groups=2, shard_dim=4)                 # 39,000 tiles: no grid of resident CTAs holds them
    with pytest.raises(fls.FlsError) as e:
        fls.fls_plan_set_resident(huge.plan, 1)
    assert e.value.code == fls.FLS_ESTATE and not fls.fls_plan_get_resident(huge.plan)
    huge.close()
    for kw in (dict(shard_dim=3), dict(shard_dim=4, ring=True), dict(shard_dim=4, wire_bf16=True), dict(shard_dim=4, max_grad_norm=0.0),
               dict(shard_dim=2, replicate_dim=2, state_per_replica=True), dict(shard_dim=4, speculative=True)):
        s = Session(4096, None, groups=2, **kw)
        assert not fls.fls_plan_get_resident(s.plan), kw
        with pytest.raises(fls.FlsError):
            fls.fls_plan_set_resident(s.plan, 1)
        s.close()


def test_resident_step_bounded_wait_runs_out(fls):
    """The wait inside the resident kernel gives up after wait_limit polls: the status word says so, the state is
    untouched, and the plan works again afterwards."""
    c = Case([40000, 30011], 2, 4, 1, H=10, Q=8, hp=orc.Hyper(max_grad_norm=0.05))
    assert fls.fls_plan_get_resident(c.sess.plan)
    c.step()
    c.compare()
    before = [x.clone() for x in c.sess.master + c.sess.m + c.sess.v + c.sess.param_bf16]
    fls.fls_plan_set_resident(c.sess.plan, -1, 20)
    fls.fls_debug_expire_next_wait(c.sess.plan)
    c.load_grads(2)
    c.sess.step()
    torch.cuda.synchronize()
    assert c.sess.status() & fls.FLS_STATUS_WAIT_EXPIRED
    assert all(torch.equal(x, y) for x, y in zip(before, c.sess.master + c.sess.m + c.sess.v + c.sess.param_bf16))
    # the same step again, normally: rebinding clears the status word, the step counter goes back by one
    c.sess.bind()
    fls.fls_set_step(c.sess.plan, 1)
    fls.fls_plan_set_resident(c.sess.plan, -1, 1 << 22)
    c.step()
    c.compare()
    assert c.sess.status() == 0
    c.close()


def _random_cases(n, seed=20260920):
    rng = np.random.default_rng(seed)
    rng_res = np.random.default_rng(seed + 1)       # its own stream, so that the other fields keep their values
    out = []
    for i in range(n):
        n_units = int(rng.integers(1, 7))
        units = [int(x) for x in rng.choice([1, 7, 8, 17, 255, 2048, 2049, 4096, 10007, 30000], n_units)]
        S = int(rng.choice([1, 2, 3, 4, 8]))
        R_rep = int(rng.choice([1, 1, 2, 3]))
        wire = bool(rng.integers(0, 4) == 0)
        dtype = "bf16" if wire or rng.integers(0, 3) else "f32"
        ring = bool(rng.integers(0, 4) == 0)
        per_replica = bool(R_rep > 1 and rng.integers(0, 3) == 0)
        clip = float(rng.choice([0.0, 0.02, 10.0]))
        spec = bool(clip > 0 and not (wire or ring or per_replica) and rng.integers(0, 2) == 0)
        out.append(dict(units=units, G=int(rng.choice([1, 2, 3, 4, 8])), S=S, R_rep=R_rep, Q=int(rng.choice([1, 4, 8, 16])),
                        dtype=dtype, opt_state=bool(rng.integers(0, 2)), fused=bool(rng.integers(0, 2)), wire=wire, ring=ring,
                        per_replica=per_replica, spec=spec, H=int(rng.choice([1, 2, 3])), clip=clip,
                        ctas=int(rng.choice([0, 0, 1, 5])), desc=int(rng.integers(0, 2)), overlap=bool(rng.integers(0, 2)),
                        keep_mb=float(rng.choice([0.0, 0.05, 64.0])), batch=int(rng.choice([-1, 0, 1])),
                        resident=int(rng_res.choice([-1, -1, 0, 1])), idx=i,
                        data_seed=1000 + i + (0 if seed == 20260920 else seed % 1000003)))
    return out


# FLS_RANDOM_CASES=n widens the draw for an occasional longer run (the first 60 cases are always the same);
# FLS_RANDOM_SEED=s draws another sequence altogether
@pytest.mark.parametrize("p", _random_cases(int(os.environ.get("FLS_RANDOM_CASES", "60")), int(os.environ.get("FLS_RANDOM_SEED", "20260920"))),
                         ids=lambda p: f"case{p['idx']}")
def test_random_combinations(fls, p):
    """Random unit tables, mesh shapes, alignment quanta, dtypes, reduction wire and order, state copies per group or per
    replica, speculative steps, resident steps, FedAvg options and launch shapes, 3 steps each."""
    hp = orc.Hyper(max_grad_norm=p["clip"], wire_bf16=p["wire"], ring=p["ring"])
    c = Case(p["units"], p["G"], p["S"], p["R_rep"], H=p["H"], Q=p["Q"], grad_dtype=p["dtype"], opt_state=p["opt_state"],
             hp=hp, fused=p["fused"], per_buffer_scale=True, seed=p["data_seed"], state_per_replica=p["per_replica"],
             speculative=p["spec"])
    for kern in (fls.FLS_KERNEL_ADAMW, fls.FLS_KERNEL_FEDAVG, fls.FLS_KERNEL_ADAMW_FEDAVG):
        fls.fls_plan_tune(c.sess.plan, kern, p["ctas"], p["desc"])
    fls.fls_plan_set_overlap(c.sess.plan, p["overlap"])
    fls.fls_plan_set_l2_keep(c.sess.plan, int(p["keep_mb"] * 2 ** 20))
    try:
        fls.fls_plan_set_batching(c.sess.plan, p["batch"])
    except fls.FlsError as e:                               # forcing it on a plan that cannot share a grid
        assert p["batch"] == 1 and e.code == fls.FLS_ESTATE
    try:
        fls.fls_plan_set_resident(c.sess.plan, p["resident"])
    except fls.FlsError as e:                               # forcing it on a plan the resident kernel does not serve
        assert p["resident"] == 1 and e.code == fls.FLS_ESTATE
    counts = [sy.sample_count(p["idx"], g) for g in range(p["G"])]
    for _ in range(3):
        c.step(counts)
        c.compare()
    assert c.sess.status() == 0
    c.close()


# ------------------------------------------------------------------ full size, in the benchmark's launch configuration
def _fill_full_size(s, cfg, L):
    """Fills a Session's device buffers from the generator by LOGICAL index (what the oracle samples)."""
    th_key = sy.stream_key(cfg["seed"], sy.KIND_MASTER)
    starts = np.concatenate([[0], np.cumsum(L.unit_numel)])
    for g in range(cfg["groups"]):
        for u, n in enumerate(L.unit_numel):
            M = L.unit_shard_numel[u]
            for sh in range(L.S):
                ln = min(M, n - sh * M)
                if ln > 0:
                    a0 = sh * L.shard_numel + L.unit_shard_offset[u]
                    sy.normal_fill_(s.master[g][a0:a0 + ln], th_key, cfg["master_sigma"], start=int(starts[u]) + sh * M)
            for k in range(s.K):
                scale = sy.uniform_scale(cfg["seed"], g, k) if cfg["per_buffer_scale"] else 1.0
                sy.normal_fill_(s.grads[g][k][L.unit_offset[u]:L.unit_offset[u] + n], sy.stream_key(cfg["seed"], sy.KIND_GRAD, 1, g, k),
                                cfg["grad_sigma"], scale, start=int(starts[u]))
    torch.cuda.synchronize()


def _oracle_norm_full(grads, S, R_rep, chunk=1 << 22, threads=16):
    """Norm of one group's mean gradient over the whole (padded, unsharded) buffers: the oracle's reduce_mean
    and grad_norm on chunks copied to the host, chunks spread over host threads, partial sums added in order."""
    from concurrent.futures import ThreadPoolExecutor
    n = grads[0].numel()
    def one(lo):
        part = [orc.bf16_bits_to_f64(bf16_bits(g[lo:lo + chunk])) for g in grads]
        return orc.grad_norm(orc.reduce_mean(part, S, R_rep)) ** 2
    with ThreadPoolExecutor(threads) as ex:
        parts = list(ex.map(one, range(0, n, chunk)))
    return math.sqrt(math.fsum(parts))


def _sample_grads(cfg, tidx, step, g, K):
    """The K gradient buffers of (step, group) at the sampled logical positions, as exact float64 values."""
    return [orc.bf16_bits_to_f64(bf16_bits(sy.normal_at(tidx, sy.stream_key(cfg["seed"], sy.KIND_GRAD, step, g, k), cfg["grad_sigma"],
                                                        sy.uniform_scale(cfg["seed"], g, k) if cfg["per_buffer_scale"] else 1.0,
                                                        torch.bfloat16))) for k in range(K)]


@pytest.mark.parametrize("cfg_index", [1, 2, 3])
def test_full_size_workloads_sampled(fls, cfg_index):
    """The GPT-2-small, Llama-3.2-1B (18 units, two-level order) and Llama-3.1-8B-block (9 tensors) workloads at
    full size on the route the benchmark times: a plan with the fused aggregation, a plain step through
    fls_sync_step, then -- with fresh gradients, so that non-zero m and v enter AdamW -- an aggregation step through
    fls_sync_step_fedavg (the sync period is set to 2 for this).  The oracle computes every group's norm over the
    full gradient of both steps, then the steps and FedAvg at sampled logical positions: the first and last 4096
    parameters, 16 around every unit and shard boundary, and 200,000 random ones."""
    from paper_2609_20359_b200.session import Session
    cfg = sy.CONFIGS[cfg_index]
    P, G, S, R_rep = cfg["n_params"], cfg["groups"], cfg["shard_dim"], cfg["replicate_dim"]
    K = S * R_rep
    hp = orc.Hyper()
    L = orc.plan(cfg["unit_numel"], S, 8)
    s = Session(P, cfg["unit_numel"], G, S, R_rep, 2, "bf16", 8, False, fused=True)
    assert s.n_padded == L.n_padded
    _fill_full_size(s, cfg, L)
    counts = [sy.sample_count(cfg["seed"], g) for g in range(G)] if cfg["weights"] == "counts" else None
    rng = np.random.default_rng(3)
    starts = np.concatenate([[0], np.cumsum(L.unit_numel)])
    edges = [starts[u] + sh * L.unit_shard_numel[u] for u in range(len(L.unit_numel)) for sh in range(S)]
    idx = np.concatenate([np.arange(0, 4096), np.arange(P - 4096, P), rng.integers(0, P, 200_000),
                          (np.asarray(edges)[:, None] + np.arange(-8, 8)[None, :]).ravel()])
    idx = np.unique(idx[(idx >= 0) & (idx < P)])
    tidx = torch.from_numpy(idx)
    j_np, a_np = orc.addresses_of(L, idx)
    jt, at = torch.from_numpy(j_np).cuda(), torch.from_numpy(a_np).cuda()
    th0 = sy.normal_at(tidx, sy.stream_key(cfg["seed"], sy.KIND_MASTER), cfg["master_sigma"]).numpy()
    assert np.array_equal(s.master[0][at].cpu().numpy(), th0)            # the fill put every sample where the oracle's planner says
    z = np.zeros(idx.size, np.float32)
    states = [orc.GroupState(th0.copy(), z.copy(), z.copy(), orc.f32_to_bf16_bits(th0)) for _ in range(G)]

    def oracle_step(t):
        norms, samp_last, gb_last = [], None, None
        for g in range(G):
            norms.append(_oracle_norm_full(s.grads[g], S, R_rep))
            samp_last = _sample_grads(cfg, tidx, t, g, K)
            gb_last = orc.reduce_mean(samp_last, S, R_rep)
            c = orc.clip_coef(norms[g], hp.max_grad_norm)
            assert c < 1.0
            st = states[g]
            st.theta, st.m, st.v, st.param_bf16 = orc.adamw(st.theta, st.m, st.v, gb_last, c, t, hp.lr, hp.beta1, hp.beta2, hp.eps,
                                                           hp.weight_decay)
        return norms, samp_last, gb_last

    def check_state(tag):
        for g in range(G):
            assert_state_close(s.master[g][at].cpu().numpy(), states[g].theta, f"{tag} master[{g}]")
            assert_state_close(s.m[g][at].cpu().numpy(), states[g].m, f"{tag} m[{g}]", 1e-5, "rms")
            assert_state_close(s.v[g][at].cpu().numpy(), states[g].v, f"{tag} v[{g}]", 1e-5, "rms")
            assert_bf16_close(bf16_bits(s.param_bf16[g][jt]), states[g].param_bf16, f"{tag} bf16[{g}]")

    # step 1: plain step of every group
    norms, samp_last, gb_last = oracle_step(1)
    assert not s.step()
    torch.cuda.synchronize()
    got_n = s.norms().cpu().numpy().astype(np.float64)
    assert np.allclose(got_n, norms, rtol=1e-6, atol=0), (got_n, norms)
    # fp32 running sum against the exactly rounded mean: identical except where a tiny addend loses bits
    got_g = s.reduced_grad()[at].cpu().numpy()
    assert np.mean(got_g == gb_last) > 0.999
    assert np.all(np.abs(got_g.astype(np.float64) - gb_last) <= 2.0 ** -24 * np.sum(np.abs(samp_last), axis=0))
    check_state("step 1")
    # step 2: new gradients, the step and the aggregation in the one fused call
    _fill_grads_full_size(s, cfg, L, 2)
    norms, _, _ = oracle_step(2)
    orc.fedavg(states, counts)
    s.step_fedavg(counts)
    torch.cuda.synchronize()
    assert s.t == 2
    got_n = s.norms().cpu().numpy().astype(np.float64)
    assert np.allclose(got_n, norms, rtol=1e-6, atol=0), (got_n, norms)
    check_state("step 2 + FedAvg")
    assert torch.equal(s.master[0], s.master[G - 1]) and torch.equal(s.param_bf16[0], s.param_bf16[G - 1])
    assert not torch.equal(s.m[0], s.m[G - 1])                            # parameters only: every group keeps its own moments
    assert s.status() == 0
    s.close()


def _fill_grads_full_size(s, cfg, L, step):
    starts = np.concatenate([[0], np.cumsum(L.unit_numel)])
    for g in range(cfg["groups"]):
        for u, n in enumerate(L.unit_numel):
            for k in range(s.K):
                scale = sy.uniform_scale(cfg["seed"], g, k) if cfg["per_buffer_scale"] else 1.0
                sy.normal_fill_(s.grads[g][k][L.unit_offset[u]:L.unit_offset[u] + n], sy.stream_key(cfg["seed"], sy.KIND_GRAD, step, g, k),
                                cfg["grad_sigma"], scale, start=int(starts[u]))
    torch.cuda.synchronize()


@pytest.mark.skipif(not os.environ.get("FLS_LONG_TESTS"), reason="full schedules take minutes; set FLS_LONG_TESTS=1")
@pytest.mark.parametrize("cfg_index", [1, 2, 3])
def test_full_schedule_sampled(fls, cfg_index):
    """The whole schedule of a workload at full size (32 / 8 / 16 steps, fresh gradients every step, FedAvg every
    H steps through the fused call): the oracle follows 100,000 sampled parameters with norms computed over the
    full gradients of every group and step; state compared after every aggregation and at the end."""
    from paper_2609_20359_b200.session import Session
    cfg = sy.CONFIGS[cfg_index]
    P, G, S, R_rep, H = cfg["n_params"], cfg["groups"], cfg["shard_dim"], cfg["replicate_dim"], cfg["sync_period"]
    K = S * R_rep
    hp = orc.Hyper()
    L = orc.plan(cfg["unit_numel"], S, 8)
    s = Session(P, cfg["unit_numel"], G, S, R_rep, H, "bf16", 8, False, fused=True)
    _fill_full_size(s, cfg, L)
    counts = [sy.sample_count(cfg["seed"], g) for g in range(G)] if cfg["weights"] == "counts" else None
    idx = np.unique(np.random.default_rng(5).integers(0, P, 100_000))
    tidx = torch.from_numpy(idx)
    j_np, a_np = orc.addresses_of(L, idx)
    jt, at = torch.from_numpy(j_np).cuda(), torch.from_numpy(a_np).cuda()
    th0 = sy.normal_at(tidx, sy.stream_key(cfg["seed"], sy.KIND_MASTER), cfg["master_sigma"]).numpy()
    z = np.zeros(idx.size, np.float32)
    states = [orc.GroupState(th0.copy(), z.copy(), z.copy(), orc.f32_to_bf16_bits(th0)) for _ in range(G)]
    worst = 0.0
    for t in range(1, cfg["steps"] + 1):
        _fill_grads_full_size(s, cfg, L, t)
        norms = [_oracle_norm_full(s.grads[g], S, R_rep) for g in range(G)]
        for g in range(G):
            samp = [orc.bf16_bits_to_f64(bf16_bits(sy.normal_at(tidx, sy.stream_key(cfg["seed"], sy.KIND_GRAD, t, g, k), cfg["grad_sigma"],
                                                                 sy.uniform_scale(cfg["seed"], g, k) if cfg["per_buffer_scale"] else 1.0,
                                                                 torch.bfloat16))) for k in range(K)]
            gb = orc.reduce_mean(samp, S, R_rep)
            st = states[g]
            st.theta, st.m, st.v, st.param_bf16 = orc.adamw(st.theta, st.m, st.v, gb, orc.clip_coef(norms[g], hp.max_grad_norm), t,
                                                           hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay)
        if t % H == 0:
            orc.fedavg(states, counts)
            s.step_fedavg(counts)
        else:
            assert not s.step()
        torch.cuda.synchronize()
        got_n = s.norms().cpu().numpy().astype(np.float64)
        assert np.allclose(got_n, norms, rtol=1e-6, atol=0), (t, got_n, norms)
        if t % H == 0 or t == cfg["steps"]:
            for g in range(G):
                th = s.master[g][at].cpu().numpy()
                worst = max(worst, float(np.max(np.abs(th.astype(np.float64) - states[g].theta))))
                assert_state_close(th, states[g].theta, f"step {t} master[{g}]")
                assert_state_close(s.m[g][at].cpu().numpy(), states[g].m, f"step {t} m[{g}]", 1e-5, "rms")
                assert_state_close(s.v[g][at].cpu().numpy(), states[g].v, f"step {t} v[{g}]", 1e-5, "rms")
                assert_bf16_close(bf16_bits(s.param_bf16[g][jt]), states[g].param_bf16, f"step {t} bf16[{g}]")
    print(f"full schedule {cfg['name']}: {cfg['steps']} steps, worst |dtheta| on the sample = {worst:.3e}")
    assert s.status() == 0
    s.close()
