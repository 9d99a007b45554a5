"""The allocation-free entry point against the plan-based one and the oracle (collected last on purpose).

fls_reduce_norm_noalloc serves callers that are not allowed to allocate device memory: its scratch is a
static array inside the library instead of a caller workspace.  It must give what the first kernel of
fls_sync_step gives for the same gradients: the same mean gradient and, within the tolerance the parity
tests use for norms (1e-6 relative), the same norm and clip coefficient -- on consecutive calls that
reuse the static scratch, whatever the previous call left in it -- and while it runs the amount of free
device memory must not move."""
import numpy as np
import pytest
import torch

import synthetic as sy
from oracle import fls_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fls():
    from paper_2609_20359_b200 import build
    build.build()
    import paper_2609_20359_b200._binding as b
    return b


def _existing_path(fls, n, S, R_rep, dtype, seed, clip):
    """Runs fls_sync_step on one group and returns (grads, mean gradient, norm, coef) from the plan's workspace."""
    from paper_2609_20359_b200.session import Session
    s = Session(n, None, groups=1, shard_dim=S, replicate_dim=R_rep, grad_dtype=dtype, align_elems=1, max_grad_norm=clip)
    assert s.n_padded == n
    for k in range(s.K):
        sy.normal_fill_(s.grads[0][k], sy.stream_key(seed, sy.KIND_GRAD, 1, 0, k), 1e-3, sy.uniform_scale(seed, 0, k))
    fls.fls_plan_set_resident(s.plan, 0)               # the two-kernel route, which stores the mean gradient
    if s.K * (4 if dtype == "f32" else 2) < 8:
        fls.fls_plan_set_recompute(s.plan, 0)          # keep the stored mean gradient so that it can be compared
    s.step()
    torch.cuda.synchronize()
    out = ([g.clone() for g in s.grads[0]], s.reduced_grad().clone(), float(s.norms()[0]), float(s.coefs()[0]))
    s.close()
    return out


def _oracle(grads, S, R_rep, dtype, clip):
    """Mean gradient, norm and clip coefficient of the same buffers by the CPU oracle."""
    if dtype == "f32":
        vals = [g.cpu().numpy().astype(np.float64) for g in grads]
    else:
        vals = [orc.bf16_bits_to_f64(g.cpu().view(torch.int16).numpy().view(np.uint16)) for g in grads]
    gbar = orc.reduce_mean(vals, S, R_rep)
    nrm = orc.grad_norm(gbar)
    return gbar, vals, nrm, orc.clip_coef(nrm, clip)


def test_no_alloc_entry_matches_plan_based_reduce_and_oracle_on_consecutive_calls(fls):
    cases = [(300_004, 4, 2, "bf16", 11, 0.01),      # ragged tail (not a multiple of 8), two-level order, clip active
             (1_000_000, 8, 1, "bf16", 12, 1.0),      # flat order, clip inactive
             (70_003 * 3, 3, 1, "f32", 13, 0.001),    # fp32 gradients, K = 3 (mean by division)
             (6, 2, 1, "bf16", 14, 1.0),              # fewer than 8 elements: the element-wise tail only
             (16384 * 3, 2, 2, "bf16", 15, 0.001)]    # a whole number of 16384-element chunks
    want = [_existing_path(fls, *c) for c in cases]
    gbar = [torch.empty(c[0], dtype=torch.float32, device="cuda") for c in cases]
    nc = [torch.zeros(2, dtype=torch.float32, device="cuda") for _ in cases]

    def call(i):
        n, S, R_rep, dtype, _, clip = cases[i]
        gbar[i].fill_(float("nan")); nc[i].zero_()
        fls.fls_reduce_norm_noalloc(want[i][0], S, R_rep, fls.FLS_GRAD_F32 if dtype == "f32" else fls.FLS_GRAD_BF16, n, clip,
                                    gbar[i], nc[i])

    # the first call on a device looks up the static array (and loads the kernel); every output exists by now
    call(0); call(2)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    # back to back on one stream, the first case twice: every call reuses the same static scratch
    for i in (0, 1, 2, 3, 4, 0):
        call(i)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_before, "device memory was allocated during the calls"
    for i, (n, S, R_rep, dtype, _, clip) in enumerate(cases):
        grads, g_ref, norm_ref, coef_ref = want[i]
        assert torch.equal(gbar[i], g_ref), f"case {i}: mean gradient differs from the plan-based path"
        norm, coef = (float(x) for x in nc[i].cpu())
        assert abs(norm - norm_ref) <= 1e-6 * norm_ref and abs(coef - coef_ref) <= 1e-6 * coef_ref, (i, norm, norm_ref, coef, coef_ref)
        # and against the oracle.  bf16 gradients: the fp32 running sum equals the exactly rounded mean except where
        # a small addend loses bits next to a large one (bound 2^-24 * sum |x_k|); fp32 gradients are summed in double,
        # as the oracle does, so the mean is the oracle's bit for bit.  Norm and coefficient to 1e-6 relative.
        g_or, vals, norm_or, coef_or = _oracle(grads, S, R_rep, dtype, clip)
        got = gbar[i].cpu().numpy()
        if dtype == "f32":
            assert np.array_equal(got, g_or), f"case {i}: mean gradient differs from the oracle"
        assert np.all(np.abs(got.astype(np.float64) - g_or) <= 2.0 ** -24 * np.sum(np.abs(vals), axis=0)), f"case {i}: mean gradient differs from the oracle"
        assert abs(norm - norm_or) <= 1e-6 * norm_or and abs(coef - coef_or) <= 1e-6 * coef_or, (i, norm, norm_or, coef, coef_or)
    assert want[0][3] < 1.0 and want[1][3] == 1.0      # both clip branches were seen


def test_no_alloc_entry_rejects_what_it_cannot_serve(fls):
    x = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(64, dtype=torch.float32, device="cuda")
    nc = torch.zeros(2, dtype=torch.float32, device="cuda")
    with pytest.raises(fls.FlsError) as e:
        fls.fls_reduce_norm_noalloc([x], 1, 1, fls.FLS_GRAD_BF16, fls.FLS_NOALLOC_MAX_ELEMS + 1, 1.0, out, nc)
    assert e.value.code == fls.FLS_ESIZE and "exceeds" in str(e.value)
    with pytest.raises(fls.FlsError) as e:
        fls.fls_reduce_norm_noalloc([x] * 65, 65, 1, fls.FLS_GRAD_BF16, 64, 1.0, out, nc)
    assert e.value.code == fls.FLS_EINVAL
    with pytest.raises(fls.FlsError) as e:
        fls.fls_reduce_norm_noalloc([x.view(torch.uint8)[2:66].view(torch.bfloat16)], 1, 1, fls.FLS_GRAD_BF16, 32, 1.0, out, nc)
    assert e.value.code == fls.FLS_EALIGN
    fls.fls_reduce_norm_noalloc([x], 1, 1, fls.FLS_GRAD_BF16, 64, 1.0, out, nc)      # still usable afterwards
    torch.cuda.synchronize()
    assert float(nc[0]) == 0.0 and float(nc[1]) == 1.0
