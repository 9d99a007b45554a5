"""The allocation-free entry point against the plan-based one (collected last on purpose).

fls_reduce_norm_noalloc serves callers that are not allowed to allocate device memory: its scratch is a
static array inside the library instead of a caller workspace.  It must give what the first kernel of
fls_sync_step gives for the same gradients: the same mean gradient and, within the tolerance the parity
tests use for norms (1e-6 relative), the same norm and clip coefficient -- on consecutive calls that
reuse the static scratch, whatever the previous call left in it."""
import numpy as np
import pytest
import torch

import synthetic as sy

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
    s.step()
    torch.cuda.synchronize()
    out = ([g.clone() for g in s.grads[0]], s.reduced_grad().clone(), float(s.norms()[0]), float(s.coefs()[0]))
    s.close()
    return out


def test_no_alloc_entry_matches_plan_based_reduce_on_consecutive_calls(fls):
    cases = [(300_004, 4, 2, "bf16", 11, 0.01),      # ragged tail (not a multiple of 8), two-level order, clip active
             (1_000_000, 8, 1, "bf16", 12, 1.0),      # flat order, clip inactive
             (70_003 * 3, 3, 1, "f32", 13, 0.001)]    # fp32 gradients, K = 3 (mean by division)
    want = [_existing_path(fls, *c) for c in cases]
    before = torch.cuda.memory_allocated()
    gbar = [torch.empty(c[0], dtype=torch.float32, device="cuda") for c in cases]
    nc = [torch.zeros(2, dtype=torch.float32, device="cuda") for _ in cases]
    # back to back on one stream, then the first case again: every call reuses the same static scratch
    order = [0, 1, 2, 0]
    for i in order:
        n, S, R_rep, dtype, _, clip = cases[i]
        gbar[i].fill_(float("nan")); nc[i].zero_()
        fls.fls_reduce_norm_noalloc(want[i][0], S, R_rep, fls.FLS_GRAD_F32 if dtype == "f32" else fls.FLS_GRAD_BF16, n, clip,
                                    gbar[i], nc[i])
    torch.cuda.synchronize()
    for i in (1, 2, 0):
        _, g_ref, norm_ref, coef_ref = want[i]
        assert torch.equal(gbar[i], g_ref), f"case {i}: mean gradient differs"
        norm, coef = (float(x) for x in nc[i].cpu())
        assert abs(norm - norm_ref) <= 1e-6 * norm_ref and abs(coef - coef_ref) <= 1e-6 * coef_ref, (i, norm, norm_ref, coef, coef_ref)
    assert (cases[0][5] < want[0][2]) and want[0][3] < 1.0 and want[1][3] == 1.0      # both clip branches were seen
    del before


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
