"""CPU-side checks of libfls: the shared library loads and exports the whole C ABI, and its host-only
parts (layout planner, argument validation, cost reporter) agree with the oracle.  No kernel runs."""
import ctypes
import math
import os
import re

import numpy as np
import pytest

from oracle import fls_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def fls():
    from paper_2609_20359_b200 import build
    build.build()
    import paper_2609_20359_b200._binding as b
    return b


def test_library_exports_every_declared_symbol(fls):
    header = open(os.path.join(ROOT, "include", "fls.h")).read()
    declared = set(re.findall(r"\b(fls_[a-z_0-9]+)\s*\(", header))
    declared -= {"fls_plan"}
    assert declared == set(fls.EXPORTS), declared ^ set(fls.EXPORTS)
    lib = ctypes.CDLL(fls.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_header_is_plain_c(tmp_path):
    """include/fls.h is the boundary: it must compile as C99 on its own, and a C program must link against the library."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    src = tmp_path / "use_fls.c"
    src.write_text('#include "fls.h"\n#include <stdio.h>\n'
                   'int main(void) {\n'
                   '  fls_plan_desc d = {0}; fls_plan* p = 0; fls_layout lay; fls_comm_costs c;\n'
                   '  d.n_params = 1000; d.groups = 2; d.shard_dim = 4; d.replicate_dim = 1; d.sync_period = 2; d.align_elems = 8;\n'
                   '  d.fedavg_what = FLS_AVG_PARAMS; d.lr = 3e-4; d.beta1 = 0.9; d.beta2 = 0.95; d.eps = 1e-8; d.weight_decay = 0.1; d.max_grad_norm = 1.0;\n'
                   '  if (fls_plan_create(&d, &p) != FLS_OK) { printf("%s\\n", fls_last_error()); return 1; }\n'
                   '  if (fls_plan_query(p, &lay) != FLS_OK || fls_comm_report(p, 0, &c) != FLS_OK) return 2;\n'
                   '  printf("%llu %llu %.0f\\n", (unsigned long long)lay.n_padded, (unsigned long long)lay.shard_numel, c.hbm_bytes_sync_step);\n'
                   '  return fls_plan_destroy(p);\n}\n')
    inc = os.path.join(ROOT, "include")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", inc, "-fsyntax-only", str(src)], check=True)
    from paper_2609_20359_b200 import build
    lib = build.build()
    exe = tmp_path / "use_fls"
    subprocess.run(["gcc", "-std=c99", "-I", inc, str(src), "-o", str(exe), lib, "-Wl,-rpath," + os.path.dirname(lib)], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.split() == ["1024", "256", str(2 * 1024 * (4 * 2 + 34))]     # G * N_pad * (K*e_g + 34), K = 4 bf16


def test_struct_sizes_match_header_layout(fls):
    # natural alignment of the C structs in include/fls.h
    assert ctypes.sizeof(fls.fls_plan_desc) == 8 + 8 + 8 + 10 * 4 + 6 * 8
    assert ctypes.sizeof(fls.fls_layout) == 8 + 8 + 4 + 4 + 3 * 8 + 8 + 4 + 4 + 4 + 4
    assert ctypes.sizeof(fls.fls_buffers) == 7 * 8
    assert ctypes.sizeof(fls.fls_comm_costs) == 15 * 8 + 16


@pytest.mark.parametrize("units,S,Q", [([17], 4, 1), ([17], 4, 8), ([5, 1, 12], 3, 1), ([5, 1, 12], 3, 4), ([1000003], 4, 1),
                                       ([1000003], 4, 8), ([7, 9, 64, 3], 8, 8), ([33], 1, 1),
                                       ([128256 * 2048] + [60821504] * 16 + [2048], 4, 8)])
def test_planner_matches_oracle(fls, units, S, Q):
    p = fls.fls_plan_create(sum(units), units, groups=2, shard_dim=S, align_elems=Q)
    lay = fls.fls_plan_query(p)
    L = orc.plan(units, S, Q)
    assert lay["n_padded"] == L.n_padded and lay["shard_numel"] == L.shard_numel
    assert lay["unit_offset"] == L.unit_offset and lay["unit_shard_numel"] == L.unit_shard_numel
    assert lay["unit_shard_offset"] == L.unit_shard_offset
    assert lay["workspace_bytes"] >= 4 * L.n_padded
    assert lay["n_segments"] == (1 if len(units) == 1 or S == 1 else len(units) * S)
    fls.fls_plan_destroy(p)


def test_planner_matches_oracle_on_random_unit_tables(fls):
    rng = np.random.default_rng(99)
    for _ in range(300):
        units = [int(x) for x in rng.integers(1, 10 ** int(rng.integers(1, 8)), int(rng.integers(1, 40)))]
        S, Q = int(rng.integers(1, 17)), int(rng.choice([1, 2, 3, 8, 16, 64]))
        p = fls.fls_plan_create(sum(units), units, groups=int(rng.integers(1, 5)), shard_dim=S, align_elems=Q)
        lay = fls.fls_plan_query(p)
        L = orc.plan(units, S, Q)
        assert (lay["n_padded"], lay["shard_numel"]) == (L.n_padded, L.shard_numel)
        assert lay["unit_offset"] == L.unit_offset and lay["unit_shard_numel"] == L.unit_shard_numel
        assert lay["unit_shard_offset"] == L.unit_shard_offset
        assert lay["vector_path"] == all(m % 8 == 0 for m in L.unit_shard_numel) or len(units) == 1 or S == 1
        fls.fls_plan_destroy(p)


def test_ring_order_plans_keep_one_segment_per_rank_and_unit(fls):
    """Ring-order kernels need the owning rank and the position inside the rank's slice, so the planner does not
    merge neighbouring runs for them; everything else about the layout is unchanged."""
    for units, S in (([4096], 4), ([40000, 30011], 4), ([7, 9, 64, 3], 8)):
        a = fls.fls_plan_create(sum(units), units, groups=2, shard_dim=S, replicate_dim=2, align_elems=8)
        b = fls.fls_plan_create(sum(units), units, groups=2, shard_dim=S, replicate_dim=2, align_elems=8, reduce_order=fls.FLS_ORDER_RING)
        la, lb = fls.fls_plan_query(a), fls.fls_plan_query(b)
        assert lb["n_segments"] == len(units) * S >= la["n_segments"]
        for k in ("n_padded", "shard_numel", "unit_offset", "unit_shard_numel", "unit_shard_offset", "n_state_copies"):
            assert la[k] == lb[k]
        fls.fls_plan_destroy(a); fls.fls_plan_destroy(b)
    c = fls.fls_plan_create(4096, None, groups=3, shard_dim=2, replicate_dim=4, state_copies=fls.FLS_STATE_PER_REPLICA)
    assert fls.fls_plan_query(c)["n_state_copies"] == 12
    for call in (lambda: fls.fls_plan_set_recompute(c, 1), lambda: fls.fls_plan_set_single_pass(c, 1), lambda: fls.fls_plan_set_speculative(c, 1)):
        with pytest.raises(fls.FlsError) as e:
            call()
        assert e.value.code == fls.FLS_ESTATE
    fls.fls_plan_destroy(c)


def test_single_unit_default_table(fls):
    p = fls.fls_plan_create(1000, None, groups=1, shard_dim=4, align_elems=8)
    lay = fls.fls_plan_query(p)
    assert lay["n_units"] == 1 and lay["n_padded"] == 1024 and lay["vector_path"]
    fls.fls_plan_destroy(p)


@pytest.mark.parametrize("kw", [dict(groups=0), dict(shard_dim=0), dict(replicate_dim=0), dict(sync_period=0), dict(align_elems=0),
                                dict(groups=65), dict(shard_dim=16, replicate_dim=8), dict(beta1=1.0), dict(beta2=-0.1),
                                dict(eps=0.0), dict(lr=-1.0), dict(lr=float("nan")), dict(grad_dtype=7), dict(fedavg_what=2),
                                dict(fedavg_what=0), dict(unit_numel=[10, 5]), dict(unit_numel=[16, 0]),
                                dict(max_grad_norm=float("nan")), dict(weight_decay=-0.5),
                                dict(reduce_wire=2), dict(reduce_wire=1, grad_dtype=1), dict(fedavg_what=8),
                                dict(reduce_order=2), dict(state_copies=2), dict(groups=33, replicate_dim=2, state_copies=1)])
def test_plan_create_rejects_bad_arguments(fls, kw):
    args = dict(n_params=16, unit_numel=None, groups=2, shard_dim=2)
    args.update(kw)
    with pytest.raises(fls.FlsError) as e:
        fls.fls_plan_create(**args)
    assert e.value.code == fls.FLS_EINVAL and fls.fls_last_error()


def test_calls_before_bind_fail_cleanly(fls):
    p = fls.fls_plan_create(16, None, groups=2, shard_dim=2)
    for call in (lambda: fls.fls_sync_step(p, stream=0), lambda: fls.fls_fedavg(p, None, stream=0),
                 lambda: fls.fls_get_norms(p), lambda: fls.fls_get_status(p)):
        with pytest.raises(fls.FlsError) as e:
            call()
        assert e.value.code == fls.FLS_ESTATE
    assert fls.fls_get_step(p) == 0
    fls.fls_set_step(p, 41)
    assert fls.fls_get_step(p) == 41 and fls.fls_get_launch_count(p) == 0
    assert fls.lib.fls_plan_destroy(None) == 0
    fls.fls_plan_destroy(p)


def test_comm_report_matches_oracle_and_paper_table(fls):
    rng = np.random.default_rng(5)
    for _ in range(20):
        units = [int(x) for x in rng.integers(1, 5000, int(rng.integers(1, 6)))]
        S, R, F, A = int(rng.integers(1, 9)), int(rng.integers(1, 8)), int(rng.integers(1, 9)), int(rng.integers(1, 17))
        f32 = bool(rng.integers(0, 2))
        bw = [float(x) for x in rng.uniform(1e9, 1e12, 3)]
        p = fls.fls_plan_create(sum(units), units, groups=F, shard_dim=S, replicate_dim=R, sync_period=A,
                                grad_dtype=fls.FLS_GRAD_F32 if f32 else fls.FLS_GRAD_BF16, align_elems=1)
        rep = fls.fls_comm_report(p, bw)
        rep0 = fls.fls_comm_report(p, None)
        L = orc.plan(units, S, 1)
        e = 4 if f32 else 2
        Mb = [m * e for m in L.unit_shard_numel]
        want_bytes = orc.comm_costs(Mb, S, R, F, A)
        want_sec = orc.comm_costs(Mb, S, R, F, A, *bw)
        for k in want_bytes:
            assert math.isclose(rep["paper_bytes"][k], want_bytes[k], rel_tol=1e-12, abs_tol=1e-9), k
            assert math.isclose(rep["seconds"][k], want_sec[k], rel_tol=1e-12, abs_tol=1e-30), k
            assert math.isnan(rep0["seconds"][k])
        # bytes a rank sends when all-gather / reduce-scatter carry the whole unit: (S-1) shards each
        assert math.isclose(rep["wire_bytes"]["fsdp"], sum(3 * (S - 1) * m for m in Mb), rel_tol=1e-12, abs_tol=1e-9)
        K = S * R
        assert rep["hbm_bytes_sync_step"] == F * L.n_padded * ((2 * K * e + 26) if K * e < 8 else (K * e + 34))
        p0 = fls.fls_plan_create(sum(units), units, groups=F, shard_dim=S, replicate_dim=R, sync_period=A, max_grad_norm=0.0,
                                 grad_dtype=fls.FLS_GRAD_F32 if f32 else fls.FLS_GRAD_BF16, align_elems=1)
        assert fls.fls_comm_report(p0)["hbm_bytes_sync_step"] == F * L.n_padded * (K * e + 26)      # no clipping: one pass
        fls.fls_plan_destroy(p0)
        assert rep["hbm_bytes_fedavg"] == F * L.n_padded * 10
        fls.fls_plan_destroy(p)


def test_comm_report_hsdp_fallback_and_bad_bandwidth(fls):
    p = fls.fls_plan_create(4096, None, groups=4, shard_dim=8, replicate_dim=1, sync_period=8)
    rep = fls.fls_comm_report(p)
    assert rep["paper_bytes"]["fl_hsdp"] == rep["paper_bytes"]["fl_fsdp"]
    M = 4096 / 8 * 2
    assert math.isclose(rep["paper_bytes"]["fl_fsdp"], M * (3 * 7 / 8 + (1 / 8) * 2 * 3 / 4), rel_tol=1e-12)
    with pytest.raises(fls.FlsError):
        fls.fls_comm_report(p, [1e9, 0.0, 1e9])
    fls.fls_plan_destroy(p)


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_20359_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cpp", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f
