"""ctypes binding of libfls.so: same names as the C ABI, argument marshalling only."""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Optional, Sequence

_PKG = os.path.dirname(os.path.abspath(__file__))
# FLS_LIBRARY points the binding at another build of the same ABI (e.g. one compiled with other tuning flags)
LIB_PATH = os.environ.get("FLS_LIBRARY") or os.path.join(_PKG, "libfls.so")

FLS_OK, FLS_EINVAL, FLS_EALIGN, FLS_EPTR, FLS_ESIZE, FLS_ECUDA, FLS_ESTATE = range(7)
FLS_GRAD_BF16, FLS_GRAD_F32 = 0, 1
FLS_WIRE_F32, FLS_WIRE_BF16 = 0, 1
FLS_ORDER_ASCENDING, FLS_ORDER_RING = 0, 1
FLS_STATE_PER_GROUP, FLS_STATE_PER_REPLICA = 0, 1
FLS_AVG_PARAMS, FLS_AVG_OPT_STATE, FLS_AVG_FUSED = 1, 2, 4
FLS_KERNEL_REDUCE, FLS_KERNEL_ADAMW, FLS_KERNEL_FEDAVG, FLS_KERNEL_ADAMW_FEDAVG, FLS_KERNEL_COUNT = 0, 1, 2, 3, 4
FLS_STATUS_NONFINITE_NORM = 1
FLS_STATUS_WAIT_EXPIRED = 2
FLS_MAX_GROUPS = 64
FLS_MAX_GRAD_BUFFERS = 64
FLS_MAX_FUSED_GROUPS = 16
FLS_MAX_STATE_COPIES = 64
FLS_BUFFER_ALIGN = 32
FLS_NOALLOC_MAX_ELEMS = 1 << 29

EXPORTS = [
    "fls_plan_create", "fls_plan_query", "fls_plan_bind", "fls_sync_step", "fls_sync_step_host", "fls_fedavg",
    "fls_sync_step_fedavg", "fls_fedavg_outer",
    "fls_get_norms", "fls_get_reduced_grad", "fls_get_status", "fls_get_step", "fls_set_step", "fls_comm_report",
    "fls_plan_bind_shadow", "fls_plan_set_speculative", "fls_get_spec_stats", "fls_get_state", "fls_plan_set_l2_keep", "fls_plan_set_batching", "fls_plan_get_batching",
    "fls_plan_set_resident", "fls_plan_get_resident", "fls_debug_expire_next_wait",
    "fls_plan_tune", "fls_plan_set_recompute", "fls_plan_set_single_pass", "fls_plan_set_overlap", "fls_set_profiling", "fls_get_kernel_ms", "fls_get_launch_count", "fls_plan_destroy",
    "fls_last_error", "fls_reduce_norm_noalloc",
]


class FlsError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"libfls error {code}: {message}")
        self.code = code


class fls_plan_desc(C.Structure):
    _fields_ = [("n_params", C.c_uint64), ("n_units", C.c_uint32), ("unit_numel", C.POINTER(C.c_uint64)),
                ("groups", C.c_uint32), ("shard_dim", C.c_uint32), ("replicate_dim", C.c_uint32),
                ("sync_period", C.c_uint32), ("grad_dtype", C.c_uint32), ("align_elems", C.c_uint32),
                ("fedavg_what", C.c_uint32), ("reduce_wire", C.c_uint32),
                ("reduce_order", C.c_uint32), ("state_copies", C.c_uint32),
                ("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
                ("weight_decay", C.c_double), ("max_grad_norm", C.c_double)]


class fls_layout(C.Structure):
    _fields_ = [("n_padded", C.c_uint64), ("shard_numel", C.c_uint64), ("n_units", C.c_uint32),
                ("grad_buffers", C.c_uint32), ("unit_offset", C.POINTER(C.c_uint64)),
                ("unit_shard_numel", C.POINTER(C.c_uint64)), ("unit_shard_offset", C.POINTER(C.c_uint64)),
                ("workspace_bytes", C.c_uint64), ("n_segments", C.c_uint32), ("vector_path", C.c_uint32),
                ("n_state_copies", C.c_uint32), ("reserved", C.c_uint32)]


class fls_buffers(C.Structure):
    _fields_ = [("grads", C.POINTER(C.c_void_p)), ("master", C.POINTER(C.c_void_p)), ("m", C.POINTER(C.c_void_p)),
                ("v", C.POINTER(C.c_void_p)), ("param_bf16", C.POINTER(C.c_void_p)), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_uint64)]


class fls_cost5(C.Structure):
    _fields_ = [(n, C.c_double) for n in ("fsdp", "hsdp", "fl", "fl_fsdp", "fl_hsdp")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class fls_comm_costs(C.Structure):
    _fields_ = [("paper_bytes", fls_cost5), ("wire_bytes", fls_cost5), ("seconds", fls_cost5),
                ("hbm_bytes_sync_step", C.c_double), ("hbm_bytes_fedavg", C.c_double)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2609_20359_b200.build` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    P = C.c_void_p
    lib.fls_plan_create.argtypes = [C.POINTER(fls_plan_desc), C.POINTER(P)]
    lib.fls_plan_query.argtypes = [P, C.POINTER(fls_layout)]
    lib.fls_plan_bind.argtypes = [P, C.POINTER(fls_buffers)]
    lib.fls_sync_step.argtypes = [P, C.c_double, P, C.POINTER(C.c_int)]
    lib.fls_sync_step_host.argtypes = [P, C.POINTER(C.c_void_p), C.c_double, P, C.POINTER(C.c_float), C.POINTER(C.c_int)]
    lib.fls_fedavg.argtypes = [P, C.POINTER(C.c_uint64), P]
    lib.fls_sync_step_fedavg.argtypes = [P, C.c_double, C.POINTER(C.c_uint64), P]
    lib.fls_fedavg_outer.argtypes = [P, C.POINTER(C.c_uint64), C.c_double, C.c_double, C.c_int, P, P, P]
    lib.fls_get_norms.argtypes = [P, C.POINTER(P), C.POINTER(P)]
    lib.fls_get_reduced_grad.argtypes = [P, C.POINTER(P)]
    lib.fls_get_status.argtypes = [P, C.POINTER(P)]
    lib.fls_get_step.argtypes = [P, C.POINTER(C.c_uint64)]
    lib.fls_set_step.argtypes = [P, C.c_uint64]
    lib.fls_comm_report.argtypes = [P, C.POINTER(C.c_double), C.POINTER(fls_comm_costs)]
    lib.fls_plan_tune.argtypes = [P, C.c_uint32, C.c_int, C.c_int]
    lib.fls_plan_bind_shadow.argtypes = [P, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.POINTER(C.c_void_p)]
    lib.fls_plan_set_speculative.argtypes = [P, C.c_int]
    lib.fls_get_spec_stats.argtypes = [P, C.POINTER(P)]
    lib.fls_get_state.argtypes = [P, C.c_uint32, C.POINTER(P), C.POINTER(P), C.POINTER(P)]
    lib.fls_plan_set_l2_keep.argtypes = [P, C.c_uint64]
    lib.fls_plan_set_batching.argtypes = [P, C.c_int]
    lib.fls_plan_get_batching.argtypes = [P, C.POINTER(C.c_int)]
    lib.fls_plan_set_resident.argtypes = [P, C.c_int, C.c_uint32]
    lib.fls_plan_get_resident.argtypes = [P, C.POINTER(C.c_int)]
    lib.fls_debug_expire_next_wait.argtypes = [P]
    lib.fls_plan_set_recompute.argtypes = [P, C.c_int]
    lib.fls_plan_set_single_pass.argtypes = [P, C.c_int]
    lib.fls_plan_set_overlap.argtypes = [P, C.c_int]
    lib.fls_set_profiling.argtypes = [P, C.c_int]
    lib.fls_get_kernel_ms.argtypes = [P, C.POINTER(C.c_double), C.POINTER(C.c_uint64)]
    lib.fls_get_launch_count.argtypes = [P, C.POINTER(C.c_uint64)]
    lib.fls_plan_destroy.argtypes = [P]
    lib.fls_reduce_norm_noalloc.argtypes = [C.POINTER(C.c_void_p), C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint64, C.c_double, P, P, P]
    lib.fls_last_error.argtypes = []
    lib.fls_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name != "fls_last_error":
            getattr(lib, name).restype = C.c_int
    return lib


lib = _load()


def _check(rc: int) -> None:
    if rc != FLS_OK:
        raise FlsError(rc, lib.fls_last_error().decode())


def _ptr(t) -> int:
    """Device (or pinned host) address of a torch tensor, or a raw integer address."""
    return int(t) if isinstance(t, int) else int(t.data_ptr())


def _ptr_array(items: Sequence) -> C.Array:
    return (C.c_void_p * len(items))(*[_ptr(t) for t in items])


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    return int(stream) if isinstance(stream, int) else int(stream.cuda_stream)


def fls_plan_create(n_params: int, unit_numel: Optional[Sequence[int]] = None, groups: int = 1, shard_dim: int = 1,
                    replicate_dim: int = 1, sync_period: int = 1, grad_dtype: int = FLS_GRAD_BF16, align_elems: int = 8,
                    fedavg_what: int = FLS_AVG_PARAMS, lr: float = 3e-4, beta1: float = 0.9, beta2: float = 0.95,
                    eps: float = 1e-8, weight_decay: float = 0.1, max_grad_norm: float = 1.0,
                    reduce_wire: int = FLS_WIRE_F32, reduce_order: int = FLS_ORDER_ASCENDING,
                    state_copies: int = FLS_STATE_PER_GROUP) -> int:
    """Returns the opaque plan handle."""
    d = fls_plan_desc()
    d.n_params = n_params
    if unit_numel is not None:
        arr = (C.c_uint64 * len(unit_numel))(*unit_numel)
        d.n_units, d.unit_numel = len(unit_numel), arr
    d.groups, d.shard_dim, d.replicate_dim, d.sync_period = groups, shard_dim, replicate_dim, sync_period
    d.grad_dtype, d.align_elems, d.fedavg_what, d.reduce_wire = grad_dtype, align_elems, fedavg_what, reduce_wire
    d.reduce_order, d.state_copies = reduce_order, state_copies
    d.lr, d.beta1, d.beta2, d.eps, d.weight_decay, d.max_grad_norm = lr, beta1, beta2, eps, weight_decay, max_grad_norm
    out = C.c_void_p()
    _check(lib.fls_plan_create(C.byref(d), C.byref(out)))
    return out.value


def fls_plan_query(plan: int) -> dict:
    lay = fls_layout()
    _check(lib.fls_plan_query(plan, C.byref(lay)))
    n = lay.n_units
    return dict(n_padded=lay.n_padded, shard_numel=lay.shard_numel, n_units=n, grad_buffers=lay.grad_buffers,
                unit_offset=[lay.unit_offset[i] for i in range(n)],
                unit_shard_numel=[lay.unit_shard_numel[i] for i in range(n)],
                unit_shard_offset=[lay.unit_shard_offset[i] for i in range(n)],
                workspace_bytes=lay.workspace_bytes, n_segments=lay.n_segments, vector_path=bool(lay.vector_path),
                n_state_copies=lay.n_state_copies)


def fls_plan_bind(plan: int, grads: Sequence, master: Sequence, m: Sequence, v: Sequence, param_bf16: Sequence,
                  workspace, workspace_bytes: Optional[int] = None) -> None:
    """grads: G*K tensors (index g*K + rho*S + sigma); master/m/v/param_bf16: n_state_copies tensors (G, or G*R_rep
    with one state copy per replica, index g*R_rep + rho); workspace: a byte tensor."""
    b = fls_buffers()
    keep = [_ptr_array(grads), _ptr_array(master), _ptr_array(m), _ptr_array(v), _ptr_array(param_bf16)]
    b.grads, b.master, b.m, b.v, b.param_bf16 = keep
    b.workspace = _ptr(workspace)
    b.workspace_bytes = workspace_bytes if workspace_bytes is not None else workspace.numel() * workspace.element_size()
    _check(lib.fls_plan_bind(plan, C.byref(b)))


def fls_sync_step(plan: int, lr: float = math.nan, stream=None) -> bool:
    """One local step of all groups; returns True when FedAvg is due."""
    due = C.c_int(0)
    _check(lib.fls_sync_step(plan, lr, _stream_handle(stream), C.byref(due)))
    return bool(due.value)


def fls_sync_step_host(plan: int, host_grads: Sequence, lr: float = math.nan, stream=None, host_norms=None) -> bool:
    """Same with gradients in (pinned) host tensors; host_norms: optional float32 CPU tensor of G entries."""
    due = C.c_int(0)
    arr = _ptr_array(host_grads)
    norms = C.cast(_ptr(host_norms), C.POINTER(C.c_float)) if host_norms is not None else None
    _check(lib.fls_sync_step_host(plan, arr, lr, _stream_handle(stream), norms, C.byref(due)))
    return bool(due.value)


def fls_fedavg(plan: int, sample_counts: Optional[Sequence[int]] = None, stream=None) -> None:
    arr = (C.c_uint64 * len(sample_counts))(*sample_counts) if sample_counts is not None else None
    _check(lib.fls_fedavg(plan, arr, _stream_handle(stream)))


def fls_fedavg_outer(plan: int, sample_counts: Optional[Sequence[int]], outer_lr: float, momentum: float, nesterov: bool,
                     global_params, outer_momentum, stream=None) -> None:
    """FedAvg followed by an SGD(+momentum/Nesterov) step on the global copy; global_params and outer_momentum
    are float32 device tensors of N_pad elements in shard order, updated in place."""
    arr = (C.c_uint64 * len(sample_counts))(*sample_counts) if sample_counts is not None else None
    _check(lib.fls_fedavg_outer(plan, arr, outer_lr, momentum, int(nesterov), _ptr(global_params), _ptr(outer_momentum),
                                _stream_handle(stream)))


def fls_sync_step_fedavg(plan: int, lr: float = math.nan, sample_counts: Optional[Sequence[int]] = None, stream=None) -> None:
    """fls_sync_step followed by fls_fedavg, fused into the optimizer kernel when the plan has FLS_AVG_FUSED."""
    arr = (C.c_uint64 * len(sample_counts))(*sample_counts) if sample_counts is not None else None
    _check(lib.fls_sync_step_fedavg(plan, lr, arr, _stream_handle(stream)))


def fls_get_norms(plan: int):
    """(device address of G norms, device address of G clip coefficients)."""
    a, b = C.c_void_p(), C.c_void_p()
    _check(lib.fls_get_norms(plan, C.byref(a), C.byref(b)))
    return a.value, b.value


def fls_get_reduced_grad(plan: int) -> int:
    a = C.c_void_p()
    _check(lib.fls_get_reduced_grad(plan, C.byref(a)))
    return a.value


def fls_get_status(plan: int) -> int:
    a = C.c_void_p()
    _check(lib.fls_get_status(plan, C.byref(a)))
    return a.value


def fls_get_step(plan: int) -> int:
    t = C.c_uint64()
    _check(lib.fls_get_step(plan, C.byref(t)))
    return t.value


def fls_set_step(plan: int, t: int) -> None:
    _check(lib.fls_set_step(plan, t))


def fls_comm_report(plan: int, bw_bytes_per_s: Optional[Sequence[float]] = None) -> dict:
    out = fls_comm_costs()
    bw = (C.c_double * 3)(*bw_bytes_per_s) if bw_bytes_per_s is not None else None
    _check(lib.fls_comm_report(plan, bw, C.byref(out)))
    return dict(paper_bytes=out.paper_bytes.as_dict(), wire_bytes=out.wire_bytes.as_dict(), seconds=out.seconds.as_dict(),
                hbm_bytes_sync_step=out.hbm_bytes_sync_step, hbm_bytes_fedavg=out.hbm_bytes_fedavg)


def fls_plan_tune(plan: int, kernel: int, ctas_per_sm: int = 0, descending: int = -1) -> None:
    _check(lib.fls_plan_tune(plan, kernel, ctas_per_sm, descending))


def fls_plan_bind_shadow(plan: int, master: Sequence, m: Sequence, v: Sequence) -> None:
    """Second set of state buffers (G tensors each) that speculative steps write to."""
    _check(lib.fls_plan_bind_shadow(plan, _ptr_array(master), _ptr_array(m), _ptr_array(v)))


def fls_plan_set_speculative(plan: int, enabled: bool) -> None:
    _check(lib.fls_plan_set_speculative(plan, int(enabled)))


def fls_get_spec_stats(plan: int) -> int:
    """Device address of two uint32 counters: group-steps kept, group-steps redone."""
    a = C.c_void_p()
    _check(lib.fls_get_spec_stats(plan, C.byref(a)))
    return a.value


def fls_get_state(plan: int, copy: int):
    """(master, m, v) device addresses of state copy `copy` as they are now."""
    a, b, c = C.c_void_p(), C.c_void_p(), C.c_void_p()
    _check(lib.fls_get_state(plan, copy, C.byref(a), C.byref(b), C.byref(c)))
    return a.value, b.value, c.value


def fls_plan_set_batching(plan: int, mode: int) -> None:
    """-1 automatic (small plans), 0 never, 1 whenever the plan allows it: all groups in one grid per kernel."""
    _check(lib.fls_plan_set_batching(plan, mode))


def fls_plan_get_batching(plan: int) -> bool:
    a = C.c_int(0)
    _check(lib.fls_plan_get_batching(plan, C.byref(a)))
    return bool(a.value)


def fls_plan_set_resident(plan: int, mode: int, wait_limit: int = 0) -> None:
    """-1 automatic (small plans that fit the device), 0 never, 1 whenever the plan fits: the whole step of all groups as one
    cooperative kernel.  wait_limit: polls before a waiting CTA gives up (0 keeps the current value)."""
    _check(lib.fls_plan_set_resident(plan, mode, wait_limit))


def fls_plan_get_resident(plan: int) -> bool:
    a = C.c_int(0)
    _check(lib.fls_plan_get_resident(plan, C.byref(a)))
    return bool(a.value)


def fls_debug_expire_next_wait(plan: int) -> None:
    """Test hook: the next resident step waits for a value nobody publishes (every CTA gives up after wait_limit polls)."""
    _check(lib.fls_debug_expire_next_wait(plan))


def fls_plan_set_l2_keep(plan: int, nbytes: int) -> None:
    _check(lib.fls_plan_set_l2_keep(plan, nbytes))


def fls_plan_set_recompute(plan: int, mode: int) -> None:
    _check(lib.fls_plan_set_recompute(plan, mode))


def fls_plan_set_single_pass(plan: int, mode: int) -> None:
    _check(lib.fls_plan_set_single_pass(plan, mode))


def fls_plan_set_overlap(plan: int, enabled: bool) -> None:
    _check(lib.fls_plan_set_overlap(plan, int(enabled)))


def fls_set_profiling(plan: int, enabled: bool) -> None:
    _check(lib.fls_set_profiling(plan, int(enabled)))


def fls_get_kernel_ms(plan: int):
    ms = (C.c_double * FLS_KERNEL_COUNT)()
    n = (C.c_uint64 * FLS_KERNEL_COUNT)()
    _check(lib.fls_get_kernel_ms(plan, ms, n))
    return list(ms), list(n)


def fls_get_launch_count(plan: int) -> int:
    n = C.c_uint64()
    _check(lib.fls_get_launch_count(plan, C.byref(n)))
    return n.value


def fls_plan_destroy(plan: int) -> None:
    _check(lib.fls_plan_destroy(plan))


def fls_reduce_norm_noalloc(grads: Sequence, shard_dim: int, replicate_dim: int, grad_dtype: int, n_elems: int,
                            max_grad_norm: float, gbar_out, norm_coef_out, stream=None) -> None:
    """Mean gradient + norm + clip coefficient of one group without a plan or workspace, for callers that
    may not allocate device memory (the scratch is a static array inside the library).  grads: K tensors;
    gbar_out: float32 tensor of n_elems; norm_coef_out: float32 tensor of 2.  n_elems <= FLS_NOALLOC_MAX_ELEMS.
    Calls share the static scratch: do not let two of them overlap on one GPU."""
    _check(lib.fls_reduce_norm_noalloc(_ptr_array(grads), shard_dim, replicate_dim, grad_dtype, n_elems, max_grad_norm,
                                       _ptr(gbar_out), _ptr(norm_coef_out), _stream_handle(stream)))


def fls_last_error() -> str:
    return lib.fls_last_error().decode()


__all__ = [n for n in dir() if n.startswith(("fls_", "FLS_"))] + ["FlsError", "lib", "LIB_PATH", "EXPORTS"]
