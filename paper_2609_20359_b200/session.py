"""Session: owns the torch tensors of one plan and binds them (device memory and streams only).

All arithmetic happens in libfls through the fls_* calls; this class allocates the flat buffers the
plan asks for, optionally fenced by guard bands, and exposes views of what the library writes.
"""
from __future__ import annotations

import math
from typing import Optional, Sequence

import torch

from . import _binding as fls

GUARD_BYTE = 0xA5


class Session:
    def __init__(self, n_params: int, unit_numel: Optional[Sequence[int]] = None, groups: int = 1, shard_dim: int = 1,
                 replicate_dim: int = 1, sync_period: int = 1, grad_dtype: str = "bf16", align_elems: int = 8,
                 opt_state: bool = False, lr: float = 3e-4, beta1: float = 0.9, beta2: float = 0.95, eps: float = 1e-8,
                 weight_decay: float = 0.1, max_grad_norm: float = 1.0, device: str = "cuda:0", guard_bytes: int = 0,
                 alloc_grads: bool = True, fused: bool = False, wire_bf16: bool = False, ring: bool = False,
                 state_per_replica: bool = False, speculative: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("libfls needs a CUDA device; there is no CPU path")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.G, self.S, self.R_rep, self.H = groups, shard_dim, replicate_dim, sync_period
        self.K = shard_dim * replicate_dim
        self.grad_torch_dtype = torch.float32 if grad_dtype == "f32" else torch.bfloat16
        self.guard = (guard_bytes + 255) // 256 * 256
        self._blocks = []
        self.plan = fls.fls_plan_create(
            n_params, unit_numel, groups, shard_dim, replicate_dim, sync_period,
            fls.FLS_GRAD_F32 if grad_dtype == "f32" else fls.FLS_GRAD_BF16, align_elems,
            fls.FLS_AVG_PARAMS | (fls.FLS_AVG_OPT_STATE if opt_state else 0) | (fls.FLS_AVG_FUSED if fused else 0),
            lr, beta1, beta2, eps, weight_decay, max_grad_norm, fls.FLS_WIRE_BF16 if wire_bf16 else fls.FLS_WIRE_F32,
            fls.FLS_ORDER_RING if ring else fls.FLS_ORDER_ASCENDING,
            fls.FLS_STATE_PER_REPLICA if state_per_replica else fls.FLS_STATE_PER_GROUP)
        self.layout = fls.fls_plan_query(self.plan)
        N = self.layout["n_padded"]
        self.n_padded, self.n_params = N, n_params
        # state copies: one per group, or one per replica (index g*R_rep + rho)
        self.n_copies = self.layout["n_state_copies"]
        self.grads = [[self._alloc(N, self.grad_torch_dtype) for _ in range(self.K)] for _ in range(groups)] if alloc_grads else None
        self._state = {"master": [self._alloc(N, torch.float32) for _ in range(self.n_copies)],
                       "m": [self._alloc(N, torch.float32) for _ in range(self.n_copies)],
                       "v": [self._alloc(N, torch.float32) for _ in range(self.n_copies)]}
        self.param_bf16 = [self._alloc(N, torch.bfloat16) for _ in range(self.n_copies)]
        self.workspace = self._alloc(self.layout["workspace_bytes"], torch.uint8, zero=False)
        self.speculative = speculative
        self._cur = self._state            # where the state is now (speculative plans move it with every step)
        self._shadow = None
        if speculative:
            # the second buffer set that speculative steps write to; which set is current changes with every step
            self._shadow = {k: [self._alloc(N, torch.float32) for _ in range(groups)] for k in ("master", "m", "v")}
        if alloc_grads:
            self.bind()

    # ------------------------------------------------------------------ memory
    def _alloc(self, numel: int, dtype: torch.dtype, zero: bool = True) -> torch.Tensor:
        nbytes = numel * torch.empty(0, dtype=dtype).element_size()
        body = (nbytes + 255) // 256 * 256
        raw = torch.empty(self.guard + body + self.guard, dtype=torch.uint8, device=self.device)
        if self.guard:
            raw[: self.guard] = GUARD_BYTE
            raw[self.guard + nbytes:] = GUARD_BYTE
        view = raw[self.guard: self.guard + nbytes].view(dtype)
        if zero:
            view.zero_()
        self._blocks.append((raw, nbytes))
        return view

    def guards_intact(self) -> bool:
        """True if no byte outside any buffer's body was modified (only meaningful with guard_bytes > 0)."""
        ok = True
        for raw, nbytes in self._blocks:
            if self.guard:
                ok &= bool((raw[: self.guard] == GUARD_BYTE).all()) and bool((raw[self.guard + nbytes:] == GUARD_BYTE).all())
        return ok

    def bind(self, grads=None) -> None:
        if grads is not None:
            self.grads = grads
        flat = [t for row in self.grads for t in row]
        st = self._cur                     # the buffers that hold the state now are the ones to bind
        fls.fls_plan_bind(self.plan, flat, st["master"], st["m"], st["v"], self.param_bf16, self.workspace)
        if self._shadow is not None:
            both = {k: self._state[k] + self._shadow[k] for k in ("master", "m", "v")}
            held = {k: {t.data_ptr() for t in st[k]} for k in both}
            other = {k: [t for t in both[k] if t.data_ptr() not in held[k]] for k in both}
            fls.fls_plan_bind_shadow(self.plan, other["master"], other["m"], other["v"])
            fls.fls_plan_set_speculative(self.plan, True)

    def _refresh(self) -> None:
        """After a step of a speculative plan: ask the library which buffer set holds the state now."""
        if self._shadow is None:
            return
        ptrs = [fls.fls_get_state(self.plan, c) for c in range(self.n_copies)]
        cur = {}
        for i, k in enumerate(("master", "m", "v")):
            by_ptr = {t.data_ptr(): t for t in self._state[k] + self._shadow[k]}
            cur[k] = [by_ptr[p[i]] for p in ptrs]
        self._cur = cur

    @property
    def master(self):
        return self._cur["master"]

    @property
    def m(self):
        return self._cur["m"]

    @property
    def v(self):
        return self._cur["v"]

    def spec_stats(self):
        """(group-steps whose guess held, group-steps redone) of a speculative plan so far."""
        t = self._ws_view(fls.fls_get_spec_stats(self.plan), 2, torch.int32).cpu()
        return int(t[0]), int(t[1])

    # ------------------------------------------------------------------ calls
    def step(self, lr: float = math.nan, stream=None) -> bool:
        due = fls.fls_sync_step(self.plan, lr, stream)
        self._refresh()
        return due

    def step_host(self, host_grads, lr: float = math.nan, stream=None, host_norms=None) -> bool:
        flat = [t for row in host_grads for t in row]
        due = fls.fls_sync_step_host(self.plan, flat, lr, stream, host_norms)
        self._refresh()
        return due

    def step_fedavg(self, sample_counts=None, lr: float = math.nan, stream=None) -> None:
        fls.fls_sync_step_fedavg(self.plan, lr, sample_counts, stream)
        self._refresh()

    def fedavg(self, sample_counts=None, stream=None) -> None:
        fls.fls_fedavg(self.plan, sample_counts, stream)

    # ------------------------------------------------------------------ views of library-written data
    def _ws_view(self, addr: int, numel: int, dtype: torch.dtype) -> torch.Tensor:
        off = addr - self.workspace.data_ptr()
        nbytes = numel * torch.empty(0, dtype=dtype).element_size()
        assert 0 <= off and off + nbytes <= self.workspace.numel()
        return self.workspace[off: off + nbytes].view(dtype)

    def norms(self) -> torch.Tensor:
        return self._ws_view(fls.fls_get_norms(self.plan)[0], self.G, torch.float32)

    def coefs(self) -> torch.Tensor:
        return self._ws_view(fls.fls_get_norms(self.plan)[1], self.G, torch.float32)

    def reduced_grad(self) -> torch.Tensor:
        return self._ws_view(fls.fls_get_reduced_grad(self.plan), self.n_padded, torch.float32)

    def status(self) -> int:
        return int(self._ws_view(fls.fls_get_status(self.plan), 1, torch.int32).item())

    @property
    def t(self) -> int:
        return fls.fls_get_step(self.plan)

    def close(self) -> None:
        if self.plan is not None:
            fls.fls_plan_destroy(self.plan)
            self.plan = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
