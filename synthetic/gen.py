"""Counter-based generator: value = f(seed, stream, index), integer-only up to the
last two IEEE multiplies, so a CPU tensor and a CUDA tensor filled by the same
call hold identical bits.

A stream is (kind, step, group, buffer).  Element `index` of a stream is built
from two 64-bit hashes of (key + index): their eight 16-bit lanes are summed
(an Irwin-Hall(8) variate: mean 0, unit variance after scaling, kurtosis 2.85,
support +-4.9 sigma), converted exactly to fp32, multiplied by 1/std and then by
sigma*scale.  bf16 tensors get the fp32 value rounded to nearest even.

These buffers stand in for real gradients and initial weights: the kernels are
pure HBM streams whose speed does not depend on the values, and the parity tests
need only that both sides read the same numbers.
"""
from __future__ import annotations

import numpy as np
import torch

_M64 = (1 << 64) - 1
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB
_GOLD = 0x9E3779B97F4A7C15
_SALT2 = 0xD1B54A32D192ED03

KIND_GRAD, KIND_MASTER, KIND_SCALE, KIND_COUNT, KIND_MISC = 1, 2, 3, 4, 5

# sum of eight independent uniform integers on [0, 65535]: mean 8*32767.5, variance 8*(2^32-1)/12
_LANES = 8
_MEAN = _LANES * 65535 // 2            # 262140 (exact: 8*32767.5)
_STD = float(np.sqrt(_LANES * ((1 << 32) - 1) / 12.0))
_INV_STD = np.float32(1.0 / _STD)


def _signed(c: int) -> int:
    c &= _M64
    return c - (1 << 64) if c >= (1 << 63) else c


def mix64_int(x: int) -> int:
    """splitmix64 finaliser on a Python int (host scalars: keys, scales, counts)."""
    x &= _M64
    x ^= x >> 30
    x = (x * _C1) & _M64
    x ^= x >> 27
    x = (x * _C2) & _M64
    x ^= x >> 31
    return x


def stream_key(seed: int, kind: int, step: int = 0, group: int = 0, buffer: int = 0) -> int:
    packed = ((kind & 0xFF) << 56) | ((step & 0xFFFFFF) << 32) | ((group & 0xFFFF) << 16) | (buffer & 0xFFFF)
    return mix64_int((seed & _M64) ^ mix64_int(packed ^ _GOLD))


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    # logical shift right on int64 storage
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64_t(x: torch.Tensor) -> torch.Tensor:
    # same finaliser on int64 tensors; int64 multiply wraps modulo 2^64 on CPU and CUDA
    x = x ^ _lsr(x, 30)
    x = x * _signed(_C1)
    x = x ^ _lsr(x, 27)
    x = x * _signed(_C2)
    x = x ^ _lsr(x, 31)
    return x


def _lane_sum(h: torch.Tensor) -> torch.Tensor:
    return (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)


def _normal_f32(idx: torch.Tensor, key: int, sigma_scale: float) -> torch.Tensor:
    """fp32 deviates for int64 indices `idx` of the stream `key`."""
    k1 = _signed(key)
    k2 = _signed(mix64_int(key ^ _SALT2))
    s = _lane_sum(_mix64_t(idx + k1)) + _lane_sum(_mix64_t(idx + k2)) - _MEAN
    z = s.to(torch.float32) * torch.tensor(_INV_STD, dtype=torch.float32, device=idx.device)
    return z * torch.tensor(np.float32(sigma_scale), dtype=torch.float32, device=idx.device)


def normal_fill_(out: torch.Tensor, key: int, sigma: float, scale: float = 1.0,
                 start: int = 0, chunk: int = 1 << 24) -> torch.Tensor:
    """Fill the 1-D fp32 or bf16 tensor `out` with elements start .. start+len-1 of stream `key`."""
    assert out.dim() == 1 and out.dtype in (torch.float32, torch.bfloat16)
    n = out.numel()
    sig = float(np.float32(sigma) * np.float32(scale))
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        idx = torch.arange(start + lo, start + hi, dtype=torch.int64, device=out.device)
        out[lo:hi] = _normal_f32(idx, key, sig).to(out.dtype)
    return out


def normal_at(indices: torch.Tensor, key: int, sigma: float, scale: float = 1.0,
              dtype: torch.dtype = torch.float32) -> torch.Tensor:
    """Values of stream `key` at arbitrary int64 `indices` (used to sample huge buffers)."""
    sig = float(np.float32(sigma) * np.float32(scale))
    return _normal_f32(indices.to(torch.int64), key, sig).to(dtype)


def uniform_scale(seed: int, group: int, buffer: int) -> float:
    """Per-(group, buffer) gradient scale in [0.5, 2), a multiple of 1.5*2^-24 above 0.5."""
    h = stream_key(seed, KIND_SCALE, 0, group, buffer)
    return float(np.float32(0.5) + np.float32(1.5) * np.float32((h >> 40) * 2.0 ** -24))


def sample_count(seed: int, group: int) -> int:
    """Per-group sample count in 1..1000 (FedAvg weight numerator)."""
    return 1 + stream_key(seed, KIND_COUNT, 0, group, 0) % 1000


# ---------------------------------------------------------------------------
# The five synthetic workloads (shapes, sizes and distributions; no arithmetic).
# shard_dim = S, replicate_dim = R_rep; a group owns K = S*R_rep gradient buffers.
# ---------------------------------------------------------------------------
_SEED0 = 0x26092035_9000000C

_LLAMA32_1B_UNITS = [128256 * 2048] + [2 * 2048 * 2048 + 2 * 512 * 2048 + 3 * 8192 * 2048 + 2 * 2048] * 16 + [2048]
_LLAMA31_8B_BLOCK_UNITS = [4096 * 4096, 1024 * 4096, 1024 * 4096, 4096 * 4096,
                           14336 * 4096, 14336 * 4096, 14336 * 4096, 4096, 4096]

_HYPER = dict(lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1, max_grad_norm=1.0)

CONFIGS = [
    dict(name="tiny_fl_fsdp", n_params=1_000_003, unit_numel=[1_000_003], groups=2, shard_dim=4,
         replicate_dim=1, sync_period=4, steps=8, grad_dtype="bf16", grad_sigma=1e-3, master_sigma=0.02,
         per_buffer_scale=False, weights="equal", seed=_SEED0 + 1, **_HYPER),
    dict(name="gpt2_small_fl_fsdp", n_params=124_439_808, unit_numel=[124_439_808], groups=4, shard_dim=8,
         replicate_dim=1, sync_period=8, steps=32, grad_dtype="bf16", grad_sigma=1e-3, master_sigma=0.02,
         per_buffer_scale=True, weights="counts", seed=_SEED0 + 2, **_HYPER),
    dict(name="llama32_1b_fl_hsdp", n_params=1_235_814_400, unit_numel=_LLAMA32_1B_UNITS, groups=2, shard_dim=4,
         replicate_dim=2, sync_period=4, steps=8, grad_dtype="bf16", grad_sigma=1e-3, master_sigma=0.02,
         per_buffer_scale=False, weights="equal", seed=_SEED0 + 3, **_HYPER),
    dict(name="llama31_8b_block_fl_fsdp", n_params=218_112_000, unit_numel=_LLAMA31_8B_BLOCK_UNITS, groups=8,
         shard_dim=8, replicate_dim=1, sync_period=16, steps=16, grad_dtype="bf16", grad_sigma=1e-3,
         master_sigma=0.02, per_buffer_scale=False, weights="counts", seed=_SEED0 + 4, **_HYPER),
]
assert sum(_LLAMA32_1B_UNITS) == 1_235_814_400 and sum(_LLAMA31_8B_BLOCK_UNITS) == 218_112_000


def config_by_name(name: str) -> dict:
    for c in CONFIGS:
        if c["name"] == name:
            return dict(c)
    raise KeyError(name)
