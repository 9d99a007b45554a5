"""Writes worked_cases.json: a few tiny sync steps and one FedAvg worked out in exact
rational arithmetic (fractions + 80-digit decimal square roots), rounding to fp32 /
bf16 only where the method stores a value.  Uses neither the oracle nor the CUDA
library.  The paper prints no worked example of this arithmetic; these follow the
definitions: mean over the K buffers, L2 norm, c = min(1, clip/(norm+1e-6)), AdamW
with decoupled weight decay and bias correction, w_g = n_g / sum(n).

    python -m tests.golden.make_worked_cases        # rewrites the json next to this file
"""
import json
import os
from decimal import Decimal, getcontext
from fractions import Fraction

getcontext().prec = 80
LR, B1, B2, EPS, WD, CLIP, CLIP_EPS = (Fraction(x) for x in (3e-4, 0.9, 0.95, 1e-8, 0.1, 1.0, 1e-6))


def _round_to_bits(q: Fraction, frac_bits: int, emin: int) -> Fraction:
    """Nearest-even rounding of q to a binary format with `frac_bits` fraction bits."""
    if q == 0:
        return Fraction(0)
    s, a = (-1 if q < 0 else 1), abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    e = max(e, emin)
    quantum = Fraction(2) ** (e - frac_bits)
    return s * round(a / quantum) * quantum          # round(): half to even


def f32(q):
    return _round_to_bits(Fraction(q), 23, -126)


def bf16_bits(q32: Fraction) -> int:
    r = _round_to_bits(q32, 7, -126)
    if r == 0:
        return 0
    s, a = (1 if r < 0 else 0), abs(r)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    frac = int((a / Fraction(2) ** e - 1) * 128)
    return (s << 15) | ((e + 127) << 7) | frac


def bf16_value(bits: int) -> Fraction:
    s = -1 if bits >> 15 else 1
    e, f = (bits >> 7) & 0xFF, bits & 0x7F
    return s * (1 + Fraction(f, 128)) * Fraction(2) ** (e - 127) if e else s * Fraction(f, 128) * Fraction(2) ** -126


def sqrt(q: Fraction) -> Fraction:
    return Fraction((Decimal(q.numerator) / Decimal(q.denominator)).sqrt())


def hexf(q: Fraction) -> str:
    return float(q).hex()


def sync_case(name, grad_bits, theta0, S, R_rep, n_steps):
    K, n = len(grad_bits), len(theta0)
    theta = [f32(Fraction(x)) for x in theta0]
    m, v = [Fraction(0)] * n, [Fraction(0)] * n
    out = dict(name=name, S=S, R_rep=R_rep, grad_bits=grad_bits, theta0=[hexf(x) for x in theta], steps=[])
    gbar = [f32(sum(bf16_value(grad_bits[k][j]) for k in range(K)) / K) for j in range(n)]
    norm = sqrt(sum(g * g for g in gbar))
    coef = min(Fraction(1), CLIP / (norm + CLIP_EPS))
    for t in range(1, n_steps + 1):
        for j in range(n):
            g = coef * gbar[j]
            th = theta[j] * (1 - LR * WD)
            mj = B1 * m[j] + (1 - B1) * g
            vj = B2 * v[j] + (1 - B2) * g * g
            th = th - LR * (mj / (1 - B1 ** t)) / (sqrt(vj / (1 - B2 ** t)) + EPS)
            theta[j], m[j], v[j] = f32(th), f32(mj), f32(vj)
        out["steps"].append(dict(t=t, norm=float(norm), coef=float(coef), theta=[hexf(x) for x in theta],
                                 m=[hexf(x) for x in m], v=[hexf(x) for x in v], bf16=[bf16_bits(x) for x in theta]))
    return out


def fedavg_case(copies, counts):
    tot = sum(counts)
    n = len(copies[0])
    avg = [f32(sum(Fraction(counts[g], tot) * f32(Fraction(copies[g][j])) for g in range(len(copies)))) for j in range(n)]
    return dict(copies=[[hexf(f32(Fraction(x))) for x in col] for col in copies], counts=counts,
                avg=[hexf(x) for x in avg], bf16=[bf16_bits(x) for x in avg])


def build():
    return dict(
        sync=[
            # one element, two buffers 2^-10 and 2^-9: mean 1.5*2^-10, norm << 1 so clipping is inactive
            sync_case("clip_inactive", [[0x3A80], [0x3B00]], [0.02], 2, 1, 2),
            # mean gradient (3, 4): norm 5, clipping active with c = 1/(5+1e-6)
            sync_case("clip_active", [[0x4040, 0x4080]], [0.5, -0.25], 1, 1, 2),
            # two-level (2 replicas x 2 shards), three elements, mixed signs
            sync_case("hsdp_2x2", [[0x3F80, 0xBF00, 0x3C00], [0x4000, 0x3E80, 0xBC00], [0xC040, 0x3F00, 0x3B80], [0x3F00, 0x3F00, 0x3B80]],
                      [0.125, -0.0625, 0.02], 2, 2, 3),
        ],
        fedavg=[
            fedavg_case([[0.5, 1.0], [-0.25, 1.0], [0.125, 1.0]], [1, 2, 5]),      # (0.5 - 0.5 + 0.625)/8 = 0.078125
            fedavg_case([[0.02, -0.3], [0.021, -0.31]], [306, 126]),
        ],
    )


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "worked_cases.json")
    with open(path, "w") as f:
        json.dump(build(), f, indent=1)
        f.write("\n")
    print("wrote", path)
