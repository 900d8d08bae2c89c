"""Exact-rational re-statement of the method for brute-force checks of the oracle.

Deliberately a different formulation from ``oracle/pipe_oracle.c``: every binary32
operation is done as an exact ``Fraction`` computation followed by one explicit
round-to-nearest-even to the binary32 grid implemented with integers, the contraction
uses Python ints, and the group selection is a full sort of (-score, index) tuples.
Only usable on tiny inputs.
"""
from fractions import Fraction

import numpy as np


def rne_int(x: Fraction) -> int:
    """Round a rational to the nearest integer, ties to even."""
    fl = x.numerator // x.denominator
    rem = x - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        return fl + 1
    return fl


def f32(x: Fraction) -> Fraction:
    """Round a rational to the nearest binary32 value (ties to even, gradual underflow)."""
    if x == 0:
        return Fraction(0)
    sign = -1 if x < 0 else 1
    ax = abs(x)
    e = ax.numerator.bit_length() - ax.denominator.bit_length()  # 2^(e-1) <= ax < 2^(e+1)
    if Fraction(2) ** e > ax:
        e -= 1
    # now 2^e <= ax < 2^(e+1); the grid step is 2^(e-23), never finer than 2^-149
    step_exp = max(e - 23, -149)
    n = rne_int(ax / Fraction(2) ** step_exp)
    out = n * Fraction(2) ** step_exp
    assert out < Fraction(2) ** 128, "overflow to infinity not modelled"
    return sign * out


def frac(v) -> Fraction:
    return Fraction(float(v))  # exact: every binary32/64 value is a dyadic rational


def expand_exact(W: np.ndarray, bits: int, K: int, g: int, n_keep: int):
    """Returns (codes[k] -> {row o: [ints]}, scales[k] -> {o: Fraction}, kept[k] -> [groups], residual)."""
    O, I = W.shape
    G = O // g
    qmax = 2 ** (bits - 1) - 1
    r = [[frac(W[o, i]) for i in range(I)] for o in range(O)]
    codes, scales, kept = [], [], []
    for k in range(K):
        a = [max(abs(v) for v in r[o]) for o in range(O)]
        if k == 0 or n_keep == G:
            kg = list(range(G))
        else:
            score = [max(a[j * g:(j + 1) * g]) for j in range(G)]
            ranked = sorted(range(G), key=lambda j: (-score[j], j))
            kg = sorted(ranked[:n_keep])
        ck, sk = {}, {}
        for j in kg:
            for o in range(j * g, (j + 1) * g):
                s = f32(a[o] / qmax)
                sk[o] = s
                if s == 0:
                    ck[o] = [0] * I
                    continue
                q = []
                for i in range(I):
                    t = f32(r[o][i] / s)
                    c = max(-qmax, min(qmax, rne_int(t)))
                    q.append(c)
                    r[o][i] = f32(r[o][i] - s * c)
                ck[o] = q
        codes.append(ck)
        scales.append(sk)
        kept.append(kg)
    return codes, scales, kept, r


def quantize_act_exact(x: np.ndarray):
    m = max(abs(frac(v)) for v in x.reshape(-1))
    sx = f32(m / 127)
    if sx == 0:
        return np.zeros(x.shape, np.int64), sx
    xq = np.array([[max(-127, min(127, rne_int(f32(frac(v) / sx)))) for v in row] for row in x], dtype=np.int64)
    return xq, sx


def forward_exact(codes, scales, xq, sx: Fraction, k_begin: int, k_end: int, O: int, bias=None):
    """y[t][o] as Fractions lying on the binary32 grid, and the integer partials {(k, o): [acc_t]}."""
    T = xq.shape[0]
    y = [[Fraction(0)] * O for _ in range(T)]
    partials = {}
    for t in range(T):
        for o in range(O):
            acc_y = Fraction(0)
            for k in range(k_begin, k_end):
                if o not in codes[k]:
                    continue
                acc = sum(int(xq[t, i]) * int(c) for i, c in enumerate(codes[k][o]))
                partials.setdefault((k, o), [0] * T)[t] = acc
                c = f32(scales[k][o] * sx)
                acc_y = f32(f32(Fraction(acc)) * c + acc_y)
            if bias is not None:
                acc_y = f32(acc_y + frac(bias[o]))
            y[t][o] = acc_y
    return y, partials
