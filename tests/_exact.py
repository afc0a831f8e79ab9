"""Exact helpers for the oracle pins: correctly rounded binary32 from
rationals, and a big-integer restatement of the explorer's generator.
Independent of oracle/ and of the CUDA sources."""
from fractions import Fraction

import numpy as np

M32 = 0xFFFFFFFF


def frac(x) -> Fraction:
    return Fraction(float(x))


def round_f32(fr: Fraction) -> np.float32:
    """Round a rational to binary32, nearest, ties to even (subnormals, overflow to inf)."""
    if fr == 0:
        return np.float32(0.0)
    neg = fr < 0
    a = -fr if neg else fr
    e = a.numerator.bit_length() - a.denominator.bit_length()
    while Fraction(2) ** e > a:
        e -= 1
    while Fraction(2) ** (e + 1) <= a:
        e += 1
    e = max(e, -126)
    ulp = Fraction(2) ** (e - 23)
    q = a / ulp
    n = q.numerator // q.denominator
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    val = n * ulp
    if val >= Fraction(2) ** 128:
        out = np.float32(np.inf)
    else:
        out = np.float32(float(val))
        assert Fraction(float(out)) == val
    return -out if neg else out


def fma_f32(a, b, c) -> np.float32:
    """a*b + c with one rounding, from exact rationals."""
    return round_f32(frac(a) * frac(b) + frac(c))


def philox_py(key, ctr):
    k0, k1 = key
    c = list(ctr)
    for r in range(10):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k0, p1 & M32, (p0 >> 32) ^ c[3] ^ k1, p0 & M32]
        if r < 9:
            k0 = (k0 + 0x9E3779B9) & M32
            k1 = (k1 + 0xBB67AE85) & M32
    return c


def round_keys_py(seed, worker, rnd):
    out = []
    for b in range(3):
        out += philox_py((seed & M32, (seed >> 32) & M32), (b, worker, rnd, 0x534C494D))
    return out


def perm_py(j, M, rk):
    b = 2
    while (1 << b) < M:
        b += 1
    a = b // 2
    c = b - a
    mask_a, mask_b = (1 << a) - 1, (1 << c) - 1
    x = j
    while True:
        A, B = x >> c, x & mask_b
        for r in range(10):
            v = ((B if r % 2 == 0 else A) ^ rk[r]) & M32
            p = v * (0xD2511F53 if r % 2 == 0 else 0xCD9E8D57)
            F = ((p >> 32) ^ p) & M32
            if r % 2 == 0:
                A = (A ^ F) & mask_a
            else:
                B = (B ^ F) & mask_b
        x = (A << c) | B
        if x < M:
            return x


def explore_py(core, n, k_exp, seed, worker, rnd):
    core_set = set(int(i) for i in core)
    noncore = [i for i in range(n) if i not in core_set]
    rk = round_keys_py(seed, worker, rnd)
    return sorted(noncore[perm_py(j, len(noncore), rk)] for j in range(k_exp))
