"""Ozaki Scheme II in Python big integers and exact fractions -- tiny inputs only.

TEST INFRASTRUCTURE ONLY.  A second, independent statement of the method used to
pin the C oracle: nothing here calls the C library, and every quantity is exact
(`int`, `fractions.Fraction`), so there is no rounding anywhere except the single
final conversion that the method itself prescribes (Sec. 2, step (iv)).

Follows Sec. 2 Eq. 1-5, Algorithm 2 with Lemma 1, and Algorithm 3.
"""
from __future__ import annotations

import math
from fractions import Fraction

SETS = {
    "S": [1089, 1024, 961, 841, 625, 529, 511, 509, 503, 499, 491, 487],
    "E": [1089, 1024, 961, 841, 625, 529, 251, 247, 241, 239, 233, 229, 227],
    "A": [256, 255, 253, 251, 247, 241, 239, 233, 229, 227, 223, 217, 211, 199, 197],
}


def product(ms):
    out = 1
    for m in ms:
        out *= m
    return out


def floor_log2(x: Fraction) -> int:
    """floor(log2 x) for an exact positive rational."""
    e = x.numerator.bit_length() - x.denominator.bit_length()
    if Fraction(2) ** e > x:
        e -= 1
    while Fraction(2) ** (e + 1) <= x:
        e += 1
    return e


def budget_maxexp(ms, k):
    T = ((product(ms) - 1) // 2 // k).bit_length() - 1
    return T - T // 2, T // 2


def cs_bound(ms, k):
    bnd = math.isqrt((product(ms) - 1) // 2)
    g = 0
    while 4 * g * g < k:
        g += 1
    return bnd - g


def shift_of_line(line, ms, rule, tbits, k):
    """line: list of floats (finite).  Returns sigma (Eq. 1)."""
    nz = [abs(Fraction(x)) for x in line if x != 0]
    if not nz:
        return 0
    E = max(floor_log2(x) for x in nz)
    if rule == "MAXEXP":
        return tbits - 1 - E
    S = sum(math.ceil(x * Fraction(2) ** (9 - E)) ** 2 for x in nz)
    G2 = cs_bound(ms, k) ** 2
    p = 0
    while 4 ** (p + 1) * S <= G2:
        p += 1
    return p + 9 - E


def esc_flatness(line, k):
    """Exponent-span check: floor(2^16 (sum abar)^2 / (k sum abar^2)), abar = ceil(|x| 2^(9-E)); None for
    a line of zeros."""
    nz = [abs(Fraction(x)) for x in line if x != 0]
    if not nz:
        return None
    E = max(floor_log2(x) for x in nz)
    ab = [math.ceil(x * Fraction(2) ** (9 - E)) for x in nz]
    return (sum(ab) ** 2 * 2 ** 16) // (k * sum(a * a for a in ab))


def esc_threshold(ms):
    """floor(2^32 (16/3) 2^104 / H) up to the truncation of H to its top bits, H = (M-1)/2."""
    return min(2 ** 32 - 1, (2 ** 120 // 3) // (((product(ms) - 1) // 2) >> 20))


def esc_rows(A, B, ms):
    """Rows of the product that go to the native FP64 path: q(a_i) against the least flat column of B,
    both capped at 2^16, below the set's threshold.  A: m x k, B: k x n nested lists."""
    k, n = len(B), len(B[0])
    qb = [esc_flatness([B[kk][j] for kk in range(k)], k) for j in range(n)]
    qb = min([min(q, 2 ** 16) for q in qb if q is not None], default=2 ** 16)
    out = []
    for row in A:
        qa = esc_flatness(row, k)
        out.append(0 if qa is None else int(min(qa, 2 ** 16) * qb < esc_threshold(ms)))
    return out


def _rn(x: Fraction) -> float:
    return float(x)          # exact rational -> nearest double, ties to even


def native_dot(a, b) -> float:
    """The compensated inner product of the native path, every floating-point operation written as
    the correctly rounded value of its exact rational result (finite data, no overflow)."""
    acc, comp = 0.0, 0.0
    for x, y in zip(a, b):
        fx, fy = Fraction(x), Fraction(y)
        p = _rn(fx * fy)
        pe = _rn(fx * fy - Fraction(p))
        s = _rn(Fraction(acc) + Fraction(p))
        bb = _rn(Fraction(s) - Fraction(acc))
        t1 = _rn(Fraction(acc) - Fraction(_rn(Fraction(s) - Fraction(bb))))
        t2 = _rn(Fraction(p) - Fraction(bb))
        se = _rn(Fraction(t1) + Fraction(t2))
        comp = _rn(Fraction(comp) + Fraction(_rn(Fraction(pe) + Fraction(se))))
        acc = s
    return _rn(Fraction(acc) + Fraction(comp))


def bound_digit(x: float, E: int) -> int:
    """Accurate mode: the smallest E4M3-representable integer that is >= |x| 2^(4-E)."""
    if x == 0:
        return 0
    g = math.ceil(abs(Fraction(x)) * Fraction(2) ** (4 - E))
    while g not in _E:
        g += 1
    return g


def shifts_accurate(A, B, ms):
    """Accurate mode (Sec. 2 "The FP8 variant": the extra magnitude-bound product).  A: m x k nested
    lists, B: k x n nested lists of finite floats.  Returns (sigma, tau, rowmax, colmax)."""
    m, k, n = len(A), len(B), len(B[0])
    rows = [A[i] for i in range(m)]
    cols = [[B[kk][j] for kk in range(k)] for j in range(n)]

    def line_exponent(line):
        nz = [abs(Fraction(x)) for x in line if x != 0]
        return max(floor_log2(x) for x in nz) if nz else None

    EA, EB = [line_exponent(l) for l in rows], [line_exponent(l) for l in cols]
    GA = [[bound_digit(x, EA[i]) if EA[i] is not None else 0 for x in rows[i]] for i in range(m)]
    GB = [[bound_digit(x, EB[j]) if EB[j] is not None else 0 for x in cols[j]] for j in range(n)]
    Cbar = [[sum(GA[i][kk] * GB[j][kk] for kk in range(k)) for j in range(n)] for i in range(m)]
    rowmax = [max(Cbar[i]) if n else 0 for i in range(m)]
    colmax = [max(Cbar[i][j] for i in range(m)) if m else 0 for j in range(n)]
    Hp = ((product(ms) - 1) // 2 // 129) * 128
    L = Hp.bit_length() - 1

    def ceil_log2(v):
        return (v - 1).bit_length() if v > 1 else 0

    sigma = [0 if EA[i] is None else (L - ceil_log2(rowmax[i])) // 2 + 4 - EA[i] for i in range(m)]
    tau = [0 if EB[j] is None else (L - ceil_log2(colmax[j])) // 2 + 4 - EB[j] for j in range(n)]
    return sigma, tau, rowmax, colmax


def quantise(x: float, sigma: int, quant: str) -> int:
    v = Fraction(x) * Fraction(2) ** sigma
    if quant == "TZ":
        return int(v)  # int() truncates toward zero
    return round(v)  # Fraction.__round__ rounds half to even


def centred(x: int, m: int) -> int:
    d = x % m
    return d - m if 2 * d >= m else d


def e4m3_integers():
    """All integers exactly representable in E4M3 (the set of Lemma 1)."""
    vals = set()
    for e in range(16):
        for f in range(8):
            if e == 15 and f == 7:
                continue
            v = Fraction(f, 8) * Fraction(2) ** -6 if e == 0 else (1 + Fraction(f, 8)) * Fraction(2) ** (e - 7)
            if v.denominator == 1:
                vals.add(int(v))
                vals.add(-int(v))
    return vals


_E = e4m3_integers()


def split(d: int, m: int):
    s = math.isqrt(m)
    if s * s == m:
        lo = s // 2
        d0 = (d + lo) % s - lo
        return [d0, (d - d0) // s]
    d0 = (d + 8) % 16 - 8
    d1 = (d - d0) // 16
    if d0 + d1 not in _E:
        sg = (d0 > 0) - (d0 < 0)
        d0, d1 = d0 - 16 * sg, d1 + sg
    return [d0, d1, d0 + d1]


def garner(res, ms) -> int:
    v = []
    for j, m in enumerate(ms):
        if j == 0:
            v.append(res[0] % m)
            continue
        partial, weight = 0, 1
        for l in range(j):
            partial += v[l] * weight
            weight *= ms[l]
        w = pow(weight, -1, m)
        v.append(((res[j] - partial) * w) % m)
    x = 0
    for j in reversed(range(len(ms))):
        x = x * ms[j] + v[j]
    M = product(ms)
    return x - M if 2 * x >= M else x


def int_to_float_rn(x: int) -> float:
    return float(Fraction(x))  # exact rational -> nearest double, ties to even


def dgemm(A, B, set_name="S", quant="RN", rule="CS"):
    """A: m x k nested lists, B: k x n nested lists -> (C, sigma, tau, R, Cint)."""
    ms = SETS[set_name]
    m, k, n = len(A), len(B), len(B[0])
    tA, tB = budget_maxexp(ms, k)
    if rule == "ACCURATE":
        sig, tau, _, _ = shifts_accurate(A, B, ms)
    else:
        sig = [shift_of_line(A[i], ms, rule, tA, k) for i in range(m)]
        tau = [shift_of_line([B[kk][j] for kk in range(k)], ms, rule, tB, k) for j in range(n)]
    QA = [[quantise(A[i][kk], sig[i], quant) for kk in range(k)] for i in range(m)]
    QB = [[quantise(B[kk][j], tau[j], quant) for kk in range(k)] for j in range(n)]
    R = [[[sum(centred(QA[i][kk], mm) * centred(QB[j][kk], mm) for kk in range(k)) % mm
           for i in range(m)] for j in range(n)] for mm in ms]
    Cint = [[garner([R[q][j][i] for q in range(len(ms))], ms) for j in range(n)] for i in range(m)]
    Cf = [[float(Fraction(int_to_float_rn(Cint[i][j])) * Fraction(2) ** -(sig[i] + tau[j]))
           for j in range(n)] for i in range(m)]
    return Cf, sig, tau, R, Cint
