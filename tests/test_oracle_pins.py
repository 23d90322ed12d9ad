"""Pins for the CPU oracle: values the paper prints, closed forms, exhaustive
identities and a Python big-integer restatement.  No GPU, no CUDA library."""
import math
import os
import random
from fractions import Fraction

import numpy as np
import pytest

from oracle import oz_bigint as big
from oracle import oz_oracle as ozo
import synth_inputs as syn

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if "=" in line:
                key, val = [t.strip() for t in line.split("=", 1)]
                out[key] = val
    return out


PAPER = read_golden("paper_constants.txt")
SETS = {"S": ozo.SET_S, "E": ozo.SET_E, "A": ozo.SET_A}


# ----------------------------------------------------------------- P1: the sets
def test_modulus_sets_match_paper():
    S = [int(v) for v in PAPER["set_S"].split()]
    assert ozo.modset(ozo.SET_S) == S
    tail = [int(v) for v in PAPER["set_E_tail"].split()]
    assert ozo.modset(ozo.SET_E) == S[:6] + tail
    assert ozo.modset(ozo.SET_A) == [int(v) for v in PAPER["set_A"].split()]


@pytest.mark.parametrize("name", ["S", "E", "A"])
def test_set_counts_and_range(name):
    ms = ozo.modset(SETS[name])
    for i, a in enumerate(ms):
        for b in ms[i + 1:]:
            assert math.gcd(a, b) == 1
    M = math.prod(ms)
    assert ozo.M(SETS[name]) == M
    assert round(math.log2(M), 1) == float(PAPER[f"log2M_{name}"])
    squares = sum(1 for m in ms if math.isqrt(m) ** 2 == m)
    assert squares == int(PAPER[f"squares_{name}"])
    assert ozo.pstore(SETS[name]) == int(PAPER[f"pstore_{name}"])
    assert 3 * len(ms) == int(PAPER[f"pmma_{name}"])
    assert 3 * len(ms) + 1 == int(PAPER[f"alpha_{name}"])
    assert sum(ozo.planes_of(m) for m in ms) == 2 * squares + 3 * (len(ms) - squares)


# ----------------------------------------------------------------- range budget
@pytest.mark.parametrize("name", ["S", "E", "A"])
@pytest.mark.parametrize("k", [1, 7, 256, 1024, 4096, 5003, 32768])
def test_budget_is_inside_crt_range(name, k):
    M = math.prod(ozo.modset(SETS[name]))
    tA, tB = ozo.budget_maxexp(SETS[name], k)
    assert tA - tB in (0, 1)
    assert k * 2 ** (tA + tB) <= (M - 1) // 2          # Eq. 2 with |a'| <= 2^t
    assert k * 2 ** (tA + tB + 1) > (M - 1) // 2       # and T is the largest such
    assert (tA, tB) == big.budget_maxexp(ozo.modset(SETS[name]), k)
    G = ozo.cs_bound(SETS[name], k)
    assert G == big.cs_bound(ozo.modset(SETS[name]), k)
    g = math.isqrt((M - 1) // 2) - G
    assert 2 * g >= math.sqrt(k) and 2 * (g - 1) < math.sqrt(k)


# ----------------------------------------------------------------- P2/P3: byte-plane reduction
def test_dp4a_worked_example():
    ex = read_golden("dp4a_worked_example.txt")
    m = int(ex["m"])
    x = int(ex["x"], 16)
    consts = [pow(256, j, m) for j in range(4)]
    assert consts == [int(v) for v in ex["constants"].split()]
    assert [c & 255 for c in consts] == [int(v) for v in ex["constants_low_limb"].split()]
    assert [c >> 8 for c in consts] == [int(v) for v in ex["constants_high_limb"].split()]
    res, u0, u1, _, _ = ozo.byteplane_residue(x, m, 4)
    assert [(x >> (8 * j)) & 255 for j in range(4)] == [int(v) for v in ex["planes"].split()]
    assert (u0, u1) == (int(ex["partial_low"]), int(ex["partial_high"]))
    assert u0 + 256 * u1 == int(ex["recombined"])
    assert res == int(ex["residue"]) == x % m
    a, b = [int(v) for v in ex["identical_high_limbs"].split()]
    assert [pow(256, j, a) >> 8 for j in range(8)] == [pow(256, j, b) >> 8 for j in range(8)]


def test_byteplane_identity_signed_equivalence():
    rng = random.Random(3)
    worst_c = 0
    for m in ozo.modset(ozo.SET_S):
        xs = list(range(-2**15, 2**15, 7)) + [-2**63, 2**63 - 1, -1, 0, 1, -m, m, -m // 2]
        xs += [rng.randrange(-2**63, 2**63) for _ in range(300)]
        xs += [rng.randrange(-2**b, 2**b) for b in range(8, 63, 6) for _ in range(20)]
        for x in xs:
            res, u0, u1, mc, mh = ozo.byteplane_residue(x, m, 8)
            assert res == x % m
            assert 0 <= u0 < int(PAPER["byte_dot_bound"]) and 0 <= u1 < int(PAPER["byte_dot_bound"])
            assert mh <= 4
            worst_c = max(worst_c, mc)
            # the centred residue function agrees with the canonical one
            d = ozo.centred_residue(x, m)
            assert (d - x) % m == 0 and -m <= 2 * d < m
    assert worst_c == int(PAPER["max_reduction_constant_S"])


def test_centred_interval_endpoint_rule():
    # "for even x the endpoint -x/2 is included and +x/2 excluded"
    assert ozo.centred_residue(512, 1024) == -512
    assert ozo.centred_residue(-512, 1024) == -512
    assert ozo.centred_residue(511, 1024) == 511
    assert ozo.centred_residue(544, 1089) == 544
    assert ozo.centred_residue(545, 1089) == -544


# ----------------------------------------------------------------- P4: Lemma 1, exhaustive
def test_e4m3_set_definition():
    # integers M*2^e with |M| <= 15 and magnitude at most 448
    want = set()
    for mant in range(-15, 16):
        for e in range(0, 9):
            v = mant * 2 ** e
            if abs(v) <= 448:
                want.add(v)
    got = {v for v in range(-600, 601) if ozo.in_e4m3(v)}
    assert got == want == {v for v in big.e4m3_integers() if abs(v) <= 600}
    for v in sorted(want):
        code = ozo.e4m3_encode(v)
        assert 0 <= code < 256 and ozo.e4m3_value(code) == v
    assert ozo.e4m3_encode(0) == 0
    assert not any(ozo.in_e4m3(v) for v in (17, 19, 21, 23, -17, 449))
    # a few codes fixed by the format itself: 1.0 = 0x38, 448 = 0x7E, -2 = 0xC0
    assert ozo.e4m3_value(0x38) == 1.0 and ozo.e4m3_value(0x7E) == 448.0
    assert ozo.e4m3_value(0xC0) == -2.0 and ozo.e4m3_value(0x01) == 2.0 ** -9


@pytest.mark.parametrize("m", [487, 491, 499, 503, 509, 511])
def test_lemma1_exhaustive(m):
    lo, hi = -(m // 2), (m - 1) // 2
    planes = {d: ozo.split(d, m) for d in range(lo, hi + 1)}
    carries = 0
    for d, (d0, d1, ds) in planes.items():
        assert d == d0 + 16 * d1 and ds == d0 + d1
        assert all(ozo.in_e4m3(v) for v in (d0, d1, ds))
        assert abs(d0) <= int(PAPER["lemma1_d0_max"])
        assert abs(d1) <= int(PAPER["lemma1_d1_max"])
        assert abs(ds) <= int(PAPER["lemma1_sum_max"])
        canon0 = (d + 8) % 16 - 8
        if d0 != canon0:
            carries += 1
            assert abs(canon0 + (d - canon0) // 16) in [int(v) for v in PAPER["lemma1_failing_sums"].split()]
        assert planes[d] == big.split(d, m)
    if m == 511:
        assert carries == int(PAPER["lemma1_carries_at_511"])
    worst_prod = worst_merged = 0
    for d, (d0, d1, ds) in planes.items():
        for e, (e0, e1, es) in planes.items():
            assert d * e == -15 * d0 * e0 + 16 * ds * es + 240 * d1 * e1          # Eq. 8
            assert d * e == -15 * (d0 * e0 - 16 * d1 * e1) + 16 * ds * es          # merged form
            worst_prod = max(worst_prod, abs(d0 * e0), abs(ds * es), abs(d1 * e1))
            worst_merged = max(worst_merged, abs(d0 * e0 - 16 * d1 * e1))
    assert worst_prod <= int(PAPER["lemma1_product_max"])
    assert worst_merged <= int(PAPER["merged_term_max"])
    if m == 511:
        assert worst_prod == int(PAPER["lemma1_product_max"])
    assert 2 ** 24 // int(PAPER["lemma1_product_max"]) == int(PAPER["lemma1_K_exact"])
    assert 2 ** 24 // int(PAPER["merged_term_max"]) == int(PAPER["merged_K_exact"])


@pytest.mark.parametrize("name", ["S", "E", "A"])
def test_merged_accumulator_layout(name):
    """N_acc = 2 per modulus: regrouped Eq. 8 with the pre-scaled plane -16*d1 on one operand."""
    ms = ozo.modset(SETS[name])
    nonsq = [m for m in ms if math.isqrt(m) ** 2 != m]
    # accumulators: 2 per modulus when merged (E and A rows of the table); S keeps 3 on its tail unmerged
    assert 2 * len(ms) == {"S": 24, "E": int(PAPER["nacc_E"]), "A": int(PAPER["nacc_A"])}[name]
    assert 2 * (len(ms) - len(nonsq)) + 3 * len(nonsq) == {"S": int(PAPER["nacc_S"]), "E": 33, "A": 44}[name]
    # the pre-scaled plane takes the place of d1 on one operand: the table's p_store is unchanged
    assert ozo.pstore_merged(SETS[name], 0) == ozo.pstore_merged(SETS[name], 1) == int(PAPER["pstore_" + name])
    worst = 0
    for m in nonsq:
        lo, hi = -(m // 2), (m - 1) // 2
        sp = {d: ozo.split(d, m) for d in range(lo, hi + 1)}
        pre = [-16 * d1 for (_, d1, _) in sp.values()]
        assert all(ozo.in_e4m3(v) for v in pre)
        if m > 256:
            assert min(pre) == int(PAPER["merged_prescaled_plane_extreme"])
        a = max(abs(d0) for (d0, _, _) in sp.values())
        b = max(abs(d1) for (_, d1, _) in sp.values())
        here = max(abs(d0 * e0 - 16 * d1 * e1) for (d0, d1, _) in sp.values()
                   for (e0, e1, _) in list(sp.values())[:: max(1, len(sp) // 97)] + [sp[lo], sp[hi]])
        assert here <= a * a + 16 * b * b
        worst = max(worst, here)
    if name == "S":
        assert worst <= int(PAPER["merged_term_max"])
    else:
        assert worst <= 1088 and 2 ** 24 // 1088 == int(PAPER["merged_K_exact_byte"])
    rng = np.random.default_rng(31)
    m_, n_, k = 5, 4, 41
    QA = rng.integers(-2**50, 2**50, size=(m_, k))
    QB = rng.integers(-2**50, 2**50, size=(n_, k))
    DA, DB = ozo.residues(QA, SETS[name]), ozo.residues(QB, SETS[name])
    PA, PB = ozo.planes_merged(0, DA, SETS[name]), ozo.planes_merged(1, DB, SETS[name])
    assert (PB == ozo.planes(DB, SETS[name], ozo.SUB_FP8)).all()
    # side 0 differs from the plain layout in exactly the d1 planes of the non-square moduli
    plain, p0 = ozo.planes(DA, SETS[name], ozo.SUB_FP8), 0
    for m in ms:
        np_ = 2 if math.isqrt(m) ** 2 == m else 3
        for q in range(np_):
            same = (PA[p0 + q] == plain[p0 + q]).all()
            assert same or (np_ == 3 and q == 1)
        if np_ == 3:
            d1 = np.array([[ozo.split(int(d), m)[1] for d in row] for row in DA[ms.index(m)]])
            want = np.array([[ozo.e4m3_encode(-16 * int(v)) for v in row] for row in d1], dtype=np.uint8)
            assert (PA[p0 + 1][:, :k] == want).all()
        p0 += np_
    R, w = ozo.plane_products_merged(PA, PB, k, SETS[name])
    assert (R == ozo.products(DA, DB, SETS[name])).all() and w <= 4095 * k


@pytest.mark.parametrize("name", ["S", "E", "A"])
def test_merged_accumulator_layout_on_int8(name):
    """The N_acc = 2 regrouping on the INT8 substrate: d e = 15 [(-d0) e0 + (4 d1)(4 e1)] + 16 dS eS.
    The identity holds for every pair of residues of every non-square modulus, every stored value
    fits a signed byte, the merged term is at most 196 + 16 * 256, and the planes reproduce the
    residue products."""
    ms = ozo.modset(SETS[name])
    nonsq = [m for m in ms if math.isqrt(m) ** 2 != m]
    worst = 0
    for m in nonsq:
        lo, hi = -(m // 2), (m - 1) // 2
        sp = {d: ozo.split(d, m) for d in range(lo, hi + 1)}
        assert all(-128 <= -d0 <= 127 and -128 <= 4 * d1 <= 127 and -128 <= ds <= 127 for (d0, d1, ds) in sp.values())
        probe = list(sp.items())[:: max(1, len(sp) // 61)] + [(lo, sp[lo]), (hi, sp[hi])]
        for d, (d0, d1, ds) in sp.items():
            for e, (e0, e1, es) in probe:
                merged = (-d0) * e0 + (4 * d1) * (4 * e1)
                assert (15 * merged + 16 * ds * es - d * e) % m == 0
                worst = max(worst, abs(merged))
    assert worst <= 196 + 16 * 256 == 4292
    rng = np.random.default_rng(33)
    m_, n_, k = 5, 4, 41
    QA = rng.integers(-2**50, 2**50, size=(m_, k))
    QB = rng.integers(-2**50, 2**50, size=(n_, k))
    DA, DB = ozo.residues(QA, SETS[name]), ozo.residues(QB, SETS[name])
    PA = ozo.planes_merged(0, DA, SETS[name], substrate=ozo.SUB_INT8)
    PB = ozo.planes_merged(1, DB, SETS[name], substrate=ozo.SUB_INT8)
    plainA, plainB, p0 = ozo.planes(DA, SETS[name], ozo.SUB_INT8), ozo.planes(DB, SETS[name], ozo.SUB_INT8), 0
    for mm in ms:
        if math.isqrt(mm) ** 2 == mm:
            assert (PA[p0:p0 + 2] == plainA[p0:p0 + 2]).all() and (PB[p0:p0 + 2] == plainB[p0:p0 + 2]).all()
            p0 += 2
            continue
        d0, d1 = plainA[p0].view(np.int8).astype(int), plainA[p0 + 1].view(np.int8).astype(int)
        assert (PA[p0].view(np.int8) == -d0).all() and (PA[p0 + 1].view(np.int8) == 4 * d1).all()
        assert (PA[p0 + 2] == plainA[p0 + 2]).all()
        e1 = plainB[p0 + 1].view(np.int8).astype(int)
        assert (PB[p0] == plainB[p0]).all() and (PB[p0 + 1].view(np.int8) == 4 * e1).all()
        assert (PB[p0 + 2] == plainB[p0 + 2]).all()
        p0 += 3
    R, w = ozo.plane_products_merged(PA, PB, k, SETS[name], ozo.SUB_INT8)
    assert (R == ozo.products(DA, DB, SETS[name])).all() and w <= 4292 * k


def test_lemma1_is_sharp_at_513():
    def rule(d):
        d0 = (d + 8) % 16 - 8
        d1 = (d - d0) // 16
        if not ozo.in_e4m3(d0 + d1):
            sg = (d0 > 0) - (d0 < 0)
            d0, d1 = d0 - 16 * sg, d1 + sg
        return d0, d1
    for m, ok in ((513, True), (514, False)):
        good = all(all(ozo.in_e4m3(v) for v in (*rule(d), sum(rule(d))))
                   for d in range(-(m // 2), (m - 1) // 2 + 1))
        assert good == ok


def test_all_byte_set_native_int8_planes():
    """Set A: every reduction constant fits a byte (largest 243, dot products < 2^19), every
    centred residue fits a signed byte (m = 256 reaches -128), one plane and one product per modulus."""
    ms = ozo.modset(ozo.SET_A)
    assert max(pow(256, j, m) for m in ms for j in range(8)) == int(PAPER["max_reduction_constant_A"])
    assert 8 * 255 * int(PAPER["max_reduction_constant_A"]) < int(PAPER["byte_dot_bound"])
    assert len(ms) + 1 == int(PAPER["alpha_A_int8_native"])
    assert ozo.pstore(ozo.SET_A, ozo.SUB_INT8_NATIVE) == len(ms) == 15
    assert ozo.pstore(ozo.SET_A, ozo.SUB_FP8) == int(PAPER["pstore_A"])
    assert ozo.centred_residue(128, 256) == -128 and ozo.centred_residue(-129, 256) == 127
    rng = np.random.default_rng(12)
    Q = rng.integers(-2**52, 2**52, size=(3, 40))
    Q[0, :15] = [m // 2 for m in ms]                    # the endpoint residues
    Q[1, :15] = [-(m // 2) for m in ms]
    D = ozo.residues(Q, ozo.SET_A)
    P = ozo.planes(D, ozo.SET_A, ozo.SUB_INT8_NATIVE)
    assert P.shape == (15, 3, 48)
    assert (P[:, :, :40].view(np.int8) == D).all() and (P[:, :, 40:] == 0).all()
    for i, m in enumerate(ms):
        assert ((D[i].astype(np.int64) - Q) % m == 0).all()
        assert D[i].min() >= -(m // 2) and D[i].max() <= (m - 1) // 2 and D[i].min() >= -128


def test_byte_moduli_never_carry():
    lo_s, hi_s = [int(v) for v in PAPER["byte_modulus_sum_range"].split()]
    for m in ozo.modset(ozo.SET_E)[6:] + ozo.modset(ozo.SET_A)[1:]:
        for d in range(-(m // 2), (m - 1) // 2 + 1):
            d0, d1, ds = ozo.split(d, m)
            assert d0 == (d + 8) % 16 - 8 and d == d0 + 16 * d1
            assert abs(d0) <= 8 and abs(d1) <= int(PAPER["byte_modulus_digit_max"])
            assert lo_s <= ds <= hi_s


# ----------------------------------------------------------------- P5: squares
@pytest.mark.parametrize("m", [1089, 1024, 961, 841, 625, 529])
def test_square_split_exhaustive(m):
    s = math.isqrt(m)
    lo, hi = -(m // 2), (m - 1) // 2
    digs = {d: ozo.split(d, m) for d in range(lo, hi + 1)}
    worst = 0
    for d, (d0, d1) in digs.items():
        assert d == d0 + s * d1
        assert ozo.in_e4m3(d0) and ozo.in_e4m3(d1)
        worst = max(worst, abs(d0), abs(d1))
        assert digs[d] == big.split(d, m)
        if s % 2 == 0:
            assert -s // 2 <= d0 <= s // 2 - 1
    assert worst <= int(PAPER["square_digit_max"])
    if m == 1089:
        assert worst == int(PAPER["square_digit_max"])          # "exactly tight at s=33"
    vals = list(digs.items())[:: max(1, len(digs) // 257)] + [(lo, digs[lo]), (hi, digs[hi])]
    for d, (d0, d1) in vals:
        for e, (e0, e1) in digs.items():
            assert (d * e - (d0 * e0 + s * (d1 * e0 + d0 * e1))) % m == 0   # epilogue {1,s,s}


# ----------------------------------------------------------------- P6: CRT round trip
@pytest.mark.parametrize("name", ["S", "E", "A"])
def test_crt_round_trip(name):
    ms = ozo.modset(SETS[name])
    M = math.prod(ms)
    w = ozo.garner_constants(SETS[name])
    for j in range(1, len(ms)):
        assert (w[j] * math.prod(ms[:j])) % ms[j] == 1 and 0 < w[j] < ms[j]
    rng = random.Random(11)
    xs = [0, 1, -1, -(M // 2), (M - 1) // 2, M // 2 - 1, -(M // 2) + 1, 12345678901234567890]
    xs += [rng.randrange(-(M // 2), (M + 1) // 2) for _ in range(400)]
    xs += [rng.randrange(-2**b, 2**b) for b in range(1, 110, 9)]
    for x in xs:
        res = [x % m for m in ms]
        assert ozo.crt_single(SETS[name], res) == x
        assert big.garner(res, ms) == x


def test_int128_to_double_is_correctly_rounded():
    rng = random.Random(5)
    xs = [0, 1, -1, 2**53, 2**53 + 1, 2**53 + 2, 2**53 + 3, -(2**53 + 1), 2**54 + 2, 2**54 + 6,
          2**100 + 2**47, 2**100 + 2**47 + 1, 2**100 + 3 * 2**47, -(2**110) - 2**57, 2**112 - 1]
    xs += [rng.randrange(-2**b, 2**b) for b in range(40, 120) for _ in range(25)]
    for x in xs:
        assert ozo.i128_to_double(x) == float(x), x   # Python's int -> float is RN-even


# ----------------------------------------------------------------- quantiser / shifts
def test_quantiser_against_exact_rationals():
    rng = np.random.default_rng(2)
    xs = np.concatenate([rng.standard_normal(200) * 10.0 ** rng.integers(-30, 30, 200),
                         [0.0, -0.0, 5e-324, -5e-324, 2.0**-1040, 1.5, 2.5, -2.5, 0.5, -0.5, 3.5]])
    for sigma in (-80, -3, 0, 1, 40, 52, 1074):
        for x in xs:
            X = np.asfortranarray(np.array([[x]]))
            sh = np.array([sigma], dtype=np.int32)
            v = Fraction(float(x)) * Fraction(2) ** sigma
            if abs(v) >= 2**62:
                continue
            assert int(ozo.quantise(0, X, sh, ozo.QUANT_RN)[0, 0]) == round(v)
            assert int(ozo.quantise(0, X, sh, ozo.QUANT_TZ)[0, 0]) == int(v)
    # ties go to even
    X = np.asfortranarray(np.array([[0.5, 1.5, 2.5, -0.5, -1.5]]))
    q = ozo.quantise(0, X, np.zeros(1, dtype=np.int32), ozo.QUANT_RN)
    assert q.tolist() == [[0, 2, 2, 0, -2]]


@pytest.mark.parametrize("rule", ["MAXEXP", "CS"])
@pytest.mark.parametrize("name", ["S", "E"])
def test_shifts_keep_product_in_range(rule, name):
    rng = np.random.default_rng(9)
    ms = ozo.modset(SETS[name])
    M = math.prod(ms)
    m, n, k = 9, 7, 33
    A = np.asfortranarray((rng.random((m, k)) - 0.5) * np.exp(3 * rng.standard_normal((m, k))))
    B = np.asfortranarray((rng.random((k, n)) - 0.5) * np.exp(3 * rng.standard_normal((k, n))))
    A[3, :] = A[3, 0]            # parallel row/column: the Cauchy-Schwarz bound is tight
    B[:, 2] = A[3, 0]
    A[5, 1:] = 0.0               # a single nonzero
    tA, tB = ozo.budget_maxexp(SETS[name], k)
    r = ozo.SCALE_MAXEXP if rule == "MAXEXP" else ozo.SCALE_CS
    sA = ozo.shifts(0, A, SETS[name], r, tA)
    sB = ozo.shifts(1, B, SETS[name], r, tB)
    for i in range(m):
        assert sA[i] == big.shift_of_line(A[i, :].tolist(), ms, rule, tA, k)
    for j in range(n):
        assert sB[j] == big.shift_of_line(B[:, j].tolist(), ms, rule, tB, k)
    for quant in (ozo.QUANT_RN, ozo.QUANT_TZ):
        QA = ozo.quantise(0, A, sA, quant).astype(object)
        QB = ozo.quantise(1, B, sB, quant).astype(object)
        Cp = QA @ QB.T
        assert max(abs(int(v)) for v in Cp.ravel()) <= (M - 1) // 2
        if rule == "MAXEXP":
            assert max(abs(int(v)) for v in QA.ravel()) <= 2**tA
            assert max(abs(int(v)) for v in QB.ravel()) <= 2**tB
            # the shift is the largest allowed: the top entry of a line uses bit t-1
            assert all(max(abs(int(v)) for v in QA[i]) >= 2**(tA - 1) for i in range(m))


# ----------------------------------------------------------------- exponent-span check
def test_esc_flatness_closed_forms_and_range():
    """q = floor(2^16 phi^2), phi^2 = ||x||_1^2 / (k ||x||_2^2) on the scan's integer magnitudes:
    1 for a constant line, 1/k for a single spike, between the two by Cauchy-Schwarz."""
    k = 48
    const = np.asfortranarray(np.full((1, k), -0.75))
    assert ozo.esc_flatness(0, const) == 65536
    spike = np.zeros((1, k), order="F")
    spike[0, 7] = 3.0e10
    assert ozo.esc_flatness(0, spike) == 65536 // k
    two = np.asfortranarray(np.array([[1.0] * 8 + [2.0 ** -3] * 40]))        # abar 512 x 8, 64 x 40
    l1, s2 = 512 * 8 + 64 * 40, 512 ** 2 * 8 + 64 ** 2 * 40
    assert ozo.esc_flatness(0, two) == (l1 * l1 * 65536) // (k * s2) == big.esc_flatness(two[0].tolist(), k)
    assert ozo.esc_flatness(1, np.asfortranarray(two.T)) == ozo.esc_flatness(0, two)   # same line as a column
    rng = np.random.default_rng(5)
    X = np.asfortranarray((rng.random((9, k)) - 0.5) * np.exp(3 * rng.standard_normal((9, k))))
    X[4, :] = 0.0                                                             # a line of zeros is skipped
    per_line = [big.esc_flatness(X[i].tolist(), k) for i in range(9)]
    assert per_line[4] is None and all(65536 // k <= q <= 65536 for q in per_line if q is not None)
    assert ozo.esc_flatness(0, X) == min(q for q in per_line if q is not None)
    X[2, 3] = np.inf                                                          # so is a line with Inf/NaN
    assert ozo.esc_flatness(0, X) == min(q for i, q in enumerate(per_line) if q is not None and i != 2)
    assert ozo.esc_flatness(0, np.zeros((3, k), order="F")) == 2 ** 32 - 1


@pytest.mark.parametrize("name", ["S", "E", "A"])
def test_esc_threshold_formula(name):
    ms = ozo.modset(SETS[name])
    H = (math.prod(ms) - 1) // 2
    thr = ozo.esc_threshold(SETS[name])
    assert thr == big.esc_threshold(ms)
    exact = Fraction(16, 3) * 2 ** 104 * 2 ** 32 / H                          # 2^32 (16/3) 2^104 / H
    assert abs(Fraction(thr) - exact) <= exact / 2 ** 20 + 1


@pytest.mark.parametrize("cfg_id,m,n,k", [(1, 64, 64, 256), (2, 48, 40, 4096), (3, 64, 48, 1024), (4, 96, 32, 4096),
                                          (5, 40, 36, 5003)])
def test_esc_check_separates_the_benchmark_distributions(cfg_id, m, n, k):
    """The check is a heuristic, so this is a calibration rather than a pin: on the five benchmark
    distributions it flags exactly the one whose measured error exceeds 2u(|A||B|) (the lognormal
    with sigma = 2), for every modulus set."""
    A, B = syn.operands(syn.CONFIGS[cfg_id], m, n, k)
    hi, lo, ab = ozo.dd_gemm(A, B)
    for name in ("S", "E", "A"):
        flagged = ozo.esc_check(A, B, SETS[name])
        worst = float((np.abs(ozo.dgemm(A, B, SETS[name]) - hi) / (2 * 2.0 ** -53 * ab)).max())
        assert flagged == (cfg_id == 5)
        assert (worst > 1.0) == flagged


# ----------------------------------------------------------------- out-of-range rows on the native FP64 path
def test_esc_rows_match_the_restatement_and_the_call_level_check():
    """Row i is re-issued when q(a_i) min_j q(b_j) < thr.  Pinned against the big-integer restatement,
    against closed-form lines (a constant row is never re-issued, a one-spike row against spiky
    columns is), and against the call-level check: a call is flagged exactly when some row is."""
    rng = np.random.default_rng(11)
    m, n, k = 14, 9, 160
    A = np.asfortranarray(rng.standard_normal((m, k)) * np.exp(2.5 * rng.standard_normal((m, k))))
    B = np.asfortranarray(rng.standard_normal((k, n)) * np.exp(2.5 * rng.standard_normal((k, n))))
    A[0, :] = 1.25                     # flat row
    A[1, :] = 0.0                      # zeros: not counted
    A[2, :] = 0.0
    A[2, 17] = -3.0                    # one spike: q = 2^16 / k
    A[3, 5] = np.nan                   # Inf/NaN rows are not re-issued (their result is NaN anyway)
    for name in ("S", "E", "A"):
        ms = ozo.modset(SETS[name])
        flag = ozo.esc_rows(A, B, SETS[name])
        A_ok = A.copy(order="F")
        A_ok[3, 5] = 1.0
        want = big.esc_rows(A_ok.tolist(), B.tolist(), ms)   # the restatement takes finite data only
        want[3] = 0
        assert flag.tolist() == want
        assert flag[1] == 0 and flag[3] == 0
        assert bool(ozo.esc_rows(A_ok, B, SETS[name]).any()) == ozo.esc_check(A_ok, B, SETS[name])
    # with perfectly flat columns the spike row passes on S (q_a q_b = 2^32 / k is far above the threshold) ...
    Bflat = np.asfortranarray(np.full((k, n), 0.5))
    assert ozo.esc_rows(A, Bflat, SETS["S"])[2] == (2 ** 32 // k < ozo.esc_threshold(SETS["S"]))
    # ... and against a one-spike column every counted row with q_a < thr k / 2^16 fails
    Bspike = np.zeros((k, n), order="F")
    Bspike[3, :] = 2.0
    f = ozo.esc_rows(A, Bspike, SETS["S"])
    per_row = [None if i == 3 else big.esc_flatness(A[i].tolist(), k) for i in range(m)]
    qb = 65536 // k
    assert [int(v) for v in f] == [0 if q is None else int(min(q, 65536) * qb < ozo.esc_threshold(SETS["S"]))
                                   for i, q in enumerate(per_row)]


def test_native_rows_are_the_compensated_dot_product_in_k_order():
    """The native path against its restatement in exact rationals (every operation = the correctly
    rounded value of its exact result), incl. cancellation, and against the bound of the compensated
    dot product: |res - a.b| <= u |a.b| + 2 (k u)^2 |a|.|b| -- far inside 2u (|A||B|)."""
    rng = np.random.default_rng(12)
    m, n, k = 5, 4, 37
    A = np.asfortranarray(rng.standard_normal((m, k)) * np.exp(4 * rng.standard_normal((m, k))))
    B = np.asfortranarray(rng.standard_normal((k, n)) * np.exp(4 * rng.standard_normal((k, n))))
    A[1, 1::2] = -A[1, 0:-1:2]                      # heavy cancellation in row 1 ...
    B[1::2, :] = B[0:-1:2, :]                       # ... against pairwise equal entries
    flag = np.array([1, 1, 0, 1, 0], dtype=np.uint8)
    C0 = np.asfortranarray(rng.standard_normal((m, n)))
    for alpha, beta in ((1.0, 0.0), (-1.0, 1.0), (1.0, 1.0)):
        got = ozo.native_rows(A, B, flag, alpha, beta, C0)
        for i in range(m):
            for j in range(n):
                if not flag[i]:
                    assert got[i, j] == C0[i, j]                     # untouched
                    continue
                v = big.native_dot(A[i].tolist(), B[:, j].tolist())
                want = alpha * v if beta == 0.0 else C0[i, j] + alpha * v
                assert got[i, j] == want
                exact = sum(Fraction(float(x)) * Fraction(float(y)) for x, y in zip(A[i], B[:, j]))
                mag = sum(abs(Fraction(float(x)) * Fraction(float(y))) for x, y in zip(A[i], B[:, j]))
                u = Fraction(1, 2 ** 53)
                assert abs(Fraction(v) - exact) <= u * abs(exact) + 2 * (k * u) ** 2 * mag
    # the order of the inner product is part of the definition: reversing k changes bits somewhere
    rev = ozo.native_rows(np.asfortranarray(A[:, ::-1]), np.asfortranarray(B[::-1, :]), flag)
    fwd = ozo.native_rows(A, B, flag)
    assert np.allclose(rev, fwd, rtol=1e-15, atol=0)
    # Inf/NaN in a column of B gives NaN in that column of the re-issued rows
    Bn = B.copy(order="F")
    Bn[4, 2] = np.inf
    out = ozo.native_rows(A, Bn, flag)
    assert np.isnan(out[flag == 1][:, 2]).all() and np.isfinite(out[flag == 1][:, [0, 1, 3]]).all()


def test_fallback_restores_the_accuracy_contract_on_the_wide_distribution():
    """Config-5 data (lognormal, sigma = 2): the plain method misses 2u (|A||B|); with the out-of-range
    rows re-issued every entry meets it, and the rows that were not re-issued are the method's."""
    A, B = syn.operands(syn.CONFIGS[5], 40, 36, 5003)
    hi, lo, ab = ozo.dd_gemm(A, B)
    bound = 2 * 2.0 ** -53 * ab
    plain = ozo.dgemm(A, B, SETS["S"])
    C, flag = ozo.dgemm_fallback(A, B, SETS["S"])
    assert (np.abs(plain - hi) > bound).any() and flag.any()
    assert (np.abs(C - hi) <= bound).all() if flag.all() else (np.abs(C - hi)[flag == 1] <= bound[flag == 1]).all()
    assert (C[flag == 0] == plain[flag == 0]).all()
    assert (C[flag == 1] == ozo.native_rows(A, B, flag)[flag == 1]).all()
    # on a benign distribution nothing is re-issued and the result is the method's, bit for bit
    A2, B2 = syn.operands(syn.CONFIGS[3], 33, 21, 512)
    C0 = np.asfortranarray(np.random.default_rng(3).standard_normal((33, 21)))
    C2, flag2 = ozo.dgemm_fallback(A2, B2, SETS["S"], alpha=-1.0, beta=1.0, C0=C0)
    assert not flag2.any() and (C2 == ozo.dgemm(A2, B2, SETS["S"], alpha=-1.0, beta=1.0, C0=C0)).all()


# ----------------------------------------------------------------- accurate mode: the "+1" bound product
def test_bound_digit_is_the_least_e4m3_upper_bound():
    """Sec. 2 "The FP8 variant": the extra product runs on FP8 operands, so its magnitude digits must
    be E4M3-exact; the digit is the least grid value not below |x| 2^(4-E)."""
    grid = sorted(v for v in range(0, 33) if ozo.in_e4m3(v))
    assert grid == list(range(0, 17)) + list(range(18, 33, 2))
    E = 3
    for num in range(0, 16 * 64 + 1):                       # |x| 2^(4-E) = num / 32, up to 32
        x = num / 32.0 * 2.0 ** (E - 4)
        g = ozo.bound_digit(x, E)
        exact = Fraction(num, 32)
        assert g in grid and g >= exact
        assert all(v < exact for v in grid if v < g)        # no smaller grid value bounds it
        assert ozo.bound_digit(-x, E) == g == big.bound_digit(x, E)
    assert ozo.bound_digit(5e-324, 0) == 1 and ozo.bound_digit(0.0, 0) == 0      # tiny but non-zero counts as 1
    assert ozo.bound_digit(float(np.nextafter(2.0 ** (E + 1), 0.0)), E) == 32


@pytest.mark.parametrize("name", ["S", "E", "A"])
def test_accurate_shifts_are_sound_and_match_the_restatement(name):
    """The shifts chosen from the bound product keep every |c'_ij| inside the CRT range -- checked by
    brute force in exact integers on random operands, on an operand pair that attains the bound
    (all entries at the top of their binade, equal signs) and with both quantisers -- and equal the
    big-integer restatement."""
    rng = np.random.default_rng(31)
    ms = ozo.modset(SETS[name])
    M = math.prod(ms)
    m, n, k = 8, 6, 40
    A = np.asfortranarray((rng.random((m, k)) - 0.5) * np.exp(3 * rng.standard_normal((m, k))))
    B = np.asfortranarray((rng.random((k, n)) - 0.5) * np.exp(3 * rng.standard_normal((k, n))))
    top = float(np.nextafter(2.0, 0.0))
    A[1, :] = top * 2.0 ** 5                                 # every digit 32, products aligned with column 2
    B[:, 2] = top * 2.0 ** -7
    A[4, 1:] = 0.0                                           # a single non-zero
    A[6, :] = 0.0                                            # a zero line
    B[:, 4] = 0.0
    sA, sB, rm, cm = ozo.shifts_accurate(A, B, SETS[name])
    sig, tau, rowmax, colmax = big.shifts_accurate(A.tolist(), B.tolist(), ms)
    assert sA.tolist() == sig and sB.tolist() == tau
    assert rm.tolist() == rowmax and cm.tolist() == colmax
    assert rm[1] == 1024 * k == cm[2] and sA[6] == 0 and sB[4] == 0
    L = ozo.accurate_budget_log2(SETS[name])
    assert 2 ** L <= ((M - 1) // 2 // 129) * 128 < 2 ** (L + 1)
    for quant in (ozo.QUANT_RN, ozo.QUANT_TZ):
        QA = ozo.quantise(0, A, sA, quant).astype(object)
        QB = ozo.quantise(1, B, sB, quant).astype(object)
        absC = np.abs(QA) @ np.abs(QB).T
        assert max(int(v) for v in absC.ravel()) <= (M - 1) // 2
    # on the pair that attains the bound the rule gives up less than three bits of the range
    # (a bit for each ceiling of a logarithm, half a bit for the halved exponent, the 1/129 margin)
    assert int(absC[1, 2]) * 8 > (M - 1) // 2
    # the whole method with this rule: C oracle == restatement
    Cm, s1, s2, R = ozo.dgemm(A, B, SETS[name], ozo.QUANT_RN, ozo.SCALE_ACCURATE, want_stages=True)
    Cf, sig2, tau2, Rb, _ = big.dgemm(A.tolist(), B.tolist(), name, "RN", "ACCURATE")
    assert s1.tolist() == sig2 == sig and s2.tolist() == tau2 and R.tolist() == Rb and Cm.tolist() == Cf


def test_accurate_rule_on_a_closed_form_case():
    """A = ones(m, k), B = ones(k, n): every digit is 16 (|x| 2^(4-0)), the bound product is 256 k,
    so sigma = tau = floor((L - ceil(log2(256 k))) / 2) + 4."""
    for name in ("S", "A"):
        L = ozo.accurate_budget_log2(SETS[name])
        for k in (1, 3, 64, 100):
            A, B = np.ones((2, k), order="F"), np.ones((k, 3), order="F")
            sA, sB, rm, cm = ozo.shifts_accurate(A, B, SETS[name])
            want = (L - math.ceil(math.log2(256 * k))) // 2 + 4
            assert rm.tolist() == [256 * k] * 2 and cm.tolist() == [256 * k] * 3
            assert sA.tolist() == [want] * 2 and sB.tolist() == [want] * 3


# ----------------------------------------------------------------- P7: brute force / big ints
@pytest.mark.parametrize("name,quant,rule", [("S", "RN", "CS"), ("S", "TZ", "MAXEXP"),
                                             ("E", "RN", "MAXEXP"), ("E", "TZ", "CS"),
                                             ("A", "RN", "CS"), ("A", "TZ", "MAXEXP")])
def test_whole_method_against_big_integers(name, quant, rule):
    rng = np.random.default_rng(21)
    m, n, k = 5, 4, 19
    A = np.asfortranarray((rng.random((m, k)) - 0.5) * np.exp(2 * rng.standard_normal((m, k))))
    B = np.asfortranarray((rng.random((k, n)) - 0.5) * np.exp(2 * rng.standard_normal((k, n))))
    A[2, 3] = 0.0
    q = ozo.QUANT_RN if quant == "RN" else ozo.QUANT_TZ
    r = ozo.SCALE_CS if rule == "CS" else ozo.SCALE_MAXEXP
    Cm, sA, sB, R = ozo.dgemm(A, B, SETS[name], q, r, want_stages=True)
    Cf, sig, tau, Rb, Cint = big.dgemm(A.tolist(), B.tolist(), name, quant, rule)
    assert sA.tolist() == sig and sB.tolist() == tau
    assert R.tolist() == Rb
    assert Cm.tolist() == Cf
    # the residue path equals the plain 128-bit product A'B' (CRT uniqueness)
    QA = ozo.quantise(0, A, sA, q)
    QB = ozo.quantise(1, B, sB, q)
    assert (ozo.crt(R, SETS[name], as_int=True) == ozo.direct(QA, QB, as_int=True)).all()
    assert ozo.direct(QA, QB, as_int=True).tolist() == Cint


@pytest.mark.parametrize("name,sub", [("S", ozo.SUB_FP8), ("S", ozo.SUB_INT8), ("E", ozo.SUB_FP8),
                                      ("A", ozo.SUB_FP8), ("A", ozo.SUB_INT8_NATIVE)])
def test_planes_reproduce_residue_products(name, sub):
    rng = np.random.default_rng(4)
    m, n, k = 6, 5, 37
    ms = ozo.modset(SETS[name])
    QA = rng.integers(-2**50, 2**50, size=(m, k))
    QB = rng.integers(-2**50, 2**50, size=(n, k))
    QA[0, :] = [(-1) ** i * (ms[i % len(ms)] // 2) for i in range(k)]   # endpoint residues
    DA, DB = ozo.residues(QA, SETS[name]), ozo.residues(QB, SETS[name])
    for i, mm in enumerate(ms):
        assert ((DA[i].astype(np.int64) - QA) % mm == 0).all()
        assert (2 * DA[i].astype(np.int64) >= -mm).all() and (2 * DA[i].astype(np.int64) < mm).all()
    PA, PB = ozo.planes(DA, SETS[name], sub), ozo.planes(DB, SETS[name], sub)
    assert PA.shape == (ozo.pstore(SETS[name], sub), m, 48) and (PA[:, :, k:] == 0).all()
    R1 = ozo.products(DA, DB, SETS[name])
    R2, worst = ozo.plane_products(PA, PB, k, SETS[name], sub)
    assert (R1 == R2).all() and worst <= (128 * 128 if sub == ozo.SUB_INT8_NATIVE else 2 * 256) * k
    want = (QA.astype(object) @ QB.astype(object).T)
    for i, mm in enumerate(ms):
        assert (R1[i].T.astype(object) == want % mm).all()


@pytest.mark.parametrize("name,sub", [("S", ozo.SUB_FP8), ("S", ozo.SUB_INT8), ("E", ozo.SUB_FP8),
                                      ("A", ozo.SUB_INT8), ("A", ozo.SUB_INT8_NATIVE)])
def test_plane_writer_equals_per_element_split_and_encode(name, sub):
    """The plane writer hoists the split and the encoding of each residue value out of its element
    loop; this holds it to the plain per-element statement of Algorithm 2: split the residue
    (Lemma 1 carry included), encode each digit, store it at [plane][line][k]."""
    rng = np.random.default_rng(11)
    ms = ozo.modset(SETS[name])
    lines, k = 3, 41
    D = np.stack([rng.integers(-(mm // 2), (mm - 1) // 2 + 1, size=(lines, k)) for mm in ms]).astype(np.int16)
    for i, mm in enumerate(ms):                      # both ends of every centred interval
        D[i, 0, 0], D[i, 0, 1] = -(mm // 2), (mm - 1) // 2
    P = ozo.planes(D, SETS[name], sub)
    plane = 0
    for i, mm in enumerate(ms):
        digits_of = (lambda d: [d]) if sub == ozo.SUB_INT8_NATIVE else (lambda d, mm=mm: ozo.split(d, mm))
        for l in range(lines):
            for kk in range(k):
                for q, dg in enumerate(digits_of(int(D[i, l, kk]))):
                    byte = ozo.e4m3_encode(dg) if sub == ozo.SUB_FP8 else dg & 0xFF
                    assert P[plane + q, l, kk] == byte
        plane += len(digits_of(0))
    assert plane == P.shape[0] and (P[:, :, k:] == 0).all()


# ----------------------------------------------------------------- P10: reduces to an exact product
def test_exact_on_small_integers():
    A, B = syn.special_operands("small_integers", 12, 10, 64)
    want = (A.astype(np.int64).astype(object) @ B.astype(np.int64).astype(object))
    for name in ("S", "E", "A"):
        for quant in (ozo.QUANT_RN, ozo.QUANT_TZ):
            for rule in (ozo.SCALE_MAXEXP, ozo.SCALE_CS):
                Cm = ozo.dgemm(A, B, SETS[name], quant, rule)
                assert (Cm == want.astype(np.float64)).all()
    assert (A @ B == want.astype(np.float64)).all()       # and so does plain FP64 here


# ----------------------------------------------------------------- P8: accuracy vs the true product
def _dd_exact(A, B):
    m, k = A.shape
    n = B.shape[1]
    out = np.empty((m, n), dtype=object)
    for i in range(m):
        for j in range(n):
            out[i, j] = sum(Fraction(A[i, t]) * Fraction(B[t, j]) for t in range(k))
    return out


def test_double_double_reference_is_accurate():
    rng = np.random.default_rng(8)
    A = np.asfortranarray(rng.standard_normal((4, 50)) * np.exp(4 * rng.standard_normal((4, 50))))
    B = np.asfortranarray(rng.standard_normal((50, 3)))
    hi, lo, ab = ozo.dd_gemm(A, B)
    ex = _dd_exact(A, B)
    exab = _dd_exact(np.abs(A), np.abs(B))
    for i in range(4):
        for j in range(3):
            err = abs(Fraction(hi[i, j]) + Fraction(lo[i, j]) - ex[i, j])
            assert err <= Fraction(2) ** -100 * exab[i, j]
            assert abs(Fraction(ab[i, j]) - exab[i, j]) <= Fraction(2) ** -50 * exab[i, j]


@pytest.mark.parametrize("cfg_id,scale", [(1, 1.0), (2, 1.0), (3, 1.0), (4, 1.0)])
def test_rn_error_bound_and_fp64_grade(cfg_id, scale):
    """Derived a-priori bound for round-to-nearest (from Eq. 1):
         |2^(s_i+t_j) (AB)_ij - c'_ij| <= 1/2 sum|a'| + 1/2 sum|b'| + k/4
       and, with the CS rule, the result is within 2 u (|A||B|)_ij of the true product
       on the well-scaled configurations."""
    cfg = syn.CONFIGS[cfg_id]
    m, n, k = 24, 20, min(cfg.k, 1024)
    A, B = syn.operands(cfg, m, n, k)
    s = SETS[cfg.sets[0]]
    Cm, sA, sB, R = ozo.dgemm(A, B, s, ozo.QUANT_RN, ozo.SCALE_CS, want_stages=True)
    QA = ozo.quantise(0, A, sA, ozo.QUANT_RN).astype(object)
    QB = ozo.quantise(1, B, sB, ozo.QUANT_RN).astype(object)
    Cp = ozo.crt(R, s, as_int=True)
    ex = _dd_exact(A, B)
    exab = _dd_exact(np.abs(A), np.abs(B))
    hi, lo, ab = ozo.dd_gemm(A, B)
    u = Fraction(2) ** -53
    worst = Fraction(0)
    for i in range(m):
        for j in range(n):
            scaled = ex[i, j] * Fraction(2) ** int(sA[i] + sB[j])
            bound = Fraction(sum(abs(v) for v in QA[i]) + sum(abs(v) for v in QB[j]), 2) + Fraction(k, 4)
            assert abs(scaled - int(Cp[i, j])) <= bound
            err = abs(Fraction(Cm[i, j]) - ex[i, j])
            worst = max(worst, err / (2 * u * exab[i, j]))
            assert abs(Fraction(hi[i, j]) + Fraction(lo[i, j]) - ex[i, j]) <= u * u * 4 * exab[i, j]
    assert worst <= 1


# ----------------------------------------------------------------- edge inputs
def test_zero_lines_subnormals_spikes_and_nonfinite():
    for kind in ("zero_lines", "subnormal", "spike"):
        A, B = syn.special_operands(kind, 8, 6, 24)
        for rule in (ozo.SCALE_MAXEXP, ozo.SCALE_CS):
            Cm, sA, sB, R = ozo.dgemm(A, B, ozo.SET_S, ozo.QUANT_RN, rule, want_stages=True)
            Cf, sig, tau, Rb, _ = big.dgemm(A.tolist(), B.tolist(), "S", "RN",
                                            "CS" if rule == ozo.SCALE_CS else "MAXEXP")
            assert sA.tolist() == sig and sB.tolist() == tau and R.tolist() == Rb
            assert Cm.tolist() == Cf
            if kind == "zero_lines":
                assert (Cm[4, :] == 0).all() and (Cm[:, 2] == 0).all() and sA[4] == 0 and sB[2] == 0
    A, B = syn.special_operands("spike", 8, 6, 24)
    A[2, 5] = np.inf
    B[7, 1] = np.nan
    Cm, sA, sB, _ = ozo.dgemm(A, B, want_stages=True)
    assert sA[2] == ozo.NONFINITE_SHIFT and sB[1] == ozo.NONFINITE_SHIFT
    assert np.isnan(Cm[2, :]).all() and np.isnan(Cm[:, 1]).all()
    mask = np.ones_like(Cm, dtype=bool)
    mask[2, :] = False
    mask[:, 1] = False
    assert np.isfinite(Cm[mask]).all()


def test_update_form_and_empty_shapes():
    cfg = syn.CONFIGS[3]
    A, B, C0 = syn.operands(cfg, 16, 12, 32, want_c=True)
    P = ozo.dgemm(A, B, ozo.SET_E)
    Cm = ozo.dgemm(A, B, ozo.SET_E, alpha=-1.0, beta=1.0, C0=C0)
    assert (Cm == C0 - P).all()
    Z = ozo.dgemm(np.zeros((3, 0), order="F"), np.zeros((0, 2), order="F"))
    assert Z.shape == (3, 2) and (Z == 0).all()
    assert ozo.dgemm(np.zeros((0, 4), order="F"), np.zeros((4, 2), order="F")).shape == (0, 2)
