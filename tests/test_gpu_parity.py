"""GPU parity: every stage entry point and the whole oz_dgemm, through the C-ABI, against the
CPU oracle on the same seeded inputs.  Integer outputs (shifts, plane bytes, residues) must be
bit-exact; FP64 outputs within 2 * 2^-53 * (|A||B|)_ij of the oracle and of a double-double GEMM."""
import numpy as np
import pytest

import synth_inputs as syn
from oracle import oz_oracle as ozo

pytestmark = pytest.mark.gpu

U = 2.0 ** -53
OSET = {"S": ozo.SET_S, "E": ozo.SET_E, "A": ozo.SET_A}
OSUB = {"fp8": ozo.SUB_FP8, "int8": ozo.SUB_INT8, "int8n": ozo.SUB_INT8_NATIVE}


def _oracle_route(sub, quant, rule):
    return (OSUB[sub],
            ozo.QUANT_RN if quant == "RN" else ozo.QUANT_TZ,
            ozo.SCALE_CS if rule == "CS" else ozo.SCALE_MAXEXP)


def _oracle_deconstruct(side, X, set_name, sub, quant, rule):
    osub, oq, orule = _oracle_route(sub, quant, rule)
    k = X.shape[1] if side == 0 else X.shape[0]
    tA, tB = ozo.budget_maxexp(OSET[set_name], max(k, 1))
    sh = ozo.shifts(side, X, OSET[set_name], orule, tA if side == 0 else tB)
    Q = ozo.quantise(side, X, sh, oq)
    D = ozo.residues(Q, OSET[set_name])
    return ozo.planes(D, OSET[set_name], osub), sh, D


# ------------------------------------------------------------------ deconstruction (a1-a4)
@pytest.mark.parametrize("side", [0, 1])
@pytest.mark.parametrize("lines,k,dist", [(256, 256, "uniform"), (37, 129, "lognormal:2.0"),
                                          (130, 1000, "normal"), (1, 1, "uniform"), (5, 17, "lognormal:0.5"),
                                          (67, 4101, "lognormal:2.0"), (300, 16, "uniform"),
                                          # too long or too large for the one-kernel deconstruction: the three-pass kernels
                                          (40, 7001, "normal"), (9, 30011, "lognormal:0.5"), (2100, 2100, "normal")])
@pytest.mark.parametrize("set_name,sub,quant,rule", [("S", "fp8", "RN", "CS"), ("S", "int8", "TZ", "MAXEXP"),
                                                     ("E", "fp8", "TZ", "CS"), ("E", "int8", "RN", "MAXEXP"),
                                                     ("A", "int8n", "RN", "CS"), ("A", "fp8", "TZ", "MAXEXP")])
def test_deconstruct_bit_exact(side, lines, k, dist, set_name, sub, quant, rule):
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(100 + lines + k)
    X = syn._draw(rng, lines, k, dist) if side == 0 else syn._draw(rng, k, lines, dist)
    P, sh, st = gh.deconstruct(side, X, set_name, gh.route(sub, quant, rule))
    Po, sho, _ = _oracle_deconstruct(side, X, set_name, sub, quant, rule)
    assert st == 0
    assert (sh == sho).all()
    assert P.shape == Po.shape and (P == Po).all()


@pytest.mark.parametrize("sub", ["fp8", "int8"])
@pytest.mark.parametrize("set_name,lines,k", [("S", 130, 1000), ("E", 67, 4101), ("A", 37, 129), ("S", 5, 4097)])
def test_merged_schedule_stages_bit_exact(set_name, lines, k, sub):
    """Merged accumulators.  FP8: the A operand carries the pre-scaled -16*d1 planes and B is unchanged.
    INT8: A carries -d0 and 4*d1, B carries 4*e1.  The two-accumulator GEMM gives the same residues."""
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(lines + k)
    A = syn._draw(rng, lines, k, "lognormal:0.5")
    B = syn._draw(rng, k, 150, "normal")
    rt = gh.route(sub, "RN", "CS", acc="merged")
    osub = OSUB[sub]
    PA, shA, st = gh.deconstruct(0, A, set_name, rt)
    PB, shB, st2 = gh.deconstruct(1, B, set_name, rt)
    _, shAo, DA = _oracle_deconstruct(0, A, set_name, sub, "RN", "CS")
    _, shBo, DB = _oracle_deconstruct(1, B, set_name, sub, "RN", "CS")
    PAo = ozo.planes_merged(0, DA, OSET[set_name], substrate=osub)
    PBo = ozo.planes_merged(1, DB, OSET[set_name], substrate=osub)
    assert st == 0 and st2 == 0 and (shA == shAo).all() and (shB == shBo).all()
    assert PA.shape == PAo.shape and (PA == PAo).all() and (PB == PBo).all()
    R, st3 = gh.residue_gemm(PA, PB, k, set_name, rt)
    assert st3 == 0 and (R == ozo.products(DA, DB, OSET[set_name])).all()


def test_merged_schedule_limits():
    import torch
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    # the re-scaled planes take the places of the plain ones: counts as in the paper's table
    assert oz.oz_plane_count_side(oz.OZ_SET_S, oz.OZ_ACC_MERGED, 0) == 30
    assert oz.oz_plane_count_side(oz.OZ_SET_S, oz.OZ_ACC_MERGED, 1) == 30
    assert oz.oz_plane_count_side(oz.OZ_SET_E, oz.OZ_ACC_MERGED, 0) == 33
    assert oz.oz_plane_count_side(oz.OZ_SET_S, oz.OZ_ACC_MERGED | oz.OZ_SUB_INT8, 0) == 30
    assert oz.oz_plane_count_side(oz.OZ_SET_S, oz.OZ_ACC_MERGED | oz.OZ_SUB_INT8, 1) == 30
    # one plane per modulus leaves nothing to merge
    assert oz.oz_plane_count_side(oz.OZ_SET_A, oz.OZ_ACC_MERGED | oz.OZ_SUB_INT8_NATIVE, 0) == 0


@pytest.mark.parametrize("set_name,k", [("S", 1100), ("S", 29700), ("S", 29900), ("E", 33000)])
def test_merged_schedule_on_int8_with_extreme_digits(set_name, k):
    """INT8 merged schedule at the edges of its host-side range checks: the largest residues everywhere
    (term 4292 on the 1089 modulus), k on either side of 29 774, where 15 * 4292 k + 16 * 484 k leaves
    INT32 and the accumulators are reduced before they are weighted, and past the FP32 depth."""
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(k)
    m, n = 70, 140
    _, DA = _random_planes(rng, set_name, "int8", m, k, extreme=True)
    _, DB = _random_planes(rng, set_name, "int8", n, k, extreme=True)
    top = 0
    for i, mod in enumerate(ozo.modset(OSET[set_name])):
        if len(ozo.split(0, mod)) == 2:      # square modulus: no merged accumulator
            continue
        # the residue whose own square gives the largest merged term 16 d1^2 - d0^2
        term = lambda d: 16 * ozo.split(d, mod)[1] ** 2 - ozo.split(d, mod)[0] ** 2
        d = max(range(-(mod // 2), (mod - 1) // 2 + 1), key=term)
        top = max(top, term(d))
        DA[i, :8, :] = DB[i, :8, :] = d
        if -(mod // 2) <= -d <= (mod - 1) // 2:
            DA[i, 8:16, :] = -d
    assert top > (4000 if set_name == "S" else 900)       # 9-bit tail of S; byte moduli
    PA = ozo.planes_merged(0, DA, OSET[set_name], substrate=ozo.SUB_INT8)
    PB = ozo.planes_merged(1, DB, OSET[set_name], substrate=ozo.SUB_INT8)
    want, worst = ozo.plane_products_merged(PA, PB, k, OSET[set_name], substrate=ozo.SUB_INT8)
    assert (want == ozo.products(DA, DB, OSET[set_name])).all() and worst >= top * k
    R, st = gh.residue_gemm(PA, PB, k, set_name, gh.route("int8", acc="merged"))
    assert st == 0 and (R == want).all()


@pytest.mark.parametrize("set_name,k", [("S", 4224), ("S", 8321), ("S", 12289), ("E", 16640), ("A", 16640)])
def test_merged_schedule_segments_long_k(set_name, k):
    """k beyond the exact depth of one merged accumulator (4097 / 15420): the kernel cuts K into
    segments, each with its own accumulator; extreme digits make a single accumulator overflow 2^24."""
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(k)
    m, n = 70, 140
    _, DA = _random_planes(rng, set_name, "fp8", m, k, extreme=True)
    _, DB = _random_planes(rng, set_name, "fp8", n, k, extreme=True)
    for i, mod in enumerate(ozo.modset(OSET[set_name])):
        DA[i, :8, :] = DB[i, :8, :] = (mod - 1) // 2      # largest residue: merged term 4095 (1088 on bytes)
    PA, PB = ozo.planes_merged(0, DA, OSET[set_name]), ozo.planes_merged(1, DB, OSET[set_name])
    _, worst = ozo.plane_products_merged(PA, PB, k, OSET[set_name])
    assert worst >= 2 ** 24            # one accumulator over all of K would not be exact
    R, st = gh.residue_gemm(PA, PB, k, set_name, gh.route("fp8", acc="merged"))
    assert st == 0 and (R == ozo.products(DA, DB, OSET[set_name])).all()


def test_merged_accumulator_exact_at_its_depth():
    """k = 4097 on set S with the largest digits: the merged accumulator reaches 4095 * 4097 < 2^24."""
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(4097)
    m, n, k = 70, 140, 4097
    _, DA = _random_planes(rng, "S", "fp8", m, k, extreme=True)
    _, DB = _random_planes(rng, "S", "fp8", n, k, extreme=True)
    DA[:, :8, :] = DA[:, :1, :1]
    DB[:, :8, :] = DB[:, :1, :1]
    PA, PB = ozo.planes_merged(0, DA, ozo.SET_S), ozo.planes_merged(1, DB, ozo.SET_S)
    want, worst = ozo.plane_products_merged(PA, PB, k, ozo.SET_S)
    assert worst < 2 ** 24 and worst > 0.5 * 4095 * k and (want == ozo.products(DA, DB, ozo.SET_S)).all()
    R, st = gh.residue_gemm(PA, PB, k, "S", gh.route("fp8", acc="merged"))
    assert st == 0 and (R == want).all()


@pytest.mark.parametrize("kind", ["zero_lines", "subnormal", "spike", "small_integers"])
@pytest.mark.parametrize("rule", ["CS", "MAXEXP"])
def test_deconstruct_edge_inputs(kind, rule):
    import tests.gpu_helpers as gh
    A, B = syn.special_operands(kind, 40, 24, 100)
    for side, X in ((0, A), (1, B)):
        P, sh, st = gh.deconstruct(side, X, "S", gh.route("fp8", "RN", rule))
        Po, sho, _ = _oracle_deconstruct(side, X, "S", "fp8", "RN", rule)
        assert st == 0 and (sh == sho).all() and (P == Po).all()


def test_deconstruct_nonfinite_contract():
    import tests.gpu_helpers as gh
    import paper_2609_09095_b200 as oz
    A, _ = syn.special_operands("spike", 16, 8, 40)
    A[3, 7] = np.inf
    A[9, 0] = np.nan
    P, sh, st = gh.deconstruct(0, A, "S", gh.route())
    Po, sho, _ = _oracle_deconstruct(0, A, "S", "fp8", "RN", "CS")
    assert st == oz.OZ_ERR_NONFINITE_INPUT
    assert sh[3] == oz.OZ_NONFINITE_SHIFT and sh[9] == oz.OZ_NONFINITE_SHIFT
    assert (sh == sho).all() and (P == Po).all()
    assert gh.sync_status() == 0   # the status word is cleared by the query


# ------------------------------------------------------------------ residue GEMMs (a5-a6)
def _random_planes(rng, set_name, sub, lines, k, extreme=False):
    """Stored planes of random centred residues (or of the residues with the largest digits)."""
    ms = ozo.modset(OSET[set_name])
    D = np.zeros((len(ms), lines, k), dtype=np.int16)
    for i, m in enumerate(ms):
        lo, hi = -(m // 2), (m - 1) // 2
        if extreme:
            if sub == "int8n":
                cand = [lo, hi, lo + 1, hi - 1]
            else:
                cand = sorted(range(lo, hi + 1), key=lambda d: -max(abs(v) for v in ozo.split(d, m)))[:4]
            D[i] = rng.choice(cand, size=(lines, k))
        else:
            D[i] = rng.integers(lo, hi + 1, size=(lines, k))
    return ozo.planes(D, OSET[set_name], OSUB[sub]), D


@pytest.mark.parametrize("m,n,k", [(128, 256, 128), (256, 512, 384), (200, 300, 200), (1, 1, 1),
                                   (129, 257, 130), (3, 700, 17), (520, 40, 1000)])
@pytest.mark.parametrize("set_name,sub", [("S", "fp8"), ("S", "int8"), ("E", "fp8"), ("A", "int8n"), ("A", "fp8")])
def test_residue_gemm_bit_exact(m, n, k, set_name, sub):
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(m * 7 + n * 3 + k)
    PA, DA = _random_planes(rng, set_name, sub, m, k)
    PB, DB = _random_planes(rng, set_name, sub, n, k)
    R, st = gh.residue_gemm(PA, PB, k, set_name, gh.route(sub))
    want = ozo.products(DA, DB, OSET[set_name])
    assert st == 0
    assert (R == want).all()


@pytest.mark.parametrize("k", [4096, 5003, 32768])
@pytest.mark.parametrize("sub", ["fp8", "int8", "int8n"])
def test_accumulation_is_exact_at_depth(k, sub):
    """Planes made of the largest digits only: accumulators reach k*484 (non-square) and
    k*512 (square, two K-loops in one accumulator) -- up to 2^24 at k = 32768."""
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(k)
    m, n = (130, 260) if k < 30000 else (40, 24)
    set_name = "A" if sub == "int8n" else "S"
    PA, DA = _random_planes(rng, set_name, sub, m, k, extreme=True)
    PB, DB = _random_planes(rng, set_name, sub, n, k, extreme=True)
    # make some rows all-equal so that terms do not cancel
    PA[:, :8, :k] = PA[:, :1, :1]
    PB[:, :8, :k] = PB[:, :1, :1]
    want, worst = ozo.plane_products(PA, PB, k, OSET[set_name], OSUB[sub])
    assert worst > 0.9 * 256 * k
    R, st = gh.residue_gemm(PA, PB, k, set_name, gh.route(sub))
    assert st == 0
    assert (R == want).all()


@pytest.mark.parametrize("set_name,sub", [("S", "fp8"), ("A", "int8n"), ("A", "fp8"), ("E", "int8")])
@pytest.mark.parametrize("m,ldr", [(200, 208), (130, 144), (64, 80), (300, 301)])
def test_residue_gemm_padded_rows(m, ldr, set_name, sub):
    """Leading dimension larger than m: aligned paddings take the vector stores with a ragged last
    tile, an odd one the element-wise path; the padding itself must stay untouched."""
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(m + ldr)
    n, k = 70, 160
    PA, DA = _random_planes(rng, set_name, sub, m, k)
    PB, DB = _random_planes(rng, set_name, sub, n, k)
    import torch
    import paper_2609_09095_b200 as oz
    r = len(ozo.modset(OSET[set_name]))
    tdt, _ = gh.residue_dtype(set_name)
    fill = 0xFF if tdt == torch.uint8 else 0xFFFF
    R = torch.full((r, n, ldr), fill, dtype=tdt, device="cuda")
    dA, dB = torch.from_numpy(PA).cuda(), torch.from_numpy(PB).cuda()
    oz.check(oz.oz_residue_gemm(m, n, k, dA, m * PA.shape[2], PA.shape[2], dB, n * PB.shape[2], PB.shape[2],
                                gh.SETS[set_name], gh.route(sub), R, ldr, n * ldr), "oz_residue_gemm")
    assert gh.sync_status() == 0
    Rh = R.cpu().numpy()
    assert (Rh[:, :, :m] == ozo.products(DA, DB, OSET[set_name])).all()
    assert (Rh[:, :, m:] == fill).all()


@pytest.mark.parametrize("k,set_name,sub,acc", [(40000, "S", "fp8", "separate"), (70001, "E", "fp8", "separate"),
                                                (40000, "S", "fp8", "merged"), (140000, "A", "int8n", None),
                                                (66000, "S", "int8", None), (65536, "A", "int8n", None),
                                                (65537, "A", "int8n", None)])
def test_split_k_beyond_one_accumulator(k, set_name, sub, acc):
    """k beyond the exact depth of one accumulator (32768 in FP32, 131071 for native INT8 residues): the
    kernel cuts K into segments and adds their reduced results modulo m.  Largest digits, constant
    rows: a single accumulator over all of K would overflow.  k = 65536 / 65537 straddle the largest
    depth served by the native route's direct drain (accumulators up to 2^30 in magnitude)."""
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(k)
    m, n = 40, 24
    _, DA = _random_planes(rng, set_name, sub, m, k, extreme=True)
    _, DB = _random_planes(rng, set_name, sub, n, k, extreme=True)
    DA[:, :8, :] = DA[:, :1, :1]
    DB[:, :8, :] = DB[:, :1, :1]
    if acc == "merged":
        PA, PB = ozo.planes_merged(0, DA, OSET[set_name]), ozo.planes_merged(1, DB, OSET[set_name])
    else:
        PA, PB = ozo.planes(DA, OSET[set_name], OSUB[sub]), ozo.planes(DB, OSET[set_name], OSUB[sub])
    R, st = gh.residue_gemm(PA, PB, k, set_name, gh.route(sub, acc=acc))
    assert st == 0 and (R == ozo.products(DA, DB, OSET[set_name])).all()


def test_dgemm_long_k():
    """The whole method at k = 33000 > 32768 (shifts from the whole k, split-K inside the GEMM)."""
    import tests.gpu_helpers as gh
    A, B = syn.operands(syn.CONFIGS[2], 48, 1030, 33000)
    for set_name, sub in (("S", "fp8"), ("A", "int8n")):
        got, st = gh.dgemm(A, B, set_name, gh.route(sub))
        want = ozo.dgemm(A, B, OSET[set_name])
        assert st == 0
        _check_against_oracle_and_dd(A, B, got, want)


# ------------------------------------------------------------------ reconstruction (a7)
@pytest.mark.parametrize("set_name", ["S", "E", "A"])
@pytest.mark.parametrize("m,n,ldr", [(256, 64, None), (1, 1, None), (7, 5, None), (130, 3, None), (258, 9, 272),
                                     (131, 4, 132), (5, 3, 8), (259, 2, 261)])
def test_reconstruct_bit_exact(set_name, m, n, ldr):
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(m + n)
    ms = ozo.modset(OSET[set_name])
    M = int(np.prod([int(v) for v in ms], dtype=object))
    R = np.stack([rng.integers(0, mm, size=(n, m)) for mm in ms]).astype(np.uint16)
    # boundary integers: -M/2, M/2-1, 0, +-1, and values whose conversion to double is a tie
    special = [-(M // 2), M // 2 - 1, 0, 1, -1, 2**53 + 1, 2**54 + 2, -(2**60 + 2**7), 2**100 + 2**47,
               2**100 + 3 * 2**47, -(2**100 + 2**47), 2**110 + 2**57 + 1]
    flat = R.reshape(len(ms), -1)
    for t, x in enumerate(special[: flat.shape[1]]):
        flat[:, t] = [x % mm for mm in ms]
    R = flat.reshape(len(ms), n, m)
    sA = rng.integers(-60, 120, size=m).astype(np.int32)
    sB = rng.integers(-60, 120, size=n).astype(np.int32)
    C0 = np.asfortranarray(rng.standard_normal((m, n)))
    CI = ozo.crt(R, OSET[set_name])
    for alpha, beta in ((1.0, 0.0), (-1.0, 1.0), (-1.0, 0.0), (1.0, 1.0)):
        got, st = gh.reconstruct(R, sA, sB, set_name, alpha, beta, C0, ldr=ldr)
        want = ozo.output(CI, sA, sB, alpha, beta, C0)
        assert st == 0
        assert (got == want).all()
    # any representative below 2 m_i that fits the element type gives the same integer
    top = 255 if set_name == "A" else 65535
    R2 = R.astype(np.int64)
    for i, mm in enumerate(ms):
        bump = (rng.integers(0, 2, size=R2[i].shape) == 1) & (R2[i] + mm <= top)
        R2[i] = R2[i] + bump * mm
    assert R.size < 64 or (R2 != R).any()
    got, st = gh.reconstruct(R2.astype(np.uint16), sA, sB, set_name, 1.0, 0.0, None, ldr=ldr)
    assert st == 0 and (got == ozo.output(CI, sA, sB, 1.0, 0.0, None)).all()


# ------------------------------------------------------------------ whole method
def _check_against_oracle_and_dd(A, B, got, want, C0=None, alpha=1.0, strict_dd=True):
    hi, lo, ab = ozo.dd_gemm(A, B)
    tol = 2 * U * ab
    assert (np.abs(got - want) <= tol).all()
    ref = alpha * hi if C0 is None else C0 + alpha * hi
    err_dd = np.abs(got - ref) / np.maximum(tol + (0 if C0 is None else U * np.abs(ref)), 1e-300)
    if strict_dd:
        assert err_dd.max() <= 1.0
    return float(err_dd.max())


@pytest.mark.parametrize("cfg_id,m,n,k,sets", [(1, 256, 256, 256, ("S",)), (2, 300, 520, 4096, ("S",)),
                                               (3, 384, 512, 1024, ("E", "S")), (4, 700, 128, 4096, ("S",)),
                                               (5, 263, 301, 5003, ("S",)), (3, 300, 260, 1024, ("A",))])
def test_dgemm_configs_cut_down(cfg_id, m, n, k, sets):
    import tests.gpu_helpers as gh
    cfg = syn.CONFIGS[cfg_id]
    A, B, C0 = syn.operands(cfg, m, n, k, want_c=True)
    for set_name in sets:
        for sub in (("int8n", "fp8") if set_name == "A" else cfg.substrates):
            rt = gh.route(sub, "RN", "CS")
            use_c0 = C0 if cfg.beta else None
            got, st = gh.dgemm(A, B, set_name, rt, cfg.alpha, cfg.beta, use_c0)
            want = ozo.dgemm(A, B, OSET[set_name], ozo.QUANT_RN, ozo.SCALE_CS, cfg.alpha, cfg.beta, use_c0)
            assert st == 0
            assert (got == want).all()      # the CRT is exact on both sides: bit-identical FP64
            # cfg 5 (very wide exponent spread) is beyond what 12 moduli can deliver against the true product
            _check_against_oracle_and_dd(A, B, got, want, use_c0, cfg.alpha, strict_dd=(cfg_id != 5))


@pytest.mark.parametrize("quant,rule,acc", [("TZ", "MAXEXP", None), ("RN", "MAXEXP", "separate"),
                                            ("TZ", "CS", "merged"), ("RN", "CS", "separate")])
def test_dgemm_variants(quant, rule, acc):
    import tests.gpu_helpers as gh
    A, B = syn.operands(syn.CONFIGS[1], 130, 70, 200)
    got, st = gh.dgemm(A, B, "S", gh.route("fp8", quant, rule, acc))
    _, oq, orule = _oracle_route("fp8", quant, rule)
    want = ozo.dgemm(A, B, ozo.SET_S, oq, orule)
    assert st == 0 and (got == want).all()


@pytest.mark.parametrize("seed", range(24))
def test_dgemm_random_shapes(seed):
    """Seeded random shapes, routes and scalars: ragged tiles in every dimension, every modulus set and
    substrate, both quantisers and scale rules, alpha / beta in their four combinations."""
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(9000 + seed)
    m, n = int(rng.integers(1, 700)), int(rng.integers(1, 700))
    k = int(rng.integers(1, 640)) if seed % 6 else int(rng.integers(4000, 9000))
    if seed % 6 == 0:
        m, n = min(m, 150), min(n, 150) + (1024 if seed % 12 == 0 else 0)
    set_name, sub = [("S", "fp8"), ("S", "int8"), ("E", "fp8"), ("E", "int8"), ("A", "int8n"), ("A", "fp8"),
                     ("A", "int8")][seed % 7]
    quant, rule = ("RN", "TZ")[int(rng.integers(2))], ("CS", "MAXEXP")[int(rng.integers(2))]
    alpha, beta = (1.0, -1.0)[int(rng.integers(2))], (0.0, 1.0)[int(rng.integers(2))]
    dist = ("uniform", "normal", "lognormal:0.5", "lognormal:2.0")[int(rng.integers(4))]
    A, B = syn._draw(rng, m, k, dist), syn._draw(rng, k, n, dist)
    C0 = np.asfortranarray(rng.standard_normal((m, n))) if beta else None
    got, st = gh.dgemm(A, B, set_name, gh.route(sub, quant, rule), alpha, beta, C0)
    _, oq, orule = _oracle_route(sub, quant, rule)
    want = ozo.dgemm(A, B, OSET[set_name], oq, orule, alpha, beta, C0)
    assert st == 0 and (got == want).all()


def test_dgemm_edge_cases():
    import tests.gpu_helpers as gh
    import paper_2609_09095_b200 as oz
    for kind in ("zero_lines", "subnormal", "spike", "small_integers"):
        A, B = syn.special_operands(kind, 33, 17, 70)
        got, st = gh.dgemm(A, B, "S", gh.route())
        assert st == 0 and (got == ozo.dgemm(A, B)).all()
    A, B = syn.special_operands("small_integers", 33, 17, 70)
    assert (gh.dgemm(A, B, "E", gh.route())[0] == A @ B).all()          # exact integer product
    A[4, 4] = np.nan
    got, st = gh.dgemm(A, B, "S", gh.route())
    want = ozo.dgemm(A, B)
    assert st == oz.OZ_ERR_NONFINITE_INPUT
    assert np.isnan(got[4, :]).all() and (np.isnan(got) == np.isnan(want)).all()
    assert (got[~np.isnan(got)] == want[~np.isnan(want)]).all()
    # k = 0: C = 0 (beta 0) or unchanged (beta 1); empty m or n: nothing to do
    Z, st = gh.dgemm(np.zeros((5, 0), order="F"), np.zeros((0, 3), order="F"), "S", gh.route())
    assert st == 0 and (Z == 0).all()


def test_argument_errors_are_reported_on_the_host():
    import torch
    import paper_2609_09095_b200 as oz
    t = torch.zeros(64, dtype=torch.float64, device="cuda")
    assert oz.oz_dgemm(4, 4, 4, t, 2, t, 4, t, 4) == oz.OZ_ERR_INVALID_ARG          # lda < m
    assert oz.oz_dgemm(4, 4, oz.OZ_K_MAX + 1, t, 4, t, oz.OZ_K_MAX + 1, t, 4) == oz.OZ_ERR_UNSUPPORTED
    assert oz.oz_dgemm_ex(4, 4, 4, 2.0, t, 4, t, 4, 0.0, t, 4) == oz.OZ_ERR_UNSUPPORTED
    assert oz.oz_dgemm(4, 4, 4, t, 4, t, 4, t, 4, 5, 0) == oz.OZ_ERR_INVALID_ARG        # unknown set
    assert oz.oz_dgemm(4, 4, 4, t, 4, t, 4, t, 4, 0, 0x003) == oz.OZ_ERR_INVALID_ARG    # two substrates
    oz.oz_set_workspace(None)
    assert oz.oz_dgemm(4, 4, 4, t, 4, t, 4, t, 4) == oz.OZ_ERR_WORKSPACE
    assert oz.oz_dgemm(0, 4, 4, t, 4, t, 4, t, 4) == oz.OZ_OK


# ------------------------------------------------------------------ host-buffer entry point
@pytest.mark.parametrize("m,n,k,alpha,beta,set_name,sub", [
    (200, 300, 260, 1.0, 0.0, "S", "fp8"),          # small: one sequential upload / download
    (4096, 4224, 96, -1.0, 1.0, "S", "fp8"),        # 138 MB of C: two column panels on side streams
    (4100, 8200, 40, 1.0, 0.0, "A", "int8n"),       # four panels, ragged, no upload of C
    (3000, 11200, 24, 1.0, 1.0, "E", "fp8"),        # four panels of unequal width
    (260, 300, 520, -1.0, 1.0, "S", "int8"),        # INT8 digit planes: merged schedule on both operands
])
def test_dgemm_host_buffers(m, n, k, alpha, beta, set_name, sub):
    """oz_dgemm_host (pinned host operands, copies inside, C in column panels when it is large) against
    the oracle on sampled rows and columns and bit for bit against the device-pointer entry point."""
    import torch
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(m + n + k)
    A = np.asfortranarray(rng.uniform(-1, 1, size=(m, k)))
    B = np.asfortranarray(rng.standard_normal((k, n)))
    C0 = np.asfortranarray(rng.standard_normal((m, n)))
    lda, ldb, ldc = m + 3, k + 1, m + 5
    hA = torch.zeros((k, lda), dtype=torch.float64).pin_memory()
    hB = torch.zeros((n, ldb), dtype=torch.float64).pin_memory()
    hC = torch.full((n, ldc), 5.0, dtype=torch.float64).pin_memory()
    hA[:, :m] = torch.from_numpy(np.ascontiguousarray(A.T))
    hB[:, :k] = torch.from_numpy(np.ascontiguousarray(B.T))
    hC[:, :m] = torch.from_numpy(np.ascontiguousarray(C0.T))
    rt = gh.route(sub)
    need = oz.oz_workspace_bytes(m, n, k, gh.SETS[set_name], rt) + 8 * (m * k + k * n + m * n) + 1024
    gh.ensure_workspace(need)
    for _ in range(2):                                  # twice: the side streams and events are reused
        hC[:, :m] = torch.from_numpy(np.ascontiguousarray(C0.T))
        oz.check(oz.oz_dgemm_host(m, n, k, alpha, hA, lda, hB, ldb, beta, hC, ldc, gh.SETS[set_name], rt),
                 "oz_dgemm_host")
        assert gh.sync_status() == 0
        got = hC.numpy().T
        assert (got[m:, :] == 5.0).all()                # rows beyond m of the host array are untouched
        dev, st = gh.dgemm(A, B, set_name, rt, alpha, beta, C0 if beta else None)
        assert st == 0 and (got[:m, :] == dev).all()
    rows = np.unique(rng.integers(0, m, size=48))
    cols = np.unique(np.concatenate([rng.integers(0, n, size=48), [0, n - 1, n // 2 - 1, n // 2]]))
    want = ozo.dgemm(np.asfortranarray(A[rows, :]), np.asfortranarray(B[:, cols]), OSET[set_name], ozo.QUANT_RN,
                     ozo.SCALE_CS, alpha, beta, np.asfortranarray(C0[np.ix_(rows, cols)]) if beta else None)
    assert (got[np.ix_(rows, cols)] == want).all()


def _stalled_then_normal(n):
    """Child process of test_bounded_waits_time_out_cleanly: the library was loaded with
    OZ_TEST_STALL_PRODUCER=once, so its first residue-GEMM launch loads nothing."""
    import time
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(5)
    m, k = 300, 256
    PA, DA = _random_planes(rng, "S", "fp8", m, k)
    PB, DB = _random_planes(rng, "S", "fp8", n, k)
    t0 = time.time()
    R, st = gh.residue_gemm(PA, PB, k, "S", gh.route("fp8"))
    elapsed = time.time() - t0
    assert st == oz.OZ_ERR_TIMEOUT, st
    assert 1.5 < elapsed < 120.0, elapsed
    R, st = gh.residue_gemm(PA, PB, k, "S", gh.route("fp8"))
    assert st == 0 and (R == ozo.products(DA, DB, OSET["S"])).all()
    print("stalled-then-normal ok")


@pytest.mark.parametrize("n", [520, 512])        # single-CTA variant, CTA-pair variant
def test_bounded_waits_time_out_cleanly(n):
    """No wait in the GEMM kernel is unbounded: with the producer told to load nothing (a test hook that
    the library reads from the environment when it is loaded, hence the child process), every role's
    wait runs into its 2 s limit, the kernel records OZ_ERR_TIMEOUT, frees its tensor memory and
    returns; the context stays usable and the next call is correct."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, OZ_TEST_STALL_PRODUCER="once")
    out = subprocess.run([sys.executable, "-c",
                          f"import tests.test_gpu_parity as t; t._stalled_then_normal({n})"],
                         cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "stalled-then-normal ok" in out.stdout, out.stdout + out.stderr


def test_whole_method_rounding_boundaries():
    """The reconstruction of the whole-method calls (tile-ordered residues) at the boundaries of its one
    rounding: with k = 1 the integer c' is the product of two chosen integers times a power of two, so
    operands can be built whose products sit exactly on ties (2^53 + 1 and friends: round to even, both
    ways), one unit either side of a tie, just below and at powers of two, and far beyond 53 bits.
    Every output must equal the oracle's (and Python's correctly rounded product), with the FP64 form of
    the reconstruction and with the one hosted on the INT8 tensor pipe."""
    import tests.gpu_helpers as gh
    from fractions import Fraction
    # factor pairs of integers of 54..60 bits with interesting low bits
    targets = []
    for base in (2 ** 53, 2 ** 54, 2 ** 57, 3 * 2 ** 52):
        for delta in (-3, -2, -1, 0, 1, 2, 3, 5, 7):
            targets.append(base + delta)
    targets += [2 ** 53 + 2 ** 20 + 1, (2 ** 53 + 1) * 3, (2 ** 53 + 3) * 5, 2 ** 60 - 1, 2 ** 60 + 2 ** 7]
    rows, cols = [], []
    for t in targets:                      # t = p * q with p small and odd if possible, else p = 1
        p = next((d for d in (3, 5, 7, 9, 11, 13, 107, 321) if t % d == 0), 1)
        q = t // p
        if q < 2 ** 53:                    # both factors must be exact doubles
            rows.append(float(p))
            cols.append(float(q))
    A = np.asfortranarray(np.array(rows + [-r for r in rows]).reshape(-1, 1))
    B = np.asfortranarray(np.array(cols).reshape(1, -1))
    exact = [[Fraction(a) * Fraction(b) for b in B[0]] for a in A[:, 0]]
    for set_name, sub, recon in (("S", "fp8", None), ("E", "int8", None), ("A", "int8n", None),
                                 ("S", "fp8", "tensor"), ("E", "fp8", "tensor"), ("A", "int8n", "tensor")):
        for quant in ("RN", "TZ"):
            got, st = gh.dgemm(A, B, set_name, gh.route(sub, quant, "CS", recon=recon))
            oq = ozo.QUANT_RN if quant == "RN" else ozo.QUANT_TZ
            want = ozo.dgemm(A, B, OSET[set_name], oq, ozo.SCALE_CS)
            assert st == 0 and (got == want).all()
            # integers this small are quantised exactly, so the result is the correctly rounded product
            assert got.tolist() == [[float(v) for v in row] for row in exact]


@pytest.mark.parametrize("set_name,sub,m,n,k,alpha,beta", [
    ("S", "fp8", 700, 515, 384, 1.0, 0.0),          # several tiles, ragged, CTA-pair tiles
    ("S", "int8", 257, 129, 1000, -1.0, 1.0),
    ("E", "fp8", 300, 260, 1024, -1.0, 1.0),        # 13 moduli: all sixteen byte positions in use
    ("A", "int8n", 520, 300, 260, 1.0, 1.0),        # byte residues: four outputs per thread
    ("A", "fp8", 64, 1030, 96, 1.0, 0.0),
    ("S", "fp8", 1, 1, 1, 1.0, 0.0),
])
def test_reconstruction_hosted_on_the_tensor_pipe(set_name, sub, m, n, k, alpha, beta):
    """OZ_RECON_TENSOR (Algorithm 3, the INT8-tensor branch of the reconstruction): the CRT
    recombination as one unsigned 8-bit tcgen05 product per 128 outputs and an integer tail.  Bit for
    bit the oracle's result, like the FP64 form, also on lines of zeros, spikes and non-finite input."""
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(m + 3 * n + 7 * k)
    A, B = syn._draw(rng, m, k, "lognormal:0.5"), syn._draw(rng, k, n, "normal")
    C0 = np.asfortranarray(rng.standard_normal((m, n)))
    if m > 8 and n > 8:
        A[3, :] = 0.0
        B[:, 5] = 0.0
        A[1, k // 2] = 7.0e30
    rt = gh.route(sub, "RN", "CS", recon="tensor")
    got, st = gh.dgemm(A, B, set_name, rt, alpha, beta, C0 if beta else None)
    want = ozo.dgemm(A, B, OSET[set_name], ozo.QUANT_RN, ozo.SCALE_CS, alpha, beta, C0 if beta else None)
    assert st == 0 and (got == want).all()
    plain, st = gh.dgemm(A, B, set_name, gh.route(sub, "RN", "CS"), alpha, beta, C0 if beta else None)
    assert st == 0 and (plain == got).all()
    if m > 8 and n > 8:
        A[2, 0] = np.nan
        got, st = gh.dgemm(A, B, set_name, rt, alpha, beta, C0 if beta else None)
        want = ozo.dgemm(A, B, OSET[set_name], ozo.QUANT_RN, ozo.SCALE_CS, alpha, beta, C0 if beta else None)
        assert st == oz.OZ_ERR_NONFINITE_INPUT
        assert (np.isnan(got) == np.isnan(want)).all() and (got[~np.isnan(want)] == want[~np.isnan(want)]).all()
