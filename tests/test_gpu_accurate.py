"""Accurate mode (Sec. 2 "The FP8 variant": one additional FP8 GEMM estimates an input magnitude
bound -- the "+1" of the 3r + 1 schedule): the shifts come from the row and column maxima of a
tensor-core product of E4M3 magnitude digits.  The whole call must be bit-identical to the oracle's
statement of the same rule, which fixes the shifts, the residues and the rounding."""
import numpy as np
import pytest

import synth_inputs as syn
from oracle import oz_oracle as ozo

pytestmark = pytest.mark.gpu

U = 2.0 ** -53
OSET = {"S": ozo.SET_S, "E": ozo.SET_E, "A": ozo.SET_A}


@pytest.mark.parametrize("set_name,sub,m,n,k,dist,quant", [
    ("S", "fp8", 300, 520, 700, "lognormal:0.5", "RN"),        # several tiles, ragged in every dimension
    ("S", "fp8", 130, 70, 5003, "lognormal:2.0", "TZ"),        # deep, wide exponent spread
    ("E", "int8", 257, 129, 260, "normal", "RN"),
    ("A", "int8n", 64, 600, 128, "uniform", "RN"),             # CTA-pair tiles
    ("S", "fp8", 1, 1, 1, "uniform", "RN"),
    ("A", "fp8", 37, 41, 16384, "uniform", "TZ"),              # the deepest supported bound product
])
def test_accurate_mode_bit_identical_to_oracle(set_name, sub, m, n, k, dist, quant):
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(m * 3 + n * 5 + k)
    A, B = syn._draw(rng, m, k, dist), syn._draw(rng, k, n, dist)
    C0 = np.asfortranarray(rng.standard_normal((m, n)))
    oq = ozo.QUANT_RN if quant == "RN" else ozo.QUANT_TZ
    for alpha, beta in ((1.0, 0.0), (-1.0, 1.0)):
        got, st = gh.dgemm(A, B, set_name, gh.route(sub, quant, "ACCURATE"), alpha, beta, C0 if beta else None)
        want = ozo.dgemm(A, B, OSET[set_name], oq, ozo.SCALE_ACCURATE, alpha, beta, C0 if beta else None)
        assert st == 0 and (got == want).all()


def test_accurate_mode_edge_inputs_and_bound_attained():
    """Zero lines, subnormal lines, single huge entries, a line with Inf/NaN, and operands whose
    magnitudes attain the bound product (every digit 32, equal signs)."""
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    for kind in ("zero_lines", "subnormal", "spike", "small_integers"):
        A, B = syn.special_operands(kind, 70, 50, 300)
        got, st = gh.dgemm(A, B, "S", gh.route("fp8", "RN", "ACCURATE"))
        want = ozo.dgemm(A, B, ozo.SET_S, ozo.QUANT_RN, ozo.SCALE_ACCURATE)
        assert st == 0 and (got == want).all(), kind
    top = float(np.nextafter(2.0, 0.0))
    A = np.asfortranarray(np.full((40, 512), top * 2.0 ** 9))
    B = np.asfortranarray(np.full((512, 33), top * 2.0 ** -3))
    A[7, :] *= -1.0
    got, st = gh.dgemm(A, B, "E", gh.route("fp8", "RN", "ACCURATE"))
    want = ozo.dgemm(A, B, ozo.SET_E, ozo.QUANT_RN, ozo.SCALE_ACCURATE)
    assert st == 0 and (got == want).all()
    A, B = syn.special_operands("spike", 20, 30, 64)
    A[4, 4] = np.nan
    B[3, 9] = np.inf
    got, st = gh.dgemm(A, B, "S", gh.route("fp8", "RN", "ACCURATE"))
    want = ozo.dgemm(A, B, ozo.SET_S, ozo.QUANT_RN, ozo.SCALE_ACCURATE)
    assert st == oz.OZ_ERR_NONFINITE_INPUT
    assert (np.isnan(got) == np.isnan(want)).all() and (got[~np.isnan(want)] == want[~np.isnan(want)]).all()


@pytest.mark.parametrize("cfg_id,m,n,k", [(1, 256, 256, 256), (2, 300, 520, 4096), (3, 384, 512, 1024),
                                          (4, 700, 128, 4096)])
def test_accurate_mode_meets_the_fp64_grade_bound(cfg_id, m, n, k):
    """On the benchmark distributions the accurate rule delivers 2u(|A||B|) against the double-double
    product, like the norm-based rule."""
    import tests.gpu_helpers as gh
    cfg = syn.CONFIGS[cfg_id]
    A, B = syn.operands(cfg, m, n, k)
    got, st = gh.dgemm(A, B, "S", gh.route("fp8", "RN", "ACCURATE"))
    hi, lo, ab = ozo.dd_gemm(A, B)
    assert st == 0 and (np.abs(got - hi) <= 2 * U * ab).all()


def test_accurate_mode_limits():
    import torch
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    rt = gh.route("fp8", "RN", "ACCURATE")
    t = torch.zeros(1 << 16, dtype=torch.float64, device="cuda")
    gh.ensure_workspace(oz.oz_workspace_bytes(2, 2, 16385, oz.OZ_SET_S, rt))
    assert oz.oz_dgemm(2, 2, 16385, t, 2, t, 16385, t, 2, oz.OZ_SET_S, rt) == oz.OZ_ERR_UNSUPPORTED
    u = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    s = torch.zeros(64, dtype=torch.int32, device="cuda")
    # the shifts of one operand depend on the other: no per-operand entry point takes the rule
    assert oz.oz_deconstruct(0, 4, 16, t, 4, oz.OZ_SET_S, rt, u, 64, 16, s, u) == oz.OZ_ERR_UNSUPPORTED
    assert oz.oz_prepare_operand(0, 4, 16, t, 4, oz.OZ_SET_S, rt, u) == oz.OZ_ERR_UNSUPPORTED


# ------------------------------------------------------------------ exponent-span check
@pytest.mark.parametrize("set_name", ["S", "E", "A"])
def test_exponent_span_status_matches_oracle(set_name):
    """Algorithm 1, "ESC check": the status of a whole-method call is OZ_ERR_RANGE exactly when the
    oracle's statement of the check flags the operands -- on the five benchmark distributions, on a
    spike, and for a single operand through the stage entry point -- and the results are untouched."""
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    sub = "int8n" if set_name == "A" else "fp8"
    cases = [syn.operands(syn.CONFIGS[c], 96, 80, kk) for c, kk in ((1, 256), (2, 1500), (3, 1024), (4, 2000), (5, 3001))]
    cases.append(syn.special_operands("spike", 40, 30, 500))
    seen = set()
    for A, B in cases:
        got, st = None, None
        m, k = A.shape
        n = B.shape[1]
        gh.ensure_workspace(oz.oz_workspace_bytes(m, n, k, gh.SETS[set_name], gh.route(sub)))
        dA, dB = gh.to_dev(A), gh.to_dev(B)
        import torch
        dC = torch.zeros((n, m), dtype=torch.float64, device="cuda")
        oz.check(oz.oz_dgemm(m, n, k, dA, m, dB, k, dC, m, gh.SETS[set_name], gh.route(sub)), "oz_dgemm")
        st = gh.sync_status(esc=True)
        flagged = ozo.esc_check(A, B, OSET[set_name])
        assert st == (oz.OZ_ERR_RANGE if flagged else 0)
        assert (gh.from_dev(dC) == ozo.dgemm(A, B, OSET[set_name])).all()
        assert gh.sync_status(esc=True) == 0                     # cleared by the query
        seen.add(flagged)
        # the other scale rules do not run the check
        oz.check(oz.oz_dgemm(m, n, k, dA, m, dB, k, dC, m, gh.SETS[set_name], gh.route(sub, "RN", "MAXEXP")), "oz_dgemm")
        assert gh.sync_status(esc=True) == 0
    assert seen == {True, False}
    # one operand through the stage entry point: the other counts as flat
    A, B = cases[4]
    thr = ozo.esc_threshold(OSET[set_name])
    for side, X in ((0, A), (1, B)):
        lines = X.shape[0] if side == 0 else X.shape[1]
        k = X.shape[1] if side == 0 else X.shape[0]
        p = oz.oz_plane_count_side(gh.SETS[set_name], gh.route(sub), side)
        pitch = oz.oz_row_pitch(k)
        planes = torch.empty((p, lines, pitch), dtype=torch.uint8, device="cuda")
        shift = torch.empty((lines,), dtype=torch.int32, device="cuda")
        scratch = torch.zeros(16 * lines + 256, dtype=torch.uint8, device="cuda")
        oz.check(oz.oz_deconstruct(side, lines, k, gh.to_dev(X), X.shape[0], gh.SETS[set_name], gh.route(sub), planes,
                                   lines * pitch, pitch, shift, scratch), "oz_deconstruct")
        want = oz.OZ_ERR_RANGE if min(ozo.esc_flatness(side, X), 65536) * 65536 < thr else 0
        assert gh.sync_status(esc=True) == want
