"""Out-of-range rows on the native FP64 path (Algorithm 1, last line: "ESC check; native-FP64 fallback
for out-of-range rows"; Algorithm 3: "ESC range check; re-issue out-of-range rows on the native-FP64
path").  The rows that fail the exponent-span check are left out of the reconstruction and computed
as compensated FP64 inner products in k order; the whole call must be bit-identical to the oracle's
statement of the same rule, and the number of re-issued rows must be the oracle's."""
import numpy as np
import pytest

import synth_inputs as syn
from oracle import oz_oracle as ozo

pytestmark = pytest.mark.gpu

OSET = {"S": ozo.SET_S, "E": ozo.SET_E, "A": ozo.SET_A}


def _wide(rng, rows, cols, sigma):
    return np.asfortranarray(rng.standard_normal((rows, cols)) * np.exp(sigma * rng.standard_normal((rows, cols))))


@pytest.mark.parametrize("set_name,sub,m,n,k,sigma,quant", [
    ("A", "fp8", 150, 100, 300, 2.5, "RN"),        # some rows fail, some pass
    ("A", "int8n", 333, 70, 161, 2.5, "TZ"),       # ragged in every dimension, several row blocks
    ("S", "fp8", 70, 130, 5003, 2.0, "RN"),        # the wide benchmark distribution: every row fails
    ("E", "int8", 65, 65, 17, 3.0, "RN"),          # one inner block with a tail
    ("S", "fp8", 1, 1, 1, 1.0, "RN"),
])
def test_fallback_bit_identical_to_oracle(set_name, sub, m, n, k, sigma, quant):
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(m * 7 + n * 3 + k)
    A, B = _wide(rng, m, k, sigma), _wide(rng, k, n, sigma)
    if m > 20:
        A[3, :] = 0.5                                   # a flat row among the wide ones
        A[5, :] = 0.0
    C0 = np.asfortranarray(rng.standard_normal((m, n)))
    oq = ozo.QUANT_RN if quant == "RN" else ozo.QUANT_TZ
    for alpha, beta in ((1.0, 0.0), (-1.0, 1.0)):
        oz.oz_query_fallback_rows()
        got, st = gh.dgemm(A, B, set_name, gh.route(sub, quant, "CS", fallback=True), alpha, beta, C0 if beta else None)
        rows = oz.oz_query_fallback_rows()
        want, flag = ozo.dgemm_fallback(A, B, OSET[set_name], oq, alpha, beta, C0 if beta else None)
        assert st == 0 and rows == int(flag.sum())
        assert (got == want).all()
        assert oz.oz_query_fallback_rows() == 0         # the count is cleared by the query


@pytest.mark.parametrize("seed", range(12))
def test_fallback_random_shapes(seed):
    """Seeded random shapes, sets, substrates, quantisers, scalars and exponent spreads on the route with
    the native path: whatever share of the rows the check sends there, the matrix is the oracle's."""
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(7000 + seed)
    m, n, k = int(rng.integers(1, 400)), int(rng.integers(1, 400)), int(rng.integers(1, 700))
    set_name, sub = [("S", "fp8"), ("A", "int8n"), ("E", "int8"), ("A", "fp8")][seed % 4]
    quant = ("RN", "TZ")[int(rng.integers(2))]
    alpha, beta = (1.0, -1.0)[int(rng.integers(2))], (0.0, 1.0)[int(rng.integers(2))]
    sigma = (0.5, 1.5, 2.0, 2.5, 3.0)[int(rng.integers(5))]
    A, B = _wide(rng, m, k, sigma), _wide(rng, k, n, sigma)
    C0 = np.asfortranarray(rng.standard_normal((m, n))) if beta else None
    oz.oz_query_fallback_rows()
    got, st = gh.dgemm(A, B, set_name, gh.route(sub, quant, "CS", fallback=True), alpha, beta, C0)
    want, flag = ozo.dgemm_fallback(A, B, OSET[set_name], ozo.QUANT_RN if quant == "RN" else ozo.QUANT_TZ,
                                    alpha, beta, C0)
    assert st == 0 and oz.oz_query_fallback_rows() == int(flag.sum())
    assert (got == want).all()


def test_fallback_mixes_and_reports():
    """Set A on the sigma = 2.5 data: the check splits the rows, so both paths write into the same C."""
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(1357)
    A, B = _wide(rng, 150, 300, 2.5), _wide(rng, 300, 100, 2.5)
    flag = ozo.esc_rows(A, B, ozo.SET_A)
    assert 0 < flag.sum() < len(flag)
    got, st = gh.dgemm(A, B, "A", gh.route("fp8", fallback=True))
    oz.oz_query_fallback_rows()
    plain, _ = gh.dgemm(A, B, "A", gh.route("fp8"))
    assert (got[flag == 0] == plain[flag == 0]).all() and (got[flag == 1] != plain[flag == 1]).any()
    # the check itself is still reported
    # run once more and read the raw status
    import torch
    m, k, n = 150, 300, 100
    dA, dB = gh.to_dev(A), gh.to_dev(B)
    dC = torch.zeros((n, m), dtype=torch.float64, device="cuda")
    oz.check(oz.oz_dgemm(m, n, k, dA, m, dB, k, dC, m, oz.OZ_SET_A, gh.route("fp8", fallback=True)), "oz_dgemm")
    assert oz.oz_query_status() == oz.OZ_ERR_RANGE
    assert oz.oz_query_fallback_rows() == int(flag.sum())
    assert (gh.from_dev(dC) == got).all()


def test_fallback_restores_the_contract_on_the_wide_distribution():
    """Config-5 data: the plain call misses 2u (|A||B|) against the double-double product, the call with
    the native path meets it everywhere."""
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    A, B = syn.operands(syn.CONFIGS[5], 200, 140, 5003)
    hi, lo, ab = ozo.dd_gemm(A, B)
    bound = 2 * 2.0 ** -53 * ab
    plain, _ = gh.dgemm(A, B, "S", gh.route("fp8"))
    got, st = gh.dgemm(A, B, "S", gh.route("fp8", fallback=True))
    assert st == 0 and oz.oz_query_fallback_rows() == 200
    assert (np.abs(plain - hi) > bound).any()
    assert (np.abs(got - hi) <= bound).all()


def test_fallback_leaves_benign_calls_alone():
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    A, B = syn.operands(syn.CONFIGS[3], 300, 260, 512)
    C0 = np.asfortranarray(np.random.default_rng(5).standard_normal((300, 260)))
    oz.oz_query_fallback_rows()
    got, st = gh.dgemm(A, B, "S", gh.route("fp8", fallback=True), -1.0, 1.0, C0)
    assert st == 0 and oz.oz_query_fallback_rows() == 0
    assert (got == ozo.dgemm(A, B, ozo.SET_S, alpha=-1.0, beta=1.0, C0=C0)).all()


def test_fallback_with_nonfinite_lines():
    """A row of A with NaN is not re-issued (its result is NaN either way); a column of B with Inf gives
    NaN in the re-issued rows too."""
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(99)
    A, B = _wide(rng, 90, 200, 2.5), _wide(rng, 200, 75, 2.5)
    A[11, 17] = np.nan
    B[3, 40] = np.inf
    got, st = gh.dgemm(A, B, "S", gh.route("fp8", fallback=True))
    want, flag = ozo.dgemm_fallback(A, B, ozo.SET_S)
    assert st == oz.OZ_ERR_NONFINITE_INPUT and flag[11] == 0 and flag.sum() > 0
    assert oz.oz_query_fallback_rows() == int(flag.sum())
    assert (np.isnan(got) == np.isnan(want)).all() and np.isnan(got[:, 40]).all() and np.isnan(got[11, :]).all()
    assert (got[~np.isnan(want)] == want[~np.isnan(want)]).all()


def test_fallback_unsupported_combinations():
    import torch
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    m = n = k = 64
    A, B = syn.operands(syn.CONFIGS[1], m, n, k)
    dA, dB = gh.to_dev(A), gh.to_dev(B)
    dC = torch.zeros((n, m), dtype=torch.float64, device="cuda")
    gh.ensure_workspace(oz.oz_workspace_bytes(m, n, k, oz.OZ_SET_S, gh.route("fp8", fallback=True)))
    for rt in (gh.route("fp8", rule="ACCURATE", fallback=True), gh.route("fp8", rule="MAXEXP", fallback=True),
               gh.route("fp8", recon="tensor", fallback=True)):
        assert oz.oz_dgemm(m, n, k, dA, m, dB, k, dC, m, oz.OZ_SET_S, rt) == oz.OZ_ERR_UNSUPPORTED
    # the workspace of the route is larger than that of the plain one, and the call checks it
    plain, fb = (oz.oz_workspace_bytes(4096, n, k, oz.OZ_SET_S, gh.route("fp8", fallback=f)) for f in (False, True))
    assert fb > plain
