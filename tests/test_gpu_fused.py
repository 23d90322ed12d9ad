"""Storage mode F (Sec. "Storage Modes", mode F; "O4: pipelining"): the product kernel converts A's
tiles itself, A's planes never exist in memory.  The residues are the same integers, so the whole call
must be bit-identical to the oracle and to the materialised path."""
import numpy as np
import pytest

import synth_inputs as syn
from oracle import oz_oracle as ozo

pytestmark = pytest.mark.gpu

OSET = {"S": ozo.SET_S, "E": ozo.SET_E, "A": ozo.SET_A}


def _fused(sub="fp8", quant="RN", rule="CS"):
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    return gh.route(sub, quant, rule) | oz.OZ_STORAGE_FUSED


@pytest.mark.parametrize("set_name,sub,m,n,k,dist,quant,rule", [
    ("S", "fp8", 64, 128, 32, "uniform", "RN", "CS"),            # one tile, one stage
    ("S", "fp8", 300, 128, 1000, "normal", "RN", "CS"),          # ragged rows, ragged k (tail of 8)
    ("S", "fp8", 1000, 70, 4097, "lognormal:0.5", "TZ", "CS"),   # the deepest exact k on S, ragged n
    ("S", "int8", 257, 100, 515, "normal", "RN", "MAXEXP"),      # INT8 digits, merged on both operands
    ("E", "fp8", 130, 1, 260, "uniform", "RN", "CS"),            # 13 moduli: the fourth pass holds one
    ("E", "int8", 77, 128, 129, "lognormal:0.5", "TZ", "CS"),
    ("A", "fp8", 200, 33, 300, "normal", "RN", "CS"),            # byte residues (15 moduli, 4 passes)
    ("A", "int8", 129, 127, 64, "uniform", "RN", "CS"),
    ("S", "fp8", 20000, 128, 256, "normal", "RN", "CS"),         # more tiles than SMs: persistent loop
    ("S", "fp8", 1, 1, 1, "uniform", "RN", "CS"),
])
def test_fused_mode_bit_identical_to_oracle(set_name, sub, m, n, k, dist, quant, rule):
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(m + 3 * n + 7 * k)
    A, B = syn._draw(rng, m, k, dist), syn._draw(rng, k, n, dist)
    C0 = np.asfortranarray(rng.standard_normal((m, n)))
    oq = ozo.QUANT_RN if quant == "RN" else ozo.QUANT_TZ
    orule = ozo.SCALE_CS if rule == "CS" else ozo.SCALE_MAXEXP
    for alpha, beta in ((1.0, 0.0), (-1.0, 1.0)):
        got, st = gh.dgemm(A, B, set_name, _fused(sub, quant, rule), alpha, beta, C0 if beta else None)
        want = ozo.dgemm(A, B, OSET[set_name], oq, orule, alpha, beta, C0 if beta else None)
        assert st == 0
        assert (got == want).all()


def test_fused_mode_special_lines():
    """Rows of zeros, subnormal rows, single huge entries, a row of A with NaN and a column of B with Inf."""
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    for kind in ("zero_lines", "subnormal", "spike", "small_integers"):
        A, B = syn.special_operands(kind, 150, 90, 300)
        got, st = gh.dgemm(A, B, "S", _fused())
        assert st == 0 and (got == ozo.dgemm(A, B, ozo.SET_S)).all(), kind
    A, B = syn.special_operands("spike", 100, 60, 200)
    A[70, 5] = np.nan
    B[9, 33] = np.inf
    got, st = gh.dgemm(A, B, "S", _fused())
    want = ozo.dgemm(A, B, ozo.SET_S)
    assert st == oz.OZ_ERR_NONFINITE_INPUT
    assert (np.isnan(got) == np.isnan(want)).all() and (got[~np.isnan(want)] == want[~np.isnan(want)]).all()


def test_fused_mode_limits():
    import torch
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    t = torch.zeros(200 * 5000, dtype=torch.float64, device="cuda")
    gh.ensure_workspace(oz.oz_workspace_bytes(200, 200, 5000, oz.OZ_SET_S, _fused()))
    # n above one tile of B lines; k beyond the exact depth of the merged FP32 accumulator on S; other modes
    assert oz.oz_dgemm(200, 129, 64, t, 200, t, 64, t, 200, oz.OZ_SET_S, _fused()) == oz.OZ_ERR_UNSUPPORTED
    assert oz.oz_dgemm(200, 64, 4098, t, 200, t, 4098, t, 200, oz.OZ_SET_S, _fused()) == oz.OZ_ERR_UNSUPPORTED
    assert oz.oz_dgemm(200, 64, 4098, t, 200, t, 4098, t, 200, oz.OZ_SET_E, _fused()) == oz.OZ_OK
    assert oz.oz_dgemm(200, 64, 64, t, 200, t, 64, t, 200, oz.OZ_SET_A, _fused("int8n")) == oz.OZ_ERR_UNSUPPORTED
    assert oz.oz_dgemm(200, 64, 64, t, 200, t, 64, t, 200, oz.OZ_SET_S, _fused(rule="ACCURATE")) == oz.OZ_ERR_UNSUPPORTED
    assert oz.oz_dgemm(200, 64, 64, t, 200, t, 64, t, 200, oz.OZ_SET_S, _fused() | oz.OZ_ACC_SEPARATE) == oz.OZ_ERR_UNSUPPORTED
    assert oz.oz_dgemm(200, 64, 64, t, 200, t, 64, t, 200, oz.OZ_SET_S, _fused() | oz.OZ_FALLBACK_FP64) == oz.OZ_ERR_UNSUPPORTED
    assert gh.sync_status() == 0
    # no planes of A in the workspace: 131072 x 128 x 4096 needs 16 GB less than the materialised mode
    plain = oz.oz_workspace_bytes(131072, 128, 4096, oz.OZ_SET_S, gh.route("fp8"))
    fused = oz.oz_workspace_bytes(131072, 128, 4096, oz.OZ_SET_S, _fused())
    assert plain - fused >= 30 * 131072 * 4096
