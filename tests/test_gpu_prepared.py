"""Planes kept across calls (storage mode P; paragraph "O1: convert-once residue-plane workspace"):
an operand deconstructed once with oz_prepare_operand serves any number of oz_dgemm_prepared calls,
and every such product is bit-identical to the whole-method call on the same matrices."""
import numpy as np
import pytest

import synth_inputs as syn
from oracle import oz_oracle as ozo

pytestmark = pytest.mark.gpu

OSET = {"S": ozo.SET_S, "E": ozo.SET_E, "A": ozo.SET_A}


@pytest.mark.parametrize("set_name,sub,m,k,widths", [
    ("S", "fp8", 700, 384, (256, 130, 515)),       # an HPL-like panel of A against three column blocks
    ("E", "int8", 300, 1000, (129, 64)),
    ("A", "int8n", 520, 260, (300, 31, 257)),
    ("S", "fp8", 260, 5003, (200,)),               # merged accumulators cut into K segments
])
def test_prepared_operands_reused_across_products(set_name, sub, m, k, widths):
    import torch
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(m * 7 + k)
    A = syn._draw(rng, m, k, "lognormal:0.5")
    rt = gh.route(sub)
    sid = gh.SETS[set_name]
    dA = gh.to_dev(A)
    opA = torch.empty(oz.oz_operand_bytes(0, m, k, sid, rt), dtype=torch.uint8, device="cuda")
    oz.check(oz.oz_prepare_operand(0, m, k, dA, m, sid, rt, opA), "oz_prepare_operand A")
    image = opA.clone()
    for rep, n in enumerate(widths):
        B = syn._draw(rng, k, n, "normal")
        C0 = syn._draw(rng, m, n, "uniform")
        alpha, beta = ((1.0, 0.0), (-1.0, 1.0))[rep % 2]
        dB = gh.to_dev(B)
        opB = torch.empty(oz.oz_operand_bytes(1, n, k, sid, rt), dtype=torch.uint8, device="cuda")
        oz.check(oz.oz_prepare_operand(1, n, k, dB, k, sid, rt, opB), "oz_prepare_operand B")
        ws = torch.empty(oz.oz_product_workspace_bytes(m, n, sid), dtype=torch.uint8, device="cuda")
        oz.check(oz.oz_set_workspace(ws), "oz_set_workspace")
        got = []
        for _ in range(2):                       # the same two operands twice: nothing is consumed
            dC = gh.to_dev(C0)
            oz.check(oz.oz_dgemm_prepared(m, n, k, alpha, opA, opB, beta, dC, m, sid, rt), "oz_dgemm_prepared")
            assert gh.sync_status() == 0
            got.append(gh.from_dev(dC))
        oz.oz_set_workspace(None)
        assert (got[0] == got[1]).all()
        whole, st = gh.dgemm(A, B, set_name, rt, alpha, beta, C0 if beta else None)
        assert st == 0 and (got[0] == whole).all()          # bit-identical to the whole-method call
        want = ozo.dgemm(A, B, OSET[set_name], ozo.QUANT_RN, ozo.SCALE_CS, alpha, beta, C0 if beta else None)
        assert (got[0] == want).all()                        # and to the oracle
    assert bool((opA == image).all())                        # the products never write the operand


def test_prepared_argument_errors():
    import torch
    import paper_2609_09095_b200 as oz
    t = torch.zeros(4096, dtype=torch.float64, device="cuda")
    block = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    assert oz.oz_prepare_operand(0, 8, 8, t, 4, oz.OZ_SET_S, 0, block) == oz.OZ_ERR_INVALID_ARG      # ldx < lines
    assert oz.oz_prepare_operand(0, 8, 8, t, 8, oz.OZ_SET_S, 0, block, 64) == oz.OZ_ERR_WORKSPACE    # block too small
    assert oz.oz_prepare_operand(1, 0, 8, t, 8, oz.OZ_SET_S, 0, block) == oz.OZ_OK
    oz.oz_set_workspace(None)
    assert oz.oz_dgemm_prepared(8, 8, 8, 1.0, block, block, 0.0, t, 8) == oz.OZ_ERR_WORKSPACE
    assert oz.oz_dgemm_prepared(8, 8, 8, 0.5, block, block, 0.0, t, 8) == oz.OZ_ERR_UNSUPPORTED
    assert oz.oz_dgemm_prepared(8, 8, 8, 1.0, None, block, 0.0, t, 8) == oz.OZ_ERR_INVALID_ARG
