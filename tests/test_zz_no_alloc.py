"""oz_deconstruct_static -- the entry point for callers that may not allocate device memory --
must give exactly what the oracle and oz_deconstruct give, call after call, and must leave the
amount of free device memory unchanged.

The file is collected after the other GPU tests so that it sees the built-in scratch in whatever
state they left it: every call clears the part it uses before use, so the test passes both alone
in a fresh process and at the end of the whole suite."""
import numpy as np
import pytest

import synth_inputs as syn
from oracle import oz_oracle as ozo

pytestmark = pytest.mark.gpu

OSET = {"S": ozo.SET_S, "E": ozo.SET_E}
OSUB = {"fp8": ozo.SUB_FP8, "int8": ozo.SUB_INT8}


def _static(side, X, set_name, rt):
    """Planes and shifts from the static entry point (outputs pre-filled with junk)."""
    import torch
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh

    lines = X.shape[0] if side == 0 else X.shape[1]
    k = X.shape[1] if side == 0 else X.shape[0]
    _, p, _ = oz.oz_set_info(gh.SETS[set_name])
    pitch = oz.oz_row_pitch(k)
    dX = gh.to_dev(X)
    planes = torch.full((p, lines, pitch), 0x55, dtype=torch.uint8, device="cuda")
    shift = torch.full((lines,), -7, dtype=torch.int32, device="cuda")
    oz.check(oz.oz_deconstruct_static(side, lines, k, dX, X.shape[0], gh.SETS[set_name], rt, planes,
                                      lines * pitch, pitch, shift), "oz_deconstruct_static")
    assert gh.sync_status() == 0
    return planes.cpu().numpy(), shift.cpu().numpy()


def _oracle(side, X, set_name, sub, quant, rule):
    k = X.shape[1] if side == 0 else X.shape[0]
    tA, tB = ozo.budget_maxexp(OSET[set_name], max(k, 1))
    sh = ozo.shifts(side, X, OSET[set_name], ozo.SCALE_CS if rule == "CS" else ozo.SCALE_MAXEXP,
                    tA if side == 0 else tB)
    Q = ozo.quantise(side, X, sh, ozo.QUANT_RN if quant == "RN" else ozo.QUANT_TZ)
    return ozo.planes(ozo.residues(Q, OSET[set_name]), OSET[set_name], OSUB[sub]), sh


def test_static_entry_matches_oracle_and_regular_entry_twice_in_a_row():
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(77)
    # calls in a row on different operands, sides and shapes: a call must not see anything an
    # earlier one left in the shared scratch (the first has MORE lines than the second)
    first = syn._draw(rng, 700, 300, "lognormal:2.0")      # side 0: 700 lines
    second = syn._draw(rng, 129, 257, "normal")            # side 1: 257 lines
    for side, X, set_name, sub, quant, rule in ((0, first, "S", "fp8", "RN", "CS"),
                                                (1, second, "E", "int8", "TZ", "CS"),
                                                (0, first, "S", "fp8", "RN", "MAXEXP")):
        rt = gh.route(sub, quant, rule)
        got_p, got_s = _static(side, X, set_name, rt)
        want_p, want_s = _oracle(side, X, set_name, sub, quant, rule)
        assert (got_s == want_s).all()
        assert got_p.shape == want_p.shape and (got_p == want_p).all()     # integer outputs: bit-exact
        ref_p, ref_s, st = gh.deconstruct(side, X, set_name, rt)          # and the same as the regular entry point
        assert st == 0 and (got_s == ref_s).all() and (got_p == ref_p).all()


def test_static_entry_allocates_nothing_and_holds_its_maximum():
    """Free device memory is the same before and after a call (after one warm-up call that lets the
    library look the scratch address up), also at the largest supported line count."""
    import torch
    import paper_2609_09095_b200 as oz
    lines, k = oz.OZ_STATIC_MAX_LINES, 16
    rng = np.random.default_rng(78)
    X = syn._draw(rng, k, lines, "uniform")                 # side 1: `lines` columns of length k
    dX = torch.from_numpy(np.ascontiguousarray(X.T)).cuda()
    _, p, _ = oz.oz_set_info(oz.OZ_SET_S)
    pitch = oz.oz_row_pitch(k)
    planes = torch.empty((p, lines, pitch), dtype=torch.uint8, device="cuda")
    shift = torch.empty((lines,), dtype=torch.int32, device="cuda")
    scratch = torch.zeros(16 * lines + 256, dtype=torch.uint8, device="cuda")
    ref_planes, ref_shift = torch.empty_like(planes), torch.empty_like(shift)
    oz.check(oz.oz_deconstruct(1, lines, k, dX, k, oz.OZ_SET_S, 0, ref_planes, lines * pitch, pitch, ref_shift,
                               scratch), "oz_deconstruct")

    def call():
        oz.check(oz.oz_deconstruct_static(1, lines, k, dX, k, oz.OZ_SET_S, 0, planes, lines * pitch, pitch, shift),
                 "oz_deconstruct_static")
        torch.cuda.synchronize()

    call()                                                  # first call on the device: address look-up
    free_before, _ = torch.cuda.mem_get_info()
    call()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert oz.oz_query_status() == 0          # uniform lines: the exponent-span check has nothing to say
    assert bool((shift == ref_shift).all()) and bool((planes == ref_planes).all())
    # the line sampled against the oracle: first, last and a few in between
    pick = np.array([0, 1, lines // 2, lines - 2, lines - 1])
    want_p, want_s = _oracle(1, np.asfortranarray(X[:, pick]), "S", "fp8", "RN", "CS")
    assert (shift.cpu().numpy()[pick] == want_s).all()
    assert (planes[:, torch.from_numpy(pick).cuda(), :].cpu().numpy() == want_p).all()


def test_static_entry_rejects_what_it_cannot_hold():
    import torch
    import paper_2609_09095_b200 as oz
    t = torch.zeros(16, dtype=torch.float64, device="cuda")
    u = torch.zeros(64, dtype=torch.uint8, device="cuda")
    s = torch.zeros(4, dtype=torch.int32, device="cuda")
    too_many = oz.OZ_STATIC_MAX_LINES + 1
    assert oz.oz_deconstruct_static(0, too_many, 1, t, too_many, oz.OZ_SET_S, 0, u, too_many * 16, 16, s) \
        == oz.OZ_ERR_WORKSPACE
    assert oz.oz_deconstruct_static(0, 0, 4, t, 1, oz.OZ_SET_S, 0, u, 16, 16, s) == oz.OZ_OK
