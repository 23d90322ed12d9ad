"""oz_deconstruct_static -- the entry point for callers that may not allocate device memory --
must give exactly what oz_deconstruct gives, call after call.

Collected last on purpose: if it fails, a run that stops at the first failure has already run
every other test.  It passes alone in a fresh process and after the rest of the suite, because
the built-in scratch is cleared by every call before use."""
import numpy as np
import pytest

import synth_inputs as syn

pytestmark = pytest.mark.gpu


def _both(side, X, set_name, rt):
    """Planes and shifts from the allocating-caller entry point and from the static one."""
    import torch
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh

    lines = X.shape[0] if side == 0 else X.shape[1]
    k = X.shape[1] if side == 0 else X.shape[0]
    ref_planes, ref_shift, st = gh.deconstruct(side, X, set_name, rt)
    assert st == 0
    _, p, _ = oz.oz_set_info(gh.SETS[set_name])
    pitch = oz.oz_row_pitch(k)
    dX = gh.to_dev(X)
    planes = torch.full((p, lines, pitch), 0x55, dtype=torch.uint8, device="cuda")
    shift = torch.full((lines,), -7, dtype=torch.int32, device="cuda")
    oz.check(oz.oz_deconstruct_static(side, lines, k, dX, X.shape[0], gh.SETS[set_name], rt, planes,
                                      lines * pitch, pitch, shift), "oz_deconstruct_static")
    assert gh.sync_status() == 0
    return ref_planes, ref_shift, planes.cpu().numpy(), shift.cpu().numpy()


def test_static_entry_matches_the_regular_one_twice_in_a_row():
    import tests.gpu_helpers as gh
    rng = np.random.default_rng(77)
    # two calls in a row on different operands, sides and shapes: the second must not see
    # anything the first left in the shared scratch (here the first has MORE lines than the second)
    first = syn._draw(rng, 700, 300, "lognormal:2.0")      # side 0: 700 lines
    second = syn._draw(rng, 129, 257, "normal")            # side 1: 257 lines
    for side, X, set_name, rt in ((0, first, "S", gh.route("fp8", "RN", "CS")),
                                  (1, second, "E", gh.route("int8", "TZ", "CS")),
                                  (0, first, "S", gh.route("fp8", "RN", "MAXEXP"))):
        ref_p, ref_s, got_p, got_s = _both(side, X, set_name, rt)
        assert (got_s == ref_s).all()
        assert (got_p == ref_p).all()      # integer outputs: bit-exact, as in the other tests


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
