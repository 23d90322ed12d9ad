"""Parity at the full benchmark sizes, in the launch configuration bench.py times: the stage entry
points and oz_dgemm_ex run on the whole problem; the oracle recomputes sampled lines / outputs
(lines of A and B are independent, so a sample of rows x columns is an exact sub-problem).
Integer outputs bit-exact; FP64 within 2 * 2^-53 * (|A||B|)_ij of the oracle (in fact identical)."""
import numpy as np
import pytest
import torch

import synth_inputs as syn
from oracle import oz_oracle as ozo

pytestmark = pytest.mark.gpu
U = 2.0 ** -53
OSET = {"S": ozo.SET_S, "E": ozo.SET_E, "A": ozo.SET_A}
OSUB = {"fp8": ozo.SUB_FP8, "int8": ozo.SUB_INT8, "int8n": ozo.SUB_INT8_NATIVE}


def _sample(n, rng, tile):
    """Indices spanning first/last lines, both sides of tile edges, and random ones."""
    fixed = [0, 1, n - 1, n - 2, tile - 1, tile, tile + 1, n // 2, (n // tile) * tile - 1, (n // tile) * tile]
    idx = {i for i in fixed if 0 <= i < n}
    idx.update(int(v) for v in rng.integers(0, n, size=40))
    return np.array(sorted(idx))


@pytest.mark.parametrize("cfg_id,set_name,sub", [(2, "S", "fp8"), (3, "S", "fp8"), (3, "E", "fp8"),
                                                 (5, "S", "fp8"), (4, "S", "int8"), (4, "S", "fp8"),
                                                 (3, "A", "int8n")])
def test_full_size_sampled(cfg_id, set_name, sub):
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    cfg = syn.CONFIGS[cfg_id]
    m, n, k = cfg.m, cfg.n, cfg.k
    rng = np.random.default_rng(cfg.seed + 17)
    A, B, C0 = syn.operands(cfg, want_c=True) if cfg.beta else (*syn.operands(cfg), None)
    rows, cols = _sample(m, rng, 256), _sample(n, rng, 128)
    As, Bs = np.asfortranarray(A[rows, :]), np.asfortranarray(B[:, cols])
    rt = gh.route(sub, "RN", "CS")
    osub = OSUB[sub]
    oset = OSET[set_name]

    # ---- oracle on the sampled sub-problem, stage by stage
    tA, tB = ozo.budget_maxexp(oset, k)
    sA = ozo.shifts(0, As, oset, ozo.SCALE_CS, tA)
    sB = ozo.shifts(1, Bs, oset, ozo.SCALE_CS, tB)
    DA = ozo.residues(ozo.quantise(0, As, sA, ozo.QUANT_RN), oset)
    DB = ozo.residues(ozo.quantise(1, Bs, sB, ozo.QUANT_RN), oset)
    PAo, PBo = ozo.planes(DA, oset, osub), ozo.planes(DB, oset, osub)
    Ro = ozo.products(DA, DB, oset)
    Cs0 = None if C0 is None else np.asfortranarray(C0[np.ix_(rows, cols)])
    Co = ozo.output(ozo.crt(Ro, oset), sA, sB, cfg.alpha, cfg.beta, Cs0)

    # ---- GPU, whole problem, stage entry points (the launchers oz_dgemm uses)
    r, _, _ = oz.oz_set_info(gh.SETS[set_name])
    p = oz.oz_plane_count(gh.SETS[set_name], rt)
    pitch = oz.oz_row_pitch(k)
    dA, dB = gh.to_dev(A), gh.to_dev(B)
    PA = torch.empty((p, m, pitch), dtype=torch.uint8, device="cuda")
    PB = torch.empty((p, n, pitch), dtype=torch.uint8, device="cuda")
    shA = torch.empty(m, dtype=torch.int32, device="cuda")
    shB = torch.empty(n, dtype=torch.int32, device="cuda")
    scr = torch.empty(16 * max(m, n) + 256, dtype=torch.uint8, device="cuda")
    oz.check(oz.oz_deconstruct(0, m, k, dA, m, gh.SETS[set_name], rt, PA, m * pitch, pitch, shA, scr), "deconstruct A")
    oz.check(oz.oz_deconstruct(1, n, k, dB, k, gh.SETS[set_name], rt, PB, n * pitch, pitch, shB, scr), "deconstruct B")
    ldr = (m + 15) // 16 * 16
    R = torch.empty((r, n, ldr), dtype=gh.residue_dtype(set_name)[0], device="cuda")
    oz.check(oz.oz_residue_gemm(m, n, k, PA, m * pitch, pitch, PB, n * pitch, pitch, gh.SETS[set_name], rt, R,
                                ldr, n * ldr), "residue gemm")
    assert gh.sync_status() == 0
    ri, ci = torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()
    assert (shA[ri].cpu().numpy() == sA).all() and (shB[ci].cpu().numpy() == sB).all()
    assert (PA[:, ri, :].cpu().numpy() == PAo).all()
    assert (PB[:, ci, :].cpu().numpy() == PBo).all()
    if R.dtype == torch.uint8:
        Rs = R[:, ci, :][:, :, ri].cpu().numpy()
    else:
        Rs = R.view(torch.int16)[:, ci, :][:, :, ri].cpu().numpy().view(np.uint16)   # torch cannot index uint16
    assert (Rs == Ro).all()
    del PA, PB, R
    torch.cuda.empty_cache()

    # ---- GPU, whole method in one call (what bench.py times)
    gh.ensure_workspace(oz.oz_workspace_bytes(m, n, k, gh.SETS[set_name], rt))
    dC = gh.to_dev(C0) if C0 is not None else torch.empty((n, m), dtype=torch.float64, device="cuda")
    oz.check(oz.oz_dgemm_ex(m, n, k, cfg.alpha, dA, m, dB, k, cfg.beta, dC, m, gh.SETS[set_name], rt), "oz_dgemm_ex")
    # exponent-span check at full size: the oracle's result on the whole operands (config 5 is flagged)
    flagged = ozo.esc_check(A, B, oset)
    assert flagged == (cfg_id == 5)
    assert gh.sync_status(esc=True) == (oz.OZ_ERR_RANGE if flagged else 0)
    got = dC[ci, :][:, ri].cpu().numpy().T
    _, _, ab = ozo.dd_gemm(As, Bs)
    assert (np.abs(got - Co) <= 2 * U * ab).all()
    assert (got == Co).all()
    # a whole-matrix property that holds at any size: no entry is left unwritten / non-finite
    assert bool(torch.isfinite(dC).all())
    if cfg_id in (3, 5):
        # the reconstruction hosted on the tensor pipe gives the same matrix, entry for entry
        dC2 = gh.to_dev(C0) if C0 is not None else torch.empty((n, m), dtype=torch.float64, device="cuda")
        oz.check(oz.oz_dgemm_ex(m, n, k, cfg.alpha, dA, m, dB, k, cfg.beta, dC2, m, gh.SETS[set_name],
                                rt | oz.OZ_RECON_TENSOR), "oz_dgemm_ex, tensor-hosted reconstruction")
        assert gh.sync_status() == 0
        assert bool((dC2 == dC).all())
        del dC2
    del dA, dB, dC
    oz.oz_set_workspace(None)
    gh._ws = None
    torch.cuda.empty_cache()


@pytest.mark.parametrize("set_name,sub", [("S", "fp8"), ("A", "int8n")])
def test_full_size_fallback_sampled(set_name, sub):
    """Config 5 at full size with the out-of-range rows re-issued on the native FP64 path: the rows the
    oracle's check flags on the whole operands are the
    compensated inner products, the others the method's; every sampled entry meets 2u (|A||B|)
    against the double-double product where it was re-issued."""
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    cfg = syn.CONFIGS[5]
    m, n, k = cfg.m, cfg.n, cfg.k
    rng = np.random.default_rng(cfg.seed + 23)
    A, B = syn.operands(cfg)
    oset = OSET[set_name]
    flag = ozo.esc_rows(A, B, oset)
    assert flag.any()          # against the least flat of 9973 columns every row fails, on either set
    rows, cols = _sample(m, rng, 256), _sample(n, rng, 128)
    As, Bs = np.asfortranarray(A[rows, :]), np.asfortranarray(B[:, cols])
    native = ozo.native_rows(As, Bs, np.ones(len(rows), dtype=np.uint8))
    method = ozo.dgemm(As, Bs, oset)          # rows and columns are independent: an exact sub-problem
    want = np.where(flag[rows][:, None] == 1, native, method)
    rt = gh.route(sub, "RN", "CS", fallback=True)
    gh.ensure_workspace(oz.oz_workspace_bytes(m, n, k, gh.SETS[set_name], rt))
    dA, dB = gh.to_dev(A), gh.to_dev(B)
    dC = torch.empty((n, m), dtype=torch.float64, device="cuda")
    oz.oz_query_fallback_rows()
    oz.check(oz.oz_dgemm(m, n, k, dA, m, dB, k, dC, m, gh.SETS[set_name], rt), "oz_dgemm, native path")
    assert gh.sync_status(esc=True) == oz.OZ_ERR_RANGE
    assert oz.oz_query_fallback_rows() == int(flag.sum())
    ri, ci = torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()
    got = dC[ci, :][:, ri].cpu().numpy().T
    assert (got == want).all()
    hi, _, ab = ozo.dd_gemm(As, Bs)
    re = flag[rows] == 1
    assert (np.abs(got - hi)[re] <= (2 * U * ab)[re]).all()
    assert bool(torch.isfinite(dC).all())
    del dA, dB, dC
    oz.oz_set_workspace(None)
    gh._ws = None
    torch.cuda.empty_cache()
