"""A whole-method call captured in a CUDA graph (after one plain call, which creates the library's
internal stream and events) and replayed on new operand values gives the oracle's result each time:
the call enqueues only kernels, event records and stream waits, so capture sees all of it."""
import numpy as np
import pytest

import synth_inputs as syn
from oracle import oz_oracle as ozo

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("m,n,k,set_name,sub,mode", [
    (256, 256, 256, "S", "fp8", None),            # one-kernel deconstruction
    (300, 2200, 2100, "A", "int8n", None),        # three-pass deconstruction of B
    (300, 100, 500, "S", "fp8", "fused"),         # storage mode F: A converted inside the product kernel
    (200, 150, 300, "A", "fp8", "fallback"),      # native FP64 path: the number of re-issued rows varies per replay
])
def test_dgemm_replayed_from_a_cuda_graph(m, n, k, set_name, sub, mode):
    import torch
    import paper_2609_09095_b200 as oz
    import tests.gpu_helpers as gh
    sid, rt = gh.SETS[set_name], gh.route(sub, fallback=(mode == "fallback"))
    if mode == "fused":
        rt |= oz.OZ_STORAGE_FUSED
    oset = {"S": ozo.SET_S, "A": ozo.SET_A}[set_name]
    rng = np.random.default_rng(k)
    gh.ensure_workspace(oz.oz_workspace_bytes(m, n, k, sid, rt))
    dA = torch.zeros((k, m), dtype=torch.float64, device="cuda")
    dB = torch.zeros((n, k), dtype=torch.float64, device="cuda")
    dC = torch.zeros((n, m), dtype=torch.float64, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        # plain call first: internal stream and events are created outside the capture
        oz.check(oz.oz_dgemm(m, n, k, dA, m, dB, k, dC, m, sid, rt, side), "oz_dgemm")
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            oz.check(oz.oz_dgemm(m, n, k, dA, m, dB, k, dC, m, sid, rt, torch.cuda.current_stream()), "oz_dgemm (capture)")
    for rep in range(3):
        if mode == "fallback":      # exponent spreads from benign to wide: none, some or all rows re-issued
            sg = (0.5, 2.5, 3.5)[rep]
            A = np.asfortranarray(rng.standard_normal((m, k)) * np.exp(sg * rng.standard_normal((m, k))))
            B = np.asfortranarray(rng.standard_normal((k, n)) * np.exp(sg * rng.standard_normal((k, n))))
        else:
            A, B = syn._draw(rng, m, k, "uniform"), syn._draw(rng, k, n, "normal")
        dA.copy_(gh.to_dev(A))
        dB.copy_(gh.to_dev(B))
        dC.fill_(-1.0)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert gh.sync_status() == 0
        if mode == "fallback":
            want, flag = ozo.dgemm_fallback(A, B, oset)
            assert oz.oz_query_fallback_rows() == int(flag.sum())
        else:
            want = ozo.dgemm(A, B, oset)
        assert (gh.from_dev(dC) == want).all()
