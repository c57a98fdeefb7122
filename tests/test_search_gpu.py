"""The search driver (decode -> evaluate -> select on the device) on the tiny pipeline: from random priority
lists it reaches the optimum of the identity placement, and what it reports agrees with the oracle."""
import numpy as np
import pytest

from paper_2503_09357_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def test_search_finds_the_pipeline_optimum_and_reports_what_the_oracle_computes():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from oracle import pe_oracle as orc
    from paper_2503_09357_b200 import binding as pe
    from paper_2503_09357_b200 import search
    w = wl.make_config(1)                         # 4 stages x 8 microbatches, F = 2, B = 4, transfer 1, capacity 8
    V, K = w.num_ops, 4096
    S, M = 4, 8
    stage = np.concatenate([np.repeat(np.arange(S), M)] * 2).astype(np.uint8)       # op -> its stage's machine
    assign = torch.from_numpy(np.repeat(stage[:, None], K, axis=1).copy()).cuda()
    gen = torch.Generator(device="cuda"); gen.manual_seed(1)
    lists = torch.argsort(torch.rand((V, K), device="cuda", generator=gen), dim=0).to(torch.int16).contiguous()
    g = pe.Graph(w)
    try:
        res = search.evolve(g, assign, lists, generations=60, swaps=2, seed=2)
        # stage s cannot start before s (f + c); the last stage then has M (f + b) of work, and its last backward
        # op is followed by S - 1 more, each after a transfer: (M + S - 1)(f + b) + 2 (S - 1) c = 72
        assert res["history"][-1] <= res["history"][0]
        assert res["best_makespan"] == 72
        a = res["best_assign"].cpu().numpy()[:, None]; o = res["best_order"].cpu().numpy().view(np.uint16)[:, None]
        ref = orc.evaluate(w, a, o)
        assert int(ref["makespan"][0]) == 72 and int(ref["status"][0]) == 0       # within the memory limit too
        dec, st = orc.decode(w, res["best_list"].cpu().numpy().view(np.uint16)[:, None])
        assert st[0] == 0 and np.array_equal(dec, o)
        # the random-key variant (same assignment in every column) reaches the same optimum
        rk = search.evolve_keys(g, assign, generations=80, seed=4)
        assert rk["best_makespan"] == 72
        o2 = rk["best_order"].cpu().numpy().view(np.uint16)[:, None]
        ref2 = orc.evaluate(w, a, o2)
        assert int(ref2["makespan"][0]) == 72 and int(ref2["status"][0]) == 0
    finally:
        g.close()


def test_search_reaches_the_zero_bubble_of_the_two_stage_bidirectional_pipeline():
    """Section V-A at the paper's unit times: for PP = 2 the bubble of the bidirectional pipeline is 0
    (tests/golden/bidirectional_pp2_zero_bubble.txt pins that value on the oracle).  The search has to find
    it from random priority lists, within the memory limit 2 x parameters + (PP + 1) activations; the PP = 4
    run is reported as context only (the paper's microbatch count is not printed)."""
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from oracle import pe_oracle as orc
    from paper_2503_09357_b200 import binding as pe
    from paper_2503_09357_b200 import search
    from paper_2503_09357_b200.workloads import graphs
    for PP, M, must in ((2, 4, 0), (4, 8, None)):
        w = graphs.bidirectional_unit(PP, M)
        V, K = w.num_ops, 8192
        slot = (np.arange(V) % PP).astype(np.uint8)                          # slot p on machine p
        assign = torch.from_numpy(np.repeat(slot[:, None], K, axis=1).copy()).cuda()
        gen = torch.Generator(device="cuda"); gen.manual_seed(PP * 100 + M)
        lists = torch.argsort(torch.rand((V, K), device="cuda", generator=gen), dim=0).to(torch.int16).contiguous()
        g = pe.Graph(w)
        try:
            res = search.evolve(g, assign, lists, generations=150, swaps=2, seed=3)
            busy = 3 * M                                                     # F + B + W of every microbatch, one unit each
            bubble = res["best_makespan"] - busy
            ref = orc.evaluate(w, res["best_assign"].cpu().numpy()[:, None],
                               res["best_order"].cpu().numpy().view(np.uint16)[:, None])
            assert int(ref["makespan"][0]) == res["best_makespan"] and int(ref["status"][0]) == 0
            assert (ref["busy"][:, 0] == busy).all() and (ref["peak_mem"][:, 0] <= 2 + PP + 1).all()
            assert bubble >= 0
            if must is not None:
                assert bubble == must
            print(f"bidirectional unit pipeline PP={PP} M={M}: bubble {bubble} "
                  f"(Section V-A: best found PP/2-1 = {PP // 2 - 1}, DualPipe 2(PP/2-1) = {2 * (PP // 2 - 1)})")
        finally:
            g.close()
