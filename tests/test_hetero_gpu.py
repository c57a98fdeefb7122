"""Heterogeneous machines on the GPU (dur_by_machine of pe_graph_desc; Section III, footnote) against the oracle."""
import copy

import numpy as np
import pytest

from paper_2503_09357_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pe():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2503_09357_b200 import binding
    return binding


@pytest.mark.parametrize("config,kw,K", [(1, {}, 1024), (2, {}, 4096), (4, {}, 777), (5, dict(V=4096, D=8), 300)])
def test_machine_dependent_durations_match_the_oracle(pe, config, kw, K):
    w = copy.copy(wl.make_config(config, **kw))
    rs = np.random.RandomState(config)
    w.dur_by_machine = rs.randint(0, 40, (w.num_ops, w.num_devices)).astype(np.int32)
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    try:
        ran = []
        for name, bit in (("auto", 0), ("shared", pe.PE_VARIANT_SHARED), ("global", pe.PE_VARIANT_GLOBAL)):
            if pe.pe_eval_variant(g.handle, K, bit) < 0:
                continue
            gu.check(g, w, assign, order, flags=bit, label=f"hetero config {config} {name}")
            ran.append(name)
        assert "global" in ran
        for bit in (pe.PE_VARIANT_WARP, pe.PE_VARIANT_TEAM):
            assert pe.pe_eval_variant(g.handle, K, bit) == pe.PE_ERR_UNSUPPORTED
        a_pos = wl.assign_by_pos(assign, order)
        gu.check(g, w, a_pos, order, flags=pe.PE_ASSIGN_BY_POS | pe.PE_TIMES_BY_OP, label="hetero layouts")
        gu.check(g, w, assign, order, flags=pe.PE_COMM_EXCLUSIVE, label="hetero exclusive channels")
    finally:
        g.close()


def test_a_constant_table_gives_the_homogeneous_result(pe):
    w = wl.make_config(2)
    K = 512
    assign, order = wl.make_candidates(w, K=K)
    g = pe.Graph(w)
    base = gu.gpu_eval(g, assign, order)
    g.close()
    w2 = copy.copy(w)
    w2.dur_by_machine = np.repeat(np.asarray(w.dur, np.int32)[:, None], w.num_devices, axis=1)
    g = pe.Graph(w2)
    same = gu.gpu_eval(g, assign, order)
    g.close()
    for key in base:
        assert np.array_equal(base[key], same[key]), key
