"""Full-size parity: the bf16 workloads at their benchmark sizes, in the launch configuration bench.py
times, against the complete CPU oracle on the same seeded inputs (about a minute of host time each)."""
import numpy as np
import pytest
import torch

from paper_2506_18145_b200 import synth

from rom_testlib import TOL, GpuLayer, assert_close, np64, oracle_layer

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["long_ctx", "zipf", "short_seqs"])
def test_layer_full_size(name):
    s = synth.CONFIGS[name]
    p = synth.make_inputs(s)
    g = GpuLayer(s, p)
    out = np64(g.forward())
    idx = g.idx.cpu().numpy(); counts = g.counts.cpu().numpy(); gates = g.gates.cpu().numpy()
    Yg_rows = g.tap("row_of_assign", torch.int32, 1).view(-1)[::s.K].long()
    Yg = np64(g.tap("Ygp", synth.torch_dtype(s), s.d_inner)[Yg_rows])
    del g
    torch.cuda.empty_cache()
    ref, im = oracle_layer(s, p)
    np.testing.assert_array_equal(idx, im["idx"])
    np.testing.assert_array_equal(counts, im["counts"])
    np.testing.assert_allclose(gates, im["gate"], rtol=2e-6)
    assert_close(Yg, im["Yg"], TOL["bf16"], "Yg")
    assert_close(out, ref, TOL["bf16"], "out")
