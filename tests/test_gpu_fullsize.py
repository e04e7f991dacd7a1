"""Full-size parity: the bf16 workloads at their benchmark sizes, in the launch configuration bench.py
times, against the complete CPU oracle on the same seeded inputs (about a minute of host time each)."""
import numpy as np
import pytest
import torch

from oracle import rom_oracle as O
from paper_2506_18145_b200 import binding as rb
from paper_2506_18145_b200 import synth

from rom_testlib import TOL, GpuLayer, assert_close, gpu_route, np64, oracle_layer

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


def test_ffn_moe_full_size_sampled_tokens():
    """FFN-MoE with shared routing at the benchmark shape (`bench.py --stage ffn`: long_ctx widths, d_ff = 4 d_model):
    the experts are per-token functions, so the oracle is evaluated on a sample of 384 tokens (every 43rd)."""
    s = synth.CONFIGS["long_ctx"]
    d_ff = 4 * s.d_model
    p = synth.make_inputs(s.replace(d_inner=64, dt_rank=16))
    g = torch.Generator().manual_seed(s.seed_base + 900)
    W_gu = (torch.randn((s.E, 2 * d_ff, s.d_model), generator=g) * 0.02).to(torch.bfloat16)
    W_down = (torch.randn((s.E, s.d_model, d_ff), generator=g) * 0.02).to(torch.bfloat16)
    r = gpu_route(s, p)
    cfg = rb.config_from_shape(s)
    idx = torch.from_numpy(r["idx"]).cuda(); gates = torch.from_numpy(r["gates"]).cuda()
    ws = torch.empty(rb.ffn_moe_workspace_size(cfg, d_ff), dtype=torch.uint8, device="cuda")
    out = torch.empty((s.B, s.L, s.d_model), dtype=torch.bfloat16, device="cuda")
    rb.rom_ffn_moe_forward(cfg, d_ff, W_gu.cuda(), W_down.cuda(), p["x"].cuda(), idx, gates, out, ws)
    torch.cuda.synchronize()
    assert rb.rom_get_status(ws) == 0
    sample = np.arange(0, s.T, 43)[:384]
    x = np64(p["x"]).reshape(s.T, s.d_model)[sample]
    ref = O.ffn_moe_shared_routing(x, np64(W_gu), np64(W_down), r["idx"][sample], r["gates"][sample].astype(np.float64))
    assert_close(np64(out).reshape(s.T, s.d_model)[sample], ref, TOL["bf16"], "ffn out (sampled tokens)")


def test_layer_step_full_size():
    """Single-token step at the benchmark shape (`bench.py --stage step`: 64 sequences, long_ctx widths): three steps
    against the oracle's step with states carried on both sides."""
    s = synth.CONFIGS["long_ctx"].replace(B=64, L=3)
    p = synth.make_inputs(s, recipe="unit")
    cfg = rb.config_from_shape(s.replace(L=1))
    dev = {k: (None if v is None else v.cuda().contiguous()) for k, v in p.items()}
    weights = rb.make_weights(dev)
    ws = rb.alloc_workspace(cfg, "cuda")
    conv_state = torch.zeros((s.B, s.d_conv - 1, s.d_inner), dtype=torch.float32, device="cuda")
    ssm_state = torch.zeros((s.B, s.d_inner, s.d_state), dtype=torch.float32, device="cuda")
    out = torch.empty((s.B, s.d_model), dtype=torch.bfloat16, device="cuda")
    o_conv = np.zeros((s.B, s.d_conv - 1, s.d_inner)); o_h = np.zeros((s.B, s.d_inner, s.d_state))
    wn = [np64(p[k]) for k in ("W_r", "b_r", "W_inz", "w_conv", "b_conv", "W_x", "W_dt", "b_dt", "A", "D", "W_out")]
    for t in range(s.L):
        rb.rom_layer_step(cfg, weights, dev["x"][:, t].contiguous(), conv_state, ssm_state, out, None, None, ws)
        torch.cuda.synchronize()
        assert rb.rom_get_status(ws) == 0
        ref, o_conv, o_h = O.rom_layer_step(np64(p["x"][:, t]), o_conv, o_h, *wn, K=s.K, dt_rank=s.dt_rank)
        assert_close(np64(out), ref, TOL["bf16"], f"step {t} out")
    assert_close(np64(ssm_state), o_h, TOL["bf16"], "state-space state")


def test_layer_full_size_per_expert_small_projections():
    """The per-expert x Proj / dt Proj mode (`bench.py --small-proj routed`) at the benchmark workload."""
    s = synth.CONFIGS["long_ctx"]
    p = synth.make_inputs(s, routed_small=True)
    g = GpuLayer(s, p)
    out = np64(g.forward())
    idx = g.idx.cpu().numpy()
    del g
    torch.cuda.empty_cache()
    ref, im = oracle_layer(s, p)
    np.testing.assert_array_equal(idx, im["idx"])
    assert_close(out, ref, TOL["bf16"], "out")


@pytest.mark.parametrize("name", ["long_ctx", "zipf"])
def test_route_balance_full_size(name):
    """Load-balance statistic of the router (Appendix A.3) at benchmark sizes."""
    s = synth.CONFIGS[name]
    p = synth.make_inputs(s.replace(d_inner=64, dt_rank=16))
    cfg = rb.config_from_shape(s)
    ws = rb.alloc_workspace(cfg)
    F = torch.empty(s.E, dtype=torch.float32, device="cuda"); Pb = torch.empty_like(F)
    loss = torch.empty(1, dtype=torch.float32, device="cuda")
    b_r = None if p["b_r"] is None else p["b_r"].cuda()
    rb.rom_route_balance(cfg, p["x"].cuda(), p["W_r"].cuda(), b_r, 1e-3, F, Pb, loss, ws)
    torch.cuda.synchronize()
    idx, gate, P, logit = O.route(np64(p["x"]).reshape(s.T, s.d_model), np64(p["W_r"]), np64(p["b_r"]), s.K)
    want, Fr = O.load_balance_loss(P, idx, alpha=1e-3)
    np.testing.assert_allclose(F.cpu().numpy(), Fr, rtol=1e-6)
    np.testing.assert_allclose(Pb.cpu().numpy(), P.mean(axis=0), rtol=2e-6)
    np.testing.assert_allclose(float(loss.item()), want, rtol=2e-6)

