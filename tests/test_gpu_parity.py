"""Parity of the CUDA path (called through the C ABI) against the CPU fp64 oracle on the same
seeded inputs.  Integer results (top-K indices, counts, offsets, permutation) must be bit-exact;
floating-point results within 1e-4 (fp32 path) / 2e-2 (bf16 path) relative, in max-norm and 2-norm."""
import numpy as np
import pytest
import torch

from oracle import rom_oracle as O
from paper_2506_18145_b200 import binding as rb
from paper_2506_18145_b200 import synth

from rom_testlib import TOL, GpuLayer, assert_close, check_route_exact, gpu_route, np64, oracle_layer

pytestmark = pytest.mark.gpu


def small_shape(**kw):
    base = dict(name="t", B=2, L=300, d_model=128, d_inner=256, d_state=16, d_conv=4, dt_rank=16, E=4, K=2,
                dtype="bf16", seed_base=77000)
    base.update(kw)
    return synth.RomShape(**base)


# ---------------------------------------------------------------------------------------------- routing
@pytest.mark.parametrize("kw", [
    dict(B=1, L=50, E=5, K=2),                       # one ragged chunk
    dict(B=3, L=333, E=8, K=1),                      # ragged tail, several blocks
    dict(B=2, L=1000, E=16, K=2),
    dict(B=1, L=257, E=64, K=8, d_model=64),         # maximum E and K
    dict(B=1, L=1, E=3, K=3),                        # a single token, K = E
    dict(B=4, L=512, E=8, K=2, dtype="f32"),
    dict(B=1, L=4096, E=1, K=1),                     # one expert
])
@pytest.mark.parametrize("gate_mode", [0, 1])
def test_route_bit_exact(kw, gate_mode):
    s = small_shape(**kw)
    p = synth.make_inputs(s, recipe="unit")
    got = gpu_route(s, p, gate_mode)
    check_route_exact(got, s, p, gate_mode)


def test_route_ties_bias_and_empty_experts():
    s = small_shape(B=2, L=200, E=8, K=2, router_bias_scale=3.0)
    p = synth.make_inputs(s, recipe="unit")
    W = p["W_r"].clone(); W[5] = W[2]; W[7] = 0; p["W_r"] = W          # duplicate rows: ties -> lowest id
    b = p["b_r"].clone(); b[5] = b[2]; b[6] = -1e9; p["b_r"] = b        # expert 6 never chosen
    got = gpu_route(s, p)
    idx, _ = check_route_exact(got, s, p)
    assert got["counts"][6] == 0
    assert not np.any(idx[:, 0] == 5)          # the duplicate of expert 2 never comes first
    # all-zero tokens: every logit equals the bias; without bias -> experts 0..K-1
    p2 = synth.make_inputs(small_shape(B=1, L=70, E=6, K=3), recipe="unit")
    p2["x"] = torch.zeros_like(p2["x"])
    s2 = small_shape(B=1, L=70, E=6, K=3)
    got2 = gpu_route(s2, p2)
    check_route_exact(got2, s2, p2)
    assert np.array_equal(got2["idx"], np.tile(np.arange(3, dtype=np.int32), (70, 1)))


@pytest.mark.parametrize("name", ["tiny_fp32", "small_bf16", "long_ctx", "zipf", "short_seqs"])
def test_route_bit_exact_full_size_configs(name):
    s = synth.CONFIGS[name]
    small = s.replace(d_inner=64, dt_rank=16)       # x, W_r, b_r depend only on the seeds and d_model
    p = synth.make_inputs(small)
    got = gpu_route(s, p)
    check_route_exact(got, s, p)
    if name == "zipf":
        ratio = got["counts"].max() / got["counts"].mean()
        assert 4.5 < ratio < 5.5, ratio


@pytest.mark.parametrize("kw", [dict(B=2, L=333, E=8, K=2), dict(B=1, L=50, E=5, K=1), dict(B=4, L=512, E=16, K=2, dtype="f32", router_bias_scale=2.0)])
def test_route_balance_statistic(kw):
    # Appendix A.3: F_i, mean softmax and alpha * E * sum F_i Pbar_i against the oracle on the same inputs
    s = small_shape(**kw)
    p = synth.make_inputs(s, recipe="unit")
    cfg = rb.config_from_shape(s)
    ws = rb.alloc_workspace(cfg)
    F = torch.empty(s.E, dtype=torch.float32, device="cuda"); Pb = torch.empty_like(F); loss = torch.empty(1, dtype=torch.float32, device="cuda")
    b_r = None if p["b_r"] is None else p["b_r"].cuda()
    rb.rom_route_balance(cfg, p["x"].cuda(), p["W_r"].cuda(), b_r, 1e-3, F, Pb, loss, ws)
    torch.cuda.synchronize()
    idx, gate, P, logit = O.route(np64(p["x"]).reshape(s.T, s.d_model), np64(p["W_r"]), np64(p["b_r"]), s.K)
    want, Fr = O.load_balance_loss(P, idx, alpha=1e-3)
    np.testing.assert_allclose(F.cpu().numpy(), Fr, rtol=1e-6)
    np.testing.assert_allclose(Pb.cpu().numpy(), P.mean(axis=0), rtol=2e-6)
    np.testing.assert_allclose(float(loss.item()), want, rtol=2e-6)
    assert abs(float(F.sum().item()) - s.K) < 1e-5


# ---------------------------------------------------------------------------------------------- scan
def run_scan(B, L, De, dtype, disc_mode, with_z, with_h0, with_D, seed, use_ws=False):
    q = synth.make_scan_inputs(B, L, De, 16, dtype, seed, with_z=with_z, with_h0=with_h0)
    if not with_D:
        q["D"] = None
    cfg = rb.make_config(B, L, 64, De, 16, 4, 16, 1, 1, dtype, 0, disc_mode)
    d = {k: (None if v is None else v.cuda()) for k, v in q.items()}
    y = torch.empty_like(d["u"])
    h_last = torch.empty((B, De, 16), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(rb.scan_workspace_size(cfg), 16), dtype=torch.uint8, device="cuda") if use_ws else None      # with a workspace long sequences run as parallel chunks
    rb.rom_scan(cfg, d["u"], d["delta"], d["A"], d["Bm"], d["Cm"], d["D"], d["z"], d["h0"], y, h_last, ws)
    torch.cuda.synchronize()
    Y, hl = O.selective_scan(np64(q["u"]), np64(q["delta"]), np64(q["A"]), np64(q["Bm"]), np64(q["Cm"]), np64(q["D"]),
                             np64(q["h0"]), disc_mode)
    if with_z:
        Y = O.gated(Y, np64(q["z"]))
    return np64(y), Y, np64(h_last), hl


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("disc_mode", [0, 1])
@pytest.mark.parametrize("B,L,De,with_z,with_h0,with_D", [
    (2, 100, 192, True, False, True),      # ragged L, channel count not a multiple of the block
    (1, 777, 64, False, True, False),      # no gate, initial state, no skip
    (3, 1, 128, True, True, True),         # single step
    (1, 2048, 256, True, False, True),     # several time tiles
])
def test_scan_parity(dtype, disc_mode, B, L, De, with_z, with_h0, with_D):
    y, Y, hl, HL = run_scan(B, L, De, dtype, disc_mode, with_z, with_h0, with_D, seed=9100 + L)
    assert_close(y, Y, TOL[dtype], "scan y")
    assert_close(hl, HL, 1e-4 if dtype == "f32" else 2e-3, "scan h_last")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("disc_mode", [0, 1])
@pytest.mark.parametrize("B,L,De,with_z,with_h0,with_D", [
    (1, 2048, 256, True, False, True),     # 8 chunks of 256 steps
    (2, 1500, 192, True, True, True),      # ragged last chunk, initial state carried through the chunk chain
    (1, 4100, 64, False, True, False),     # chunk length rounded up: trailing chunks are empty
    (3, 100, 128, True, True, True),       # too short to chunk: the workspace is simply unused
])
def test_scan_parity_chunked(dtype, disc_mode, B, L, De, with_z, with_h0, with_D):
    y, Y, hl, HL = run_scan(B, L, De, dtype, disc_mode, with_z, with_h0, with_D, seed=9500 + L, use_ws=True)
    assert_close(y, Y, TOL[dtype], "chunked scan y")
    assert_close(hl, HL, 1e-4 if dtype == "f32" else 2e-3, "chunked scan h_last")


def test_scan_long_memory_small_delta():
    # Delta*A down to -1e-3: the regime where exp(x) - 1 cancels; the fp32 path must still hold 1e-4
    B, L, De = 1, 4096, 64
    q = synth.make_scan_inputs(B, L, De, 16, "f32", 9300, with_z=False)
    q["delta"] = q["delta"] * 0.05
    q["A"] = -torch.ones_like(q["A"]) * torch.linspace(0.2, 1.0, 16)[None, :]
    cfg = rb.make_config(B, L, 64, De, 16, 4, 16, 1, 1, "f32")
    d = {k: (None if v is None else v.cuda()) for k, v in q.items()}
    y = torch.empty_like(d["u"])
    rb.rom_scan(cfg, d["u"], d["delta"], d["A"], d["Bm"], d["Cm"], d["D"], None, None, y, None)
    torch.cuda.synchronize()
    Y, _ = O.selective_scan(np64(q["u"]), np64(q["delta"]), np64(q["A"]), np64(q["Bm"]), np64(q["Cm"]), np64(q["D"]))
    assert_close(np64(y), Y, 1e-4, "long-memory scan")


# ---------------------------------------------------------------------------------------------- layer
def check_layer(s, recipe, with_D=True, gate_mode=0, disc_mode=0, flags=0, check_taps=True, routed_small=False):
    p = synth.make_inputs(s, recipe=recipe, with_D=with_D, routed_small=routed_small)
    ref, im = oracle_layer(s, p, gate_mode, disc_mode)
    g = GpuLayer(s, p, gate_mode, disc_mode, flags)
    out = g.forward()
    tol = TOL[s.dtype]
    np.testing.assert_array_equal(g.idx.cpu().numpy(), im["idx"])
    np.testing.assert_array_equal(g.counts.cpu().numpy(), im["counts"])
    np.testing.assert_allclose(g.gates.cpu().numpy(), im["gate"], rtol=2e-6)
    if check_taps:
        tdt = synth.torch_dtype(s)
        assert_close(np64(g.tap("U", tdt, s.d_inner)), im["U"], tol, "U")
        assert_close(np64(g.tap("Bm", torch.float32, s.d_state)), im["Bm"], tol, "Bm")
        assert_close(np64(g.tap("Cm", torch.float32, s.d_state)), im["Cm"], tol, "Cm")
        assert_close(np64(g.tap("Delta", tdt, s.d_inner)), im["Delta"], tol, "Delta")
        rows = g.tap("row_of_assign", torch.int32, 1).view(-1)[::s.K].long()      # slot 0 row of each token
        assert_close(np64(g.tap("Ygp", tdt, s.d_inner)[rows]), im["Yg"], tol, "Yg")
    e = assert_close(np64(out), ref, tol, "out")
    assert rb.last_launch_count() >= 6
    return e


@pytest.mark.parametrize("recipe,with_D", [("paper", True), ("unit", True), ("unit", False)])
def test_layer_tiny_fp32_config(recipe, with_D):
    check_layer(synth.CONFIGS["tiny_fp32"], recipe, with_D)


@pytest.mark.parametrize("kw", [
    dict(),                                                       # K = 2, ragged L
    dict(E=8, K=1, B=3, L=130),
    dict(E=3, K=3, L=64, d_conv=3),
    dict(E=4, K=1, d_conv=2, dt_rank=32, B=1, L=1),               # one token
    dict(E=6, K=2, router_bias_scale=4.0, L=513),                 # skewed loads, some experts nearly empty
])
@pytest.mark.parametrize("dtype,flags", [("f32", 0), ("bf16", rb.ROM_FLAG_SIMT_GEMM), ("bf16", 0)])
def test_layer_small_shapes(kw, dtype, flags):
    s = small_shape(dtype=dtype, **kw)
    check_layer(s, "unit", flags=flags)


@pytest.mark.parametrize("gate_mode,disc_mode", [(1, 0), (0, 1), (1, 1)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_layer_modes(gate_mode, disc_mode, dtype):
    s = small_shape(dtype=dtype, L=200)
    check_layer(s, "unit", gate_mode=gate_mode, disc_mode=disc_mode)


# per-expert x Proj / dt Proj (the "(Conv, Gate, dt, x, Out)" ablation row of Section 5.3)
@pytest.mark.parametrize("kw", [
    dict(),                                                       # K = 2, ragged L
    dict(E=8, K=1, B=3, L=130),
    dict(E=3, K=3, L=64, d_conv=3),
    dict(E=4, K=1, dt_rank=32, B=1, L=1),                         # one token
    dict(E=6, K=2, router_bias_scale=4.0, L=513),                 # skewed loads, some experts nearly empty
])
@pytest.mark.parametrize("dtype,flags", [("f32", 0), ("bf16", rb.ROM_FLAG_SIMT_GEMM), ("bf16", 0)])
def test_layer_routed_small_projections(kw, dtype, flags):
    s = small_shape(dtype=dtype, **kw)
    check_layer(s, "unit", flags=flags, routed_small=True)


def test_layer_routed_small_projections_small_bf16_config():
    check_layer(synth.CONFIGS["small_bf16"], "unit", routed_small=True)


def test_layer_routed_small_with_identical_experts_matches_shared_path_on_gpu():
    """E copies of one x Proj / dt Proj, top-1: the per-expert path must reproduce the shared path's rows."""
    s = small_shape(E=4, K=1, L=400)
    p = synth.make_inputs(s, recipe="unit")
    shared = GpuLayer(s, p).forward().clone()
    q = dict(p)
    q["W_x"] = p["W_x"][None].repeat(s.E, 1, 1).contiguous(); q["W_dt"] = p["W_dt"][None].repeat(s.E, 1, 1).contiguous()
    routed = GpuLayer(s, q).forward()
    assert_close(np64(routed), np64(shared), 1e-2, "per-expert vs shared")


def test_layer_single_expert_is_dense_mamba_on_gpu():
    s = small_shape(E=1, K=1, L=256, dtype="bf16")
    check_layer(s, "unit")


@pytest.mark.parametrize("recipe,with_D", [("paper", True), ("unit", False)])
def test_layer_small_bf16_config(recipe, with_D):
    check_layer(synth.CONFIGS["small_bf16"], recipe, with_D)


def test_layer_batch_permutation_invariance_on_gpu():
    s = small_shape(B=4, L=128, E=4, K=2)
    p = synth.make_inputs(s, recipe="unit")
    g = GpuLayer(s, p)
    out = g.forward().clone()
    counts = g.counts.clone()
    pi = torch.tensor([2, 0, 3, 1], device="cuda")
    out2 = g.forward(g.dev["x"][pi].contiguous())
    assert torch.equal(out2, out[pi])
    assert torch.equal(g.counts, counts)


# ---------------------------------------------------------------------------------------------- FFN-MoE with shared routing
def run_ffn(s, d_ff, flags=0, seed=91000, bad_index=False):
    """Route on the GPU (rom_route), hand idx / gates to rom_ffn_moe_forward, compare with the oracle fed the oracle's own
    routing of the same inputs (indices are bit-exact, so both sides use the same experts)."""
    p = synth.make_inputs(s, recipe="unit")
    tdt = synth.torch_dtype(s)
    g = torch.Generator().manual_seed(seed)
    W_gu = (torch.randn((s.E, 2 * d_ff, s.d_model), generator=g) / s.d_model ** 0.5).to(tdt)
    W_down = (torch.randn((s.E, s.d_model, d_ff), generator=g) / d_ff ** 0.5).to(tdt)
    r = gpu_route(s, p)
    cfg = rb.config_from_shape(s, flags=flags)
    idx = torch.from_numpy(r["idx"]).cuda(); gates = torch.from_numpy(r["gates"]).cuda()
    if bad_index:
        idx[0, 0] = s.E + 3
    ws = torch.empty(rb.ffn_moe_workspace_size(cfg, d_ff), dtype=torch.uint8, device="cuda")
    out = torch.empty((s.B, s.L, s.d_model), dtype=tdt, device="cuda")
    rb.rom_ffn_moe_forward(cfg, d_ff, W_gu.cuda(), W_down.cuda(), p["x"].cuda(), idx, gates, out, ws)
    torch.cuda.synchronize()
    code = rb.rom_get_status(ws)
    if bad_index:
        return code
    assert code == 0, rb.status_string(code)
    x = np64(p["x"]).reshape(s.T, s.d_model)
    o_idx, o_gate, _, _ = O.route(x, np64(p["W_r"]), np64(p["b_r"]), s.K, 0)
    np.testing.assert_array_equal(r["idx"], o_idx)
    ref = O.ffn_moe_shared_routing(x, np64(W_gu), np64(W_down), o_idx, o_gate)
    return assert_close(np64(out).reshape(s.T, s.d_model), ref, TOL[s.dtype], "ffn out")


@pytest.mark.parametrize("kw,d_ff", [
    (dict(), 256),                                               # K = 2, ragged L
    (dict(E=8, K=1, B=3, L=130), 384),                           # top-1: gate and token order fused into the down projection
    (dict(E=3, K=3, L=64), 128),
    (dict(E=4, K=1, B=1, L=1), 128),                             # one token
    (dict(E=6, K=2, router_bias_scale=4.0, L=513), 256),         # skewed loads, some experts nearly empty
])
@pytest.mark.parametrize("dtype,flags", [("f32", 0), ("bf16", rb.ROM_FLAG_SIMT_GEMM), ("bf16", 0)])
def test_ffn_moe_shared_routing(kw, d_ff, dtype, flags):
    run_ffn(small_shape(dtype=dtype, **kw), d_ff, flags)


def test_ffn_moe_small_bf16_config():
    s = synth.CONFIGS["small_bf16"]
    run_ffn(s, 4 * s.d_model)


def test_ffn_moe_reports_an_index_out_of_range():
    code = run_ffn(small_shape(E=4, K=2, L=100), 128, bad_index=True)
    assert code == -1 and "invalid" in rb.status_string(code)


# ---------------------------------------------------------------------------------------------- single-token step
def run_steps(s, n_steps, flags=0, routed_small=False):
    """Feed the first n_steps tokens of every sequence one at a time through rom_layer_step (states carried on the GPU) and
    through the oracle's step (states carried in fp64); compare every output and the final states."""
    p = synth.make_inputs(s, recipe="unit", routed_small=routed_small)
    tdt = synth.torch_dtype(s)
    s1 = s.replace(L=1)
    cfg = rb.config_from_shape(s1, flags=flags, small_proj_experts=s.E if routed_small else 0)
    dev = {k: (None if v is None else v.cuda().contiguous()) for k, v in p.items()}
    weights = rb.make_weights(dev)
    ws = rb.alloc_workspace(cfg, "cuda")
    conv_state = torch.zeros((s.B, s.d_conv - 1, s.d_inner), dtype=torch.float32, device="cuda")
    ssm_state = torch.zeros((s.B, s.d_inner, s.d_state), dtype=torch.float32, device="cuda")
    out = torch.empty((s.B, s.d_model), dtype=tdt, device="cuda")
    idx = torch.empty((s.B, s.K), dtype=torch.int32, device="cuda")
    o_conv = np.zeros((s.B, s.d_conv - 1, s.d_inner)); o_h = np.zeros((s.B, s.d_inner, s.d_state))
    wnames = ("W_r", "b_r", "W_inz", "w_conv", "b_conv", "W_x", "W_dt", "b_dt", "A", "D", "W_out")
    wn = [np64(p[k]) for k in wnames]
    tol = TOL[s.dtype]
    outs = []
    for t in range(n_steps):
        x_t = dev["x"][:, t].contiguous()
        rb.rom_layer_step(cfg, weights, x_t, conv_state, ssm_state, out, idx, None, ws)
        torch.cuda.synchronize()
        assert rb.rom_get_status(ws) == 0
        ref, o_conv, o_h = O.rom_layer_step(np64(p["x"][:, t]), o_conv, o_h, *wn, K=s.K, dt_rank=s.dt_rank)
        assert_close(np64(out), ref, tol, f"step {t} out")
        outs.append(out.clone())
    assert_close(np64(conv_state), o_conv, tol, "conv state")
    assert_close(np64(ssm_state), o_h, tol, "state-space state")
    return p, torch.stack(outs, dim=1)


@pytest.mark.parametrize("kw", [
    dict(B=3, L=12, E=4, K=2),
    dict(B=5, L=12, E=8, K=1),
    dict(B=2, L=12, E=3, K=3, d_conv=3),
    dict(B=1, L=12, E=4, K=1, d_conv=2, dt_rank=32),
    dict(B=5, L=12, E=4, K=1, d_inner=2048),                      # wide enough for the thread-split x Proj kernel
])
@pytest.mark.parametrize("dtype,flags", [("f32", 0), ("bf16", rb.ROM_FLAG_SIMT_GEMM), ("bf16", 0)])
def test_layer_step_parity(kw, dtype, flags):
    run_steps(small_shape(dtype=dtype, **kw), 12, flags)


def test_layer_step_routed_small_projections():
    run_steps(small_shape(B=4, L=8, E=4, K=2), 8, routed_small=True)


def test_layer_steps_reproduce_the_full_forward_on_gpu():
    """fp32 path: twelve single-token steps against rom_layer_forward on the same twelve tokens."""
    s = small_shape(B=3, L=12, E=4, K=2, dtype="f32")
    p, stepped = run_steps(s, 12)
    full = GpuLayer(s, p).forward()
    assert_close(np64(stepped), np64(full), 1e-4, "steps vs full forward")


def test_layer_step_rejects_a_sequence_length_other_than_one():
    s = small_shape(B=2, L=4)
    cfg = rb.config_from_shape(s)
    p = synth.make_inputs(s, recipe="unit")
    dev = {k: (None if v is None else v.cuda().contiguous()) for k, v in p.items()}
    ws = rb.alloc_workspace(cfg, "cuda")
    cs = torch.zeros((s.B, s.d_conv - 1, s.d_inner), device="cuda"); hs = torch.zeros((s.B, s.d_inner, s.d_state), device="cuda")
    out = torch.empty((s.B, s.d_model), dtype=torch.bfloat16, device="cuda")
    rc = rb.rom_layer_step(cfg, rb.make_weights(dev), dev["x"][:, 0].contiguous(), cs, hs, out, None, None, ws, check=False)
    assert rc == -1


def test_layer_forward_host_matches_the_device_entry_point():
    """rom_layer_forward_host (pinned host in / out, copies enqueued by the library) gives the device path's bits."""
    s = small_shape(B=2, L=333, E=4, K=2)
    p = synth.make_inputs(s, recipe="unit")
    g = GpuLayer(s, p)
    ref = g.forward().clone()
    x_host = p["x"].contiguous().pin_memory()
    out_host = torch.empty_like(p["x"]).pin_memory()
    x_dev = torch.empty_like(g.dev["x"]); out_dev = torch.empty_like(g.dev["x"])
    rb.rom_layer_forward_host(g.cfg, g.weights, x_host, out_host, x_dev, out_dev, g.ws)
    torch.cuda.synchronize()
    assert rb.rom_get_status(g.ws) == 0
    assert torch.equal(out_host, ref.cpu())


# ---------------------------------------------------------------------------------------------- ragged widths, size limits
@pytest.mark.parametrize("dtype,flags", [("f32", 0), ("bf16", rb.ROM_FLAG_SIMT_GEMM), ("bf16", 0)])
@pytest.mark.parametrize("kw", [
    dict(d_model=192, d_inner=320, dt_rank=48, E=5, K=2, B=2, L=257),      # widths that are multiples of 64 only
    dict(d_model=64, d_inner=64, dt_rank=16, E=2, K=1, B=1, L=700),        # the smallest widths
    dict(d_model=128, d_inner=192, dt_rank=16, E=64, K=8, B=1, L=300),     # the largest expert count and top-K
    dict(d_model=128, d_inner=2048, dt_rank=16, E=4, K=2, B=1, L=99),      # few tokens, wide: thread-split x Proj kernel
])
def test_layer_ragged_widths_and_limits(kw, dtype, flags):
    check_layer(small_shape(dtype=dtype, **kw), "unit", flags=flags)


def test_scan_many_short_sequences():
    """Many sequences of a few steps each: one block per (sequence, channel group), tiles mostly empty."""
    y, Y, hl, HL = run_scan(B=700, L=5, De=128, dtype="bf16", disc_mode=0, with_z=True, with_h0=True, with_D=True, seed=99100)
    assert_close(y, Y, TOL["bf16"], "scan y"); assert_close(hl, HL, 2e-3, "scan h_last")
    y, Y, hl, HL = run_scan(B=3, L=1, De=64, dtype="f32", disc_mode=1, with_z=False, with_h0=False, with_D=False, seed=99200)
    assert_close(y, Y, 1e-4, "scan y"); assert_close(hl, HL, 1e-4, "scan h_last")


def test_argument_errors_launch_nothing():
    s = small_shape()
    p = synth.make_inputs(s, recipe="unit")
    g = GpuLayer(s, p)
    bad = rb.config_from_shape(s)
    bad.K = s.E + 1
    assert rb.rom_layer_forward(bad, g.weights, g.dev["x"], g.out, None, None, None, g.ws, check=False) == -1
    bad = rb.config_from_shape(s); bad.d_state = 8
    assert rb.rom_layer_forward(bad, g.weights, g.dev["x"], g.out, None, None, None, g.ws, check=False) == -2
    bad = rb.config_from_shape(s); bad.small_proj_experts = 3
    assert rb.rom_layer_forward(bad, g.weights, g.dev["x"], g.out, None, None, None, g.ws, check=False) == -1
    small_ws = g.ws[:1024]
    assert rb.rom_layer_forward(g.cfg, g.weights, g.dev["x"], g.out, None, None, None, small_ws, check=False) == -3
    g.forward()                                       # nothing was enqueued by the rejected calls; the layer still runs


# ---------------------------------------------------------------------------------------------- debug checks, device-side timeout
def _status_detail(ws):
    v = ws[:12].view(torch.int32).cpu()
    return int(v[0]), int(v[1]), int(v[2])


@pytest.mark.parametrize("kw", [dict(), dict(E=8, K=1, B=3, L=130), dict(E=6, K=2, router_bias_scale=4.0, L=513)])
def test_debug_checks_pass_on_good_runs_and_change_nothing(kw):
    s = small_shape(**kw)
    p = synth.make_inputs(s, recipe="unit")
    plain = GpuLayer(s, p)
    want = plain.forward().clone()
    g = GpuLayer(s, p, flags=rb.ROM_FLAG_DEBUG_CHECKS)
    assert rb.workspace_size(g.cfg) > rb.workspace_size(plain.cfg)      # canaries between the sub-buffers
    got = g.forward()                                                     # asserts a clean status word
    assert torch.equal(got, want)
    n_debug = rb.last_launch_count()
    plain.forward()
    assert n_debug == rb.last_launch_count() + 3                          # canary write, table check, canary compare


def test_debug_checks_report_a_damaged_table_and_a_damaged_canary():
    """The damage is planted from the host into the workspace of a finished forward; the checks run again on demand."""
    s = small_shape(E=4, K=2, L=200)
    p = synth.make_inputs(s, recipe="unit")
    g = GpuLayer(s, p, flags=rb.ROM_FLAG_DEBUG_CHECKS)
    g.forward()
    roa = g.tap("row_of_assign", torch.int32, 1).view(-1)
    saved = roa[5].clone()
    roa[5] = 10 ** 6                                                      # a row far outside the padded range
    rb.rom_debug_check(g.cfg, g.ws)
    torch.cuda.synchronize()
    assert _status_detail(g.ws) == (-8, 10, 5)
    assert rb.rom_get_status(g.ws) == -8 and "debug check" in rb.status_string(-8)
    roa[5] = saved
    rb.rom_debug_check(g.cfg, g.ws)
    assert rb.rom_get_status(g.ws) == 0
    off, n = rb.workspace_find(g.cfg, "U")
    canary = (off + n + 255) // 256 * 256                                 # the canary that follows U
    g.ws[canary + 17] ^= 0xFF
    rb.rom_debug_check(g.cfg, g.ws)
    torch.cuda.synchronize()
    code, where, _ = _status_detail(g.ws)
    assert (code, where) == (-8, 20)
    assert rb.rom_get_status(g.ws) == -8
    g.forward()                                                           # canaries are rewritten by the next forward: clean again


def test_device_wait_that_runs_out_is_reported_and_the_workspace_stays_usable():
    """Fault injection on the host's request (ROM_FLAG_TEST_STALL): the producer of the first grouped projection never
    issues the copies of one operand stage, so the MMA issuer's bounded wait runs out; the kernel must latch
    ROM_ERR_DEVICE_TIMEOUT, wait for what it already issued, free its tensor memory and return; the launches after it
    still run (on unspecified data, with valid indices).  The next ordinary forward on the same workspace is checked
    against the oracle."""
    s = small_shape(E=4, K=1, B=2, L=300, d_model=256)
    p = synth.make_inputs(s, recipe="unit")
    g = GpuLayer(s, p, flags=rb.ROM_FLAG_TEST_STALL)
    rb.rom_layer_forward(g.cfg, g.weights, g.dev["x"], g.out, g.idx, g.gates, g.counts, g.ws)
    torch.cuda.synchronize()
    assert rb.rom_get_status(g.ws) == -6
    good = GpuLayer(s, p)
    good.ws = g.ws                                                        # same workspace, ordinary flags
    out = good.forward()
    ref, im = oracle_layer(s, p)
    np.testing.assert_array_equal(good.idx.cpu().numpy(), im["idx"])
    assert_close(np64(out), ref, TOL["bf16"], "out after a timed-out call")


# ---------------------------------------------------------------------------------------------- fused conv + x Proj + dt Proj
@pytest.mark.parametrize("kw", [
    dict(E=8, K=1, B=3, L=130),                                   # ragged last row tile, several sequences inside one tile
    dict(E=4, K=1, B=1, L=700, d_conv=3, dt_rank=32),
    dict(E=4, K=1, B=2, L=257, d_conv=2, dt_rank=64, d_inner=512),
    dict(E=2, K=1, B=5, L=33, dt_rank=128, d_inner=320),           # d_r = 128: two K blocks of the dt Proj; D_e not a multiple of 256
])
def test_fused_small_projections_match_the_three_launches_and_the_oracle(kw):
    """ROM_FLAG_FUSED_SMALL runs conv + x Proj + dt Proj as one tcgen05 kernel (top-1, tensor path); the default is three
    launches.  Both against the oracle (taps U, B, C, Delta and the output), and against each other."""
    s = small_shape(**kw)
    check_layer(s, "unit")
    check_layer(s, "unit", flags=rb.ROM_FLAG_FUSED_SMALL)
    p = synth.make_inputs(s, recipe="unit")
    a = GpuLayer(s, p, flags=rb.ROM_FLAG_FUSED_SMALL)
    out_a = a.forward().clone()
    n_fused = rb.last_launch_count()
    b = GpuLayer(s, p)
    out_b = b.forward()
    assert rb.last_launch_count() == n_fused + 2
    tdt = synth.torch_dtype(s)
    assert_close(np64(a.tap("U", tdt, s.d_inner)), np64(b.tap("U", tdt, s.d_inner)), 1e-2, "U fused vs unfused")
    assert_close(np64(a.tap("Delta", tdt, s.d_inner)), np64(b.tap("Delta", tdt, s.d_inner)), 1e-2, "Delta fused vs unfused")
    assert_close(np64(out_a), np64(out_b), 1e-2, "out fused vs unfused")


def test_fused_small_projections_small_bf16_config():
    check_layer(synth.CONFIGS["small_bf16"], "unit", with_D=False, flags=rb.ROM_FLAG_FUSED_SMALL)
