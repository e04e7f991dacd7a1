"""Parity of the backward kernels (called through the C ABI) against the CPU fp64 backward oracle on the same seeded
inputs: 1e-4 (fp32 storage) / 2e-2 (bf16 storage) relative, in max-norm and 2-norm, per gradient tensor."""
import numpy as np
import pytest
import torch

from oracle import rom_oracle as O
from oracle import rom_oracle_grad as G
from paper_2506_18145_b200 import binding as rb
from paper_2506_18145_b200 import synth

from rom_testlib import TOL, assert_close, np64

pytestmark = pytest.mark.gpu


def run_scan_backward(B, L, De, dtype, disc_mode, with_z, with_h0, with_D, with_dh, seed):
    q = synth.make_scan_inputs(B, L, De, 16, dtype, seed, with_z=with_z, with_h0=with_h0)
    if not with_D:
        q["D"] = None
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    g = torch.Generator().manual_seed(seed + 77)
    dy = torch.randn((B, L, De), generator=g).to(tdt)
    dh = torch.randn((B, De, 16), generator=g) if with_dh else None
    cfg = rb.make_config(B, L, 64, De, 16, 4, 16, 1, 1, dtype, 0, disc_mode)
    d = {k: (None if v is None else v.cuda()) for k, v in q.items()}
    f32 = lambda *s: torch.empty(s, dtype=torch.float32, device="cuda")
    out = dict(du=torch.empty_like(d["u"]), ddelta=f32(B, L, De), dA=f32(De, 16), dBm=f32(B, L, 16), dCm=f32(B, L, 16),
               dD=f32(De) if with_D else None, dz=torch.empty_like(d["u"]) if with_z else None, dh0=f32(B, De, 16))
    ws = torch.empty(rb.scan_backward_workspace_size(cfg), dtype=torch.uint8, device="cuda")
    rb.rom_scan_backward(cfg, dy.cuda(), d["u"], d["delta"], d["A"], d["Bm"], d["Cm"], d["D"], d["z"], d["h0"],
                         None if dh is None else dh.cuda(), out["du"], out["ddelta"], out["dA"], out["dBm"], out["dCm"], out["dD"],
                         out["dz"], out["dh0"], ws)
    torch.cuda.synchronize()
    # oracle: gradient arriving at the pre-gate scan output, then the reverse recurrence
    dYg = np64(dy)
    if with_z:
        Y, _ = O.selective_scan(np64(q["u"]), np64(q["delta"]), np64(q["A"]), np64(q["Bm"]), np64(q["Cm"]), np64(q["D"]),
                                np64(q["h0"]), disc_mode)
        dY, dZ = G.gated_backward(dYg, Y, np64(q["z"]))
    else:
        dY, dZ = dYg, None
    ref = G.selective_scan_backward(dY, np64(q["u"]), np64(q["delta"]), np64(q["A"]), np64(q["Bm"]), np64(q["Cm"]), np64(q["D"]),
                                    np64(q["h0"]), disc_mode, dh_last=np64(dh))
    ref["dz"] = dZ
    tol = TOL[dtype]
    for name in ("dU", "dDelta", "dA", "dBm", "dCm", "dD", "dz", "dh0"):
        got = out[{"dU": "du", "dDelta": "ddelta"}.get(name, name)]
        if got is None:
            continue
        assert_close(np64(got), ref[name], tol, f"scan backward {name}")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("disc_mode", [0, 1])
@pytest.mark.parametrize("B,L,De,with_z,with_h0,with_D,with_dh", [
    (2, 100, 192, True, False, True, False),     # ragged last chunk of steps, gate, skip
    (1, 333, 64, False, True, False, True),      # no gate, initial state, gradient arriving at the final state
    (3, 1, 128, True, True, True, True),         # a single step
    (1, 1024, 256, True, False, True, False),    # 32 chunks
])
def test_scan_backward_parity(dtype, disc_mode, B, L, De, with_z, with_h0, with_D, with_dh):
    run_scan_backward(B, L, De, dtype, disc_mode, with_z, with_h0, with_D, with_dh, seed=9900 + L)


def test_scan_backward_small_bf16_config_size():
    s = synth.CONFIGS["small_bf16"]
    run_scan_backward(s.B, s.L, s.d_inner, "bf16", 0, True, False, True, False, seed=9990)


def test_scan_backward_argument_errors():
    cfg = rb.make_config(1, 64, 64, 64, 16, 4, 16, 1, 1, "f32")
    t = torch.zeros(64 * 64, device="cuda")
    ws = torch.empty(rb.scan_backward_workspace_size(cfg), dtype=torch.uint8, device="cuda")
    args = [t] * 6 + [None, None, None, None] + [t] * 5 + [None, None, None]
    assert rb.rom_scan_backward(cfg, *args, ws, check=False) == 0
    bad = list(args); bad[6] = t                   # D without dD
    assert rb.rom_scan_backward(cfg, *bad, ws, check=False) == -1
    assert rb.rom_scan_backward(cfg, *args, ws[:64], check=False) == -3


# ---------------------------------------------------------------------------------------------- the whole layer
GRAD_NAMES = ("dW_r", "db_r", "dW_inz", "dw_conv", "db_conv", "dW_x", "dW_dt", "db_dt", "dA", "dD", "dW_out")


def run_layer_backward(s, recipe="unit", gate_mode=0, disc_mode=0, flags=0, with_D=True, seed=4242):
    p = synth.make_inputs(s, recipe=recipe, with_D=with_D)
    tdt = synth.torch_dtype(s)
    g = torch.Generator().manual_seed(seed)
    dout = torch.randn(p["x"].shape, generator=g).to(tdt)
    cfg = rb.config_from_shape(s, gate_mode, disc_mode, flags)
    dev = {k: (None if v is None else v.cuda().contiguous()) for k, v in p.items()}
    weights = rb.make_weights(dev)
    grads = {n: torch.empty(p[n[1:]].shape, dtype=torch.float32, device="cuda") for n in GRAD_NAMES if p.get(n[1:]) is not None}
    if "db_r" not in grads:                       # no router bias in the forward: its gradient is still defined, ask for it
        grads["db_r"] = torch.empty((s.E,), dtype=torch.float32, device="cuda")
    dx = torch.empty_like(dev["x"])
    ws = torch.empty(rb.layer_backward_workspace_size(cfg), dtype=torch.uint8, device="cuda")
    rb.rom_layer_backward(cfg, weights, dev["x"], dout.cuda(), dx, rb.make_grads(grads), ws)
    torch.cuda.synchronize()
    assert rb.rom_get_status(ws) == 0
    f = lambda v: None if v is None else np64(v)
    ref = G.rom_layer_backward(f(dout), f(p["x"]), f(p["W_r"]), f(p["b_r"]), f(p["W_inz"]), f(p["w_conv"]), f(p["b_conv"]), f(p["W_x"]),
                               f(p["W_dt"]), f(p["b_dt"]), f(p["A"]), f(p["D"]), f(p["W_out"]), K=s.K, dt_rank=s.dt_rank,
                               gate_mode=gate_mode, disc_mode=disc_mode)
    tol = TOL[s.dtype]
    assert_close(np64(dx), ref["dx"], tol, "dx")
    for n, t in grads.items():
        assert_close(np64(t), ref[n], tol, n)


def bshape(**kw):
    base = dict(name="b", B=2, L=150, d_model=128, d_inner=256, d_state=16, d_conv=4, dt_rank=16, E=4, K=2, dtype="bf16", seed_base=66000)
    base.update(kw)
    return synth.RomShape(**base)


@pytest.mark.parametrize("kw", [
    dict(),                                              # top-2, ragged L
    dict(E=8, K=1, B=3, L=130),                          # top-1
    dict(E=3, K=3, L=64, d_conv=3),
    dict(E=6, K=2, router_bias_scale=2.0, L=257, d_conv=2, dt_rank=32),
])
@pytest.mark.parametrize("dtype,flags", [("f32", 0), ("bf16", rb.ROM_FLAG_SIMT_GEMM), ("bf16", 0)])
def test_layer_backward_parity(kw, dtype, flags):
    run_layer_backward(bshape(dtype=dtype, **kw), flags=flags)


@pytest.mark.parametrize("gate_mode,disc_mode", [(1, 0), (0, 1), (1, 1)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_layer_backward_modes(gate_mode, disc_mode, dtype):
    run_layer_backward(bshape(dtype=dtype, L=200), gate_mode=gate_mode, disc_mode=disc_mode)


def test_layer_backward_without_skip_and_single_expert():
    run_layer_backward(bshape(E=1, K=1, L=96, dtype="f32"), with_D=False)


def test_layer_backward_small_bf16_config():
    """The small bf16 configuration (B=4, L=2048, d_model=1024, d_inner=2048, 8 experts, top-1) on the tensor path."""
    run_layer_backward(synth.CONFIGS["small_bf16"])
