"""Parity of RoM on a Mamba2-style block (rom_mamba2_layer_forward, through the C ABI) against its CPU fp64 oracle on the same
seeded inputs: routing bit-exact, outputs within 1e-4 (fp32) / 2e-2 (bf16) in max-norm and 2-norm."""
import numpy as np
import pytest
import torch

from oracle import rom_mamba2_oracle as M
from paper_2506_18145_b200 import binding as rb
from paper_2506_18145_b200 import synth

from rom_testlib import TOL, assert_close, np64

pytestmark = pytest.mark.gpu


def run_mamba2(s, headdim, flags=0, gate_mode=0):
    p = synth.make_mamba2_inputs(s, headdim)
    cfg = rb.config_from_shape(s, gate_mode, 0, flags)
    dev = {k: (None if v is None else v.cuda().contiguous()) for k, v in p.items()}
    ws = torch.empty(rb.mamba2_workspace_size(cfg, headdim), dtype=torch.uint8, device="cuda")
    out = torch.empty_like(dev["x"])
    idx = torch.empty((s.T, s.K), dtype=torch.int32, device="cuda")
    gates = torch.empty((s.T, s.K), dtype=torch.float32, device="cuda")
    counts = torch.empty((s.E,), dtype=torch.int32, device="cuda")
    rb.rom_mamba2_layer_forward(cfg, headdim, rb.make_mamba2_weights(dev), dev["x"], out, idx, gates, counts, ws)
    torch.cuda.synchronize()
    assert rb.rom_get_status(ws) == 0
    f = lambda v: None if v is None else np64(v)
    ref, im = M.rom_mamba2_forward(f(p["x"]), f(p["W_r"]), f(p["b_r"]), f(p["W_in"]), f(p["w_conv"]), f(p["b_conv"]), f(p["dt_bias"]),
                                   f(p["A"]), f(p["D"]), f(p["w_norm"]), f(p["W_out"]), K=s.K, headdim=headdim, d_state=s.d_state,
                                   gate_mode=gate_mode, return_intermediates=True)
    np.testing.assert_array_equal(idx.cpu().numpy(), im["idx"])
    np.testing.assert_array_equal(counts.cpu().numpy(), im["counts"])
    np.testing.assert_allclose(gates.cpu().numpy(), im["gate"], rtol=2e-6)
    assert_close(np64(out), ref, TOL[s.dtype], "out")


def m2shape(**kw):
    base = dict(name="m2", B=2, L=150, d_model=128, d_inner=256, d_state=16, d_conv=4, dt_rank=16, E=4, K=2, dtype="bf16", seed_base=55000)
    base.update(kw)
    return synth.RomShape(**base)


@pytest.mark.parametrize("kw,headdim", [
    (dict(), 32),                                            # top-2, ragged L, 8 heads
    (dict(E=8, K=1, B=3, L=130), 16),                        # top-1: gate and token order fused into the output projection
    (dict(E=3, K=3, L=64, d_conv=3), 32),
    (dict(E=6, K=2, router_bias_scale=2.0, L=513, d_conv=2), 32),
    (dict(E=4, K=1, B=1, L=1), 32),                          # one token
])
@pytest.mark.parametrize("dtype,flags", [("f32", 0), ("bf16", rb.ROM_FLAG_SIMT_GEMM), ("bf16", 0)])
def test_mamba2_layer_parity(kw, headdim, dtype, flags):
    run_mamba2(m2shape(dtype=dtype, **kw), headdim, flags)


def test_mamba2_layer_gate_mode_1():
    run_mamba2(m2shape(L=200), 32, gate_mode=1)


def test_mamba2_layer_small_bf16_widths():
    """The small bf16 configuration's sizes (B=4, L=2048, d_model=1024, d_inner=2048, 8 experts, top-1), headdim 64."""
    run_mamba2(synth.CONFIGS["small_bf16"], 64)


def test_mamba2_argument_errors():
    s = m2shape()
    cfg = rb.config_from_shape(s)
    with pytest.raises(rb.RomError):
        rb.mamba2_workspace_size(cfg, 48)              # d_inner not a multiple of headdim
    with pytest.raises(rb.RomError):
        rb.mamba2_workspace_size(cfg, 64)              # 4 heads: not a multiple of 8
