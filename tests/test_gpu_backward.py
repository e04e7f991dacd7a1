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
