"""Helpers shared by the parity tests: run the CUDA path through the C ABI binding, run the CPU
oracle on the same seeded inputs, compare.  (Test infrastructure; not part of the product.)"""
from __future__ import annotations

import numpy as np
import torch

from oracle import rom_oracle as O
from paper_2506_18145_b200 import binding as rb
from paper_2506_18145_b200 import synth

TOL = {"f32": 1e-4, "bf16": 2e-2}     # relative tolerances of the fp32 and bf16 paths


def np64(t):
    return None if t is None else t.detach().cpu().double().numpy()


def rel_errors(got, ref):
    """(max-norm relative, 2-norm relative) of got vs ref, both numpy float64."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    d = got - ref
    mx = float(np.max(np.abs(ref)))
    n2 = float(np.linalg.norm(ref.ravel()))
    return (float(np.max(np.abs(d))) / mx if mx > 0 else float(np.max(np.abs(d))),
            float(np.linalg.norm(d.ravel())) / n2 if n2 > 0 else float(np.linalg.norm(d.ravel())))


def assert_close(got, ref, tol, what=""):
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    e_max, e_2 = rel_errors(got, ref)
    assert e_max <= tol and e_2 <= tol, f"{what}: rel err max-norm {e_max:.3e}, 2-norm {e_2:.3e} > {tol:g}"
    return e_max, e_2


def oracle_layer(shape, p, gate_mode=0, disc_mode=0, intermediates=True):
    return O.rom_layer_forward(np64(p["x"]), np64(p["W_r"]), np64(p["b_r"]), np64(p["W_inz"]), np64(p["w_conv"]),
                               np64(p["b_conv"]), np64(p["W_x"]), np64(p["W_dt"]), np64(p["b_dt"]), np64(p["A"]),
                               np64(p["D"]), np64(p["W_out"]), K=shape.K, dt_rank=shape.dt_rank, gate_mode=gate_mode,
                               disc_mode=disc_mode, return_intermediates=intermediates)


class GpuLayer:
    """One configured layer on the GPU: weights resident, workspace allocated, forward through the C ABI."""

    def __init__(self, shape, p, gate_mode=0, disc_mode=0, flags=0, device="cuda"):
        self.shape = shape
        # three-dimensional W_x: one x Proj / dt Proj per expert
        self.cfg = rb.config_from_shape(shape, gate_mode, disc_mode, flags, shape.E if p["W_x"].dim() == 3 else 0)
        self.dev = {k: (None if v is None else v.to(device).contiguous()) for k, v in p.items()}
        self.weights = rb.make_weights(self.dev)
        self.ws = rb.alloc_workspace(self.cfg, device)
        T = shape.T
        self.out = torch.empty((shape.B, shape.L, shape.d_model), dtype=synth.torch_dtype(shape), device=device)
        self.idx = torch.empty((T, shape.K), dtype=torch.int32, device=device)
        self.gates = torch.empty((T, shape.K), dtype=torch.float32, device=device)
        self.counts = torch.empty((shape.E,), dtype=torch.int32, device=device)

    def forward(self, x=None):
        rb.rom_layer_forward(self.cfg, self.weights, self.dev["x"] if x is None else x, self.out, self.idx, self.gates,
                             self.counts, self.ws)
        torch.cuda.synchronize()
        code = rb.rom_get_status(self.ws)
        assert code == 0, rb.status_string(code)
        return self.out

    def tap(self, name, dtype, cols):
        off, nbytes = rb.workspace_find(self.cfg, name)
        return self.ws[off:off + nbytes].view(dtype).view(-1, cols)


def gpu_route(shape, p, gate_mode=0, device="cuda"):
    cfg = rb.config_from_shape(shape, gate_mode)
    T, K, E = shape.T, shape.K, shape.E
    ws = rb.alloc_workspace(cfg, device)
    idx = torch.empty((T, K), dtype=torch.int32, device=device)
    gates = torch.empty((T, K), dtype=torch.float32, device=device)
    counts = torch.empty((E,), dtype=torch.int32, device=device)
    offsets = torch.empty((E + 1,), dtype=torch.int32, device=device)
    perm = torch.empty((T * K,), dtype=torch.int32, device=device)
    inv = torch.empty((T * K,), dtype=torch.int32, device=device)
    b_r = None if p["b_r"] is None else p["b_r"].to(device)
    rb.rom_route(cfg, p["x"].to(device), p["W_r"].to(device), b_r, idx, gates, counts, offsets, perm, inv, ws)
    torch.cuda.synchronize()
    return dict(idx=idx.cpu().numpy(), gates=gates.cpu().numpy(), counts=counts.cpu().numpy(),
                offsets=offsets.cpu().numpy(), perm=perm.cpu().numpy(), inv_perm=inv.cpu().numpy())


def top_k_margin(logit, idx):
    """min over tokens of (last selected logit - best unselected logit) / max|logit|, ignoring exact ties; inf if K = E."""
    T, E = logit.shape
    if idx.shape[1] >= E:
        return float("inf")
    sel = np.zeros((T, E), dtype=bool)
    sel[np.arange(T)[:, None], idx] = True
    lo = np.where(sel, logit, np.inf).min(axis=1)
    hi = np.where(sel, -np.inf, logit).max(axis=1)
    gap = (lo - hi) / np.maximum(np.abs(logit).max(axis=1), 1e-300)
    gap = gap[gap > 0]
    return float(gap.min()) if gap.size else float("inf")


def check_route_exact(got, shape, p, gate_mode=0):
    x = np64(p["x"]).reshape(shape.T, shape.d_model)
    idx, gate, P, logit = O.route(x, np64(p["W_r"]), np64(p["b_r"]), shape.K, gate_mode)
    counts, offsets, perm, inv = O.permutation_tables(idx, shape.E)
    # smallest relative gap between the K-th selected logit and the best unselected one (exact ties aside): the GPU adds the
    # exact fp64 products in another order than the oracle, so a gap near 1e-16 would explain a flipped index, a larger one would not
    margin = top_k_margin(logit, idx)
    np.testing.assert_array_equal(got["idx"], idx, err_msg=f"smallest non-zero top-K boundary margin of the oracle's logits: {margin:.3e}")
    np.testing.assert_array_equal(got["counts"], counts)
    np.testing.assert_array_equal(got["offsets"], offsets)
    np.testing.assert_array_equal(got["perm"], perm)
    np.testing.assert_array_equal(got["inv_perm"], inv)
    np.testing.assert_allclose(got["gates"], gate, rtol=2e-6, atol=1e-30)
    return idx, gate
