"""Seeded synthetic inputs for one Routing-Mamba (RoM) layer.

This module only draws random numbers and shapes them; it holds none of the
method's arithmetic.  Both the CPU oracle and the CUDA path are fed the very
same bits produced here (bf16/fp32 tensors; the oracle widens them exactly to
fp64).  The shapes are the layer widths of the paper's scaling table
(Appendix A.2, "Scaling Law Model Sizes"), with 8 experts / top-1 as in
Section 5; the value distributions are stated in `make_inputs`.

Importing this module does not load the CUDA library.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import torch


@dataclasses.dataclass(frozen=True)
class RomShape:
    """Problem statement of one RoM layer forward (Section 4.2 notation in comments)."""
    name: str
    B: int            # sequences
    L: int            # sequence length
    d_model: int      # D_m
    d_inner: int      # D_e
    d_state: int      # D_s
    d_conv: int       # k
    dt_rank: int      # d_r
    E: int            # number of experts N
    K: int            # top-K
    dtype: str        # "f32" | "bf16"  storage of x, weights, big intermediates
    seed_base: int    # tensor i is drawn with seed seed_base + i
    router_bias_scale: Optional[float] = None  # s in b_r[e] = -s * 1.2 * ln(e+1); None = no bias

    @property
    def T(self) -> int:
        return self.B * self.L

    def replace(self, **kw) -> "RomShape":
        return dataclasses.replace(self, **kw)


# The five seeded workloads.  `zipf` has no d_conv / dt_rank stated by its
# definition; k = 4 and d_r = d_model / 16 are the paper's values (Section 3.1).
# Its router_bias_scale was found once by bisection (with the CPU oracle's
# router) so that the busiest expert receives about 5x the mean load on the
# seeded input, then frozen here.
CONFIGS: Dict[str, RomShape] = {
    "tiny_fp32": RomShape("tiny_fp32", 1, 256, 256, 512, 16, 4, 16, 4, 1, "f32", 0),
    "small_bf16": RomShape("small_bf16", 4, 2048, 1024, 2048, 16, 4, 64, 8, 1, "bf16", 2000),
    "long_ctx": RomShape("long_ctx", 1, 16384, 2048, 4096, 16, 4, 128, 8, 1, "bf16", 3000),
    "zipf": RomShape("zipf", 8, 4096, 2048, 4096, 16, 4, 128, 16, 2, "bf16", 4000,
                     router_bias_scale=0.657),
    "short_seqs": RomShape("short_seqs", 64, 1024, 1536, 3072, 16, 4, 96, 8, 2, "bf16", 5000),
}

_TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}

# tensor ids (seed offsets); fixed so that adding a tensor never reshuffles the others
_TID = {"x": 1, "W_r": 2, "W_inz": 3, "w_conv": 4, "W_x": 5, "W_dt": 6, "W_out": 7, "b_dt": 8,
        "u": 11, "delta": 12, "Bm": 13, "Cm": 14, "z": 15, "h0": 16}


def torch_dtype(shape: RomShape) -> torch.dtype:
    return _TORCH_DTYPE[shape.dtype]


def _randn(seed: int, size, std: float = 1.0) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return torch.randn(size, generator=g, dtype=torch.float32) * std


def _rand(seed: int, size) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return torch.rand(size, generator=g, dtype=torch.float32)


def make_inputs(shape: RomShape, recipe: str = "paper", with_D: bool = True,
                routed_small: bool = False) -> Dict[str, Optional[torch.Tensor]]:
    """Draw x and every weight of one RoM layer on the CPU.

    recipe "paper": x ~ N(0,1); all projection / conv / router weights ~ N(0, 0.02^2);
        A[c,n] = -(n+1); D = 1; conv bias 0; dt bias = softplus^-1(dt0) with dt0
        log-uniform in [1e-3, 1e-1].
    recipe "unit": same draws rescaled so that every stage has O(1) outputs
        (projection std 1/sqrt(fan_in), conv taps std 0.5, router std 1/sqrt(D_m) * 2):
        with the 0.02 weights the state-space term is ~1e-4 of the D*u skip, so a
        parity test on that recipe alone would not see the scan.

    Storage dtype is the shape's dtype for x and the matrices; A, D and the biases are fp32.
    Layouts (row-major):
        x[B,L,D_m]  W_r[E,D_m]  W_inz[E,2*D_e,D_m] (rows [0,D_e) Conv Proj, [D_e,2D_e) Gate Proj)
        w_conv[k,D_e] (tap k-1 multiplies the current token)  W_x[R+2N, D_e] (rows delta|B|C)
        W_dt[D_e,R]  W_out[E,D_m,D_e]  A[D_e,N]  D[D_e]  b_conv[D_e]  b_dt[D_e]  b_r[E] or None
    routed_small: W_x[E, R+2N, D_e] and W_dt[E, D_e, R], one x Proj / dt Proj per expert (the
        ablation row of Section 5.3), same distributions.
    """
    s = shape
    dt = torch_dtype(s)
    R, N = s.dt_rank, s.d_state
    sb = s.seed_base
    if recipe == "paper":
        std = dict(W_r=0.02, W_inz=0.02, w_conv=0.02, W_x=0.02, W_dt=0.02, W_out=0.02)
    elif recipe == "unit":
        std = dict(W_r=2.0 / math.sqrt(s.d_model), W_inz=1.0 / math.sqrt(s.d_model), w_conv=0.5,
                   W_x=1.0 / math.sqrt(s.d_inner), W_dt=1.0 / math.sqrt(R),
                   W_out=1.0 / math.sqrt(s.d_inner))
    else:
        raise ValueError(f"unknown recipe {recipe!r}")

    out: Dict[str, Optional[torch.Tensor]] = {}
    out["x"] = _randn(sb + _TID["x"], (s.B, s.L, s.d_model)).to(dt)
    out["W_r"] = _randn(sb + _TID["W_r"], (s.E, s.d_model), std["W_r"]).to(dt)
    out["W_inz"] = _randn(sb + _TID["W_inz"], (s.E, 2 * s.d_inner, s.d_model), std["W_inz"]).to(dt)
    out["w_conv"] = _randn(sb + _TID["w_conv"], (s.d_conv, s.d_inner), std["w_conv"]).to(dt)
    lead = (s.E,) if routed_small else ()
    out["W_x"] = _randn(sb + _TID["W_x"], lead + (R + 2 * N, s.d_inner), std["W_x"]).to(dt)
    out["W_dt"] = _randn(sb + _TID["W_dt"], lead + (s.d_inner, R), std["W_dt"]).to(dt)
    out["W_out"] = _randn(sb + _TID["W_out"], (s.E, s.d_model, s.d_inner), std["W_out"]).to(dt)

    out["A"] = -(torch.arange(1, N + 1, dtype=torch.float32)).repeat(s.d_inner, 1).contiguous()
    out["D"] = torch.ones(s.d_inner, dtype=torch.float32) if with_D else None
    out["b_conv"] = torch.zeros(s.d_inner, dtype=torch.float32)
    # dt0 log-uniform in [1e-3, 1e-1]; stored as the pre-softplus bias: b = dt0 + log(1 - exp(-dt0))
    u01 = _rand(sb + _TID["b_dt"], (s.d_inner,)).double()
    dt0 = torch.exp(u01 * (math.log(1e-1) - math.log(1e-3)) + math.log(1e-3))
    out["b_dt"] = (dt0 + torch.log(-torch.expm1(-dt0))).float()
    if s.router_bias_scale is None:
        out["b_r"] = None
    else:
        e = torch.arange(s.E, dtype=torch.float64)
        out["b_r"] = (-s.router_bias_scale * 1.2 * torch.log(e + 1.0)).float()
    return out


def make_scan_inputs(B: int, L: int, d_inner: int, d_state: int, dtype: str, seed_base: int,
                     with_z: bool = True, with_h0: bool = False) -> Dict[str, Optional[torch.Tensor]]:
    """Direct inputs of the selective scan with O(1) magnitudes.

    u, z ~ N(0,1) in the storage dtype; delta log-uniform in [1e-3, 2e-1] (fp32);
    Bm, Cm ~ N(0,1) fp32; A[c,n] = -(n+1) * (0.5 + rand) (not an arithmetic
    progression, so nothing can exploit A's structure); D ~ N(0,1); h0 ~ N(0,1) if asked.
    """
    dt = _TORCH_DTYPE[dtype]
    sb = seed_base
    out: Dict[str, Optional[torch.Tensor]] = {}
    out["u"] = _randn(sb + _TID["u"], (B, L, d_inner)).to(dt)
    r = _rand(sb + _TID["delta"], (B, L, d_inner)).double()
    out["delta"] = torch.exp(r * (math.log(2e-1) - math.log(1e-3)) + math.log(1e-3)).float()
    out["Bm"] = _randn(sb + _TID["Bm"], (B, L, d_state))
    out["Cm"] = _randn(sb + _TID["Cm"], (B, L, d_state))
    n = torch.arange(1, d_state + 1, dtype=torch.float32)
    out["A"] = (-(n[None, :]) * (0.5 + _rand(sb + 20, (d_inner, d_state)))).contiguous()
    out["D"] = _randn(sb + 21, (d_inner,))
    out["z"] = _randn(sb + _TID["z"], (B, L, d_inner)).to(dt) if with_z else None
    out["h0"] = _randn(sb + _TID["h0"], (B, d_inner, d_state)) if with_h0 else None
    return out


def make_mamba2_inputs(shape: RomShape, headdim: int) -> Dict[str, Optional[torch.Tensor]]:
    """x and every weight of one RoM layer on a Mamba2-style block, O(1) outputs at every stage ("unit" scaling):
    projection std 1/sqrt(fan_in), conv taps std 0.5, router std 2/sqrt(D_m), A_h = -(0.5 + rand) * (1 + h mod 8),
    D ~ N(0,1), dt bias = softplus^-1(dt0) with dt0 log-uniform in [1e-3, 1e-1], norm weight 1 + 0.1 N(0,1).
    Layouts: W_in[E, 2 D_e + 2 N + heads, D_m] rows z | x | B | C | dt; w_conv[k, D_e + 2 N]; W_out[E, D_m, D_e]."""
    s = shape
    dt = torch_dtype(s)
    De, N, Dm = s.d_inner, s.d_state, s.d_model
    H = De // headdim
    W = 2 * De + 2 * N + H
    sb = s.seed_base + 300
    out: Dict[str, Optional[torch.Tensor]] = {}
    out["x"] = _randn(sb + 1, (s.B, s.L, Dm)).to(dt)
    out["W_r"] = _randn(sb + 2, (s.E, Dm), 2.0 / math.sqrt(Dm)).to(dt)
    out["W_in"] = _randn(sb + 3, (s.E, W, Dm), 1.0 / math.sqrt(Dm)).to(dt)
    out["w_conv"] = _randn(sb + 4, (s.d_conv, De + 2 * N), 0.5).to(dt)
    out["b_conv"] = _randn(sb + 5, (De + 2 * N,), 0.1)
    u01 = _rand(sb + 6, (H,)).double()
    dt0 = torch.exp(u01 * (math.log(1e-1) - math.log(1e-3)) + math.log(1e-3))
    out["dt_bias"] = (dt0 + torch.log(-torch.expm1(-dt0))).float()
    out["A"] = (-(0.5 + _rand(sb + 7, (H,))) * (1.0 + (torch.arange(H) % 8).float())).contiguous()
    out["D"] = _randn(sb + 8, (H,))
    out["w_norm"] = 1.0 + 0.1 * _randn(sb + 9, (De,))
    out["W_out"] = _randn(sb + 10, (s.E, Dm, De), 1.0 / math.sqrt(De)).to(dt)
    if s.router_bias_scale is None:
        out["b_r"] = None
    else:
        e = torch.arange(s.E, dtype=torch.float64)
        out["b_r"] = (-s.router_bias_scale * 1.2 * torch.log(e + 1.0)).float()
    return out
