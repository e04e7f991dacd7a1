"""CPU oracle for Routing Mamba (RoM) applied to a Mamba2-style block.

TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64 numpy, one function per step; shares no code with the
CUDA path.  Only tests, the smoke check and the benchmark's cpu-baseline leg may import this package.

What the paper says (Section 5.2, "RoM on other linear recurrent architectures"; Section 5.4, first insight;
Appendix A.2, last sentence on the architecture figure): RoM is deployed on Mamba2 "following the same logic"
as on Mamba, and for blocks with a unified design the best results come from turning ALL major projection
layers of the block into experts under the one shared routing decision.  It prints no equations for this
variant, so the block is the Mamba2 block as published (Dao & Gu, 2024, one B/C group) and the reading is:

  * one router per layer, P = softmax(X W_r), top-K, gates R_i exactly as in `rom_oracle.route`;
  * the fused input projection is per expert, indicator-only sum as for H_t and G in Section 4.2:
        [z | x | B | C | dt]_t = sum_i 1_i X_t W_in,i        (widths D_e | D_e | N | N | heads)
  * shared by all experts: the causal depthwise conv + SiLU over the (x, B, C) channels, the per-head scalars
    A_h < 0, D_h, the dt bias, and the weight of the gated RMS norm;
  * per head h (P = headdim channels, state N), with dt_t,h = softplus(dt_raw + dt_bias_h), a_t = exp(dt_t,h A_h):
        H_t = a_t H_{t-1} + dt_t,h x_t,(h,:) (x) B_t ,   y_t,(h,p) = sum_n C_t,n H_t[p,n] + D_h x_t,(h,p)
  * gated norm: g = y * SiLU(z);  y^ = g / sqrt(mean_c g_c^2 + eps) * w_norm   (eps = 1e-5)
  * the output projection is per expert and carries the gate:  O_t = sum_i R_i y^_t W_out,i.

Pins (tests/test_oracle_mamba2_pins.py): E = K = 1 against an independently typed dense Mamba2 block whose
state-space part is the quadratic (attention-like) dual form, not a recurrence; the recurrence against the
brute-force unrolled sum; the norm against the library RMS norm; K = E uniform gates = the dense block on
summed input / mean output experts; batch-permutation invariance; a constant-input geometric series.
"""
from __future__ import annotations

import numpy as np

from . import rom_oracle as R

F64 = np.float64


def split_widths(d_inner, d_state, headdim):
    """(z, x, B, C, dt) column widths of the fused input projection."""
    return d_inner, d_inner, d_state, d_state, d_inner // headdim


def expert_in_proj(x, W_in, idx):
    """ZXBCDT_t = sum_i 1_i X_t W_in,i  (indicator only).  x[T,D_m]; W_in[E, W, D_m]; idx[T,K]."""
    x = np.asarray(x, dtype=F64)
    W_in = np.asarray(W_in, dtype=F64)
    T = x.shape[0]
    E, W, _ = W_in.shape
    out = np.zeros((T, W), dtype=F64)
    for k in range(idx.shape[1]):
        for e in range(E):
            tok = np.nonzero(idx[:, k] == e)[0]
            if tok.size:
                out[tok] += x[tok] @ W_in[e].T
    return out


def conv_silu(V, w_conv, b_conv=None):
    """SiLU of the causal depthwise conv over the sequence; V[B,L,C], w_conv[k,C], tap k-1 on the current token."""
    return R.conv_silu(V, w_conv, b_conv)


def ssd_scan(xh, dt, A, Bm, Cm, D=None, h0=None):
    """Scalar-decay state-space recurrence of a Mamba2 block, one scalar A per head.
    xh[B,L,H,P]; dt[B,L,H] (after softplus); A[H] (negative); Bm, Cm[B,L,N]; D[H] or None; h0[B,H,P,N] or None.
    Returns y[B,L,H,P], h_last[B,H,P,N]."""
    xh = np.asarray(xh, dtype=F64)
    dt = np.asarray(dt, dtype=F64)
    A = np.asarray(A, dtype=F64)
    Bm = np.asarray(Bm, dtype=F64)
    Cm = np.asarray(Cm, dtype=F64)
    Bsz, L, H, P = xh.shape
    N = Bm.shape[2]
    h = np.zeros((Bsz, H, P, N), dtype=F64) if h0 is None else np.array(h0, dtype=F64)
    y = np.zeros_like(xh)
    for t in range(L):
        a = np.exp(dt[:, t, :] * A[None, :])                                   # [B,H]
        upd = (dt[:, t, :, None] * xh[:, t])[:, :, :, None] * Bm[:, t, None, None, :]   # dt x (x) B
        h = a[:, :, None, None] * h + upd
        y[:, t] = np.sum(h * Cm[:, t, None, None, :], axis=3)
    if D is not None:
        y = y + np.asarray(D, dtype=F64)[None, None, :, None] * xh
    return y, h


def gated_rmsnorm(y, z, w_norm, eps=1e-5):
    """y^ = g / sqrt(mean_c g_c^2 + eps) * w_norm with g = y * SiLU(z); rows are tokens."""
    g = np.asarray(y, dtype=F64) * R.silu(z)
    ms = np.mean(g * g, axis=-1, keepdims=True)
    return g / np.sqrt(ms + eps) * np.asarray(w_norm, dtype=F64)


def rom_mamba2_forward(x, W_r, b_r, W_in, w_conv, b_conv, dt_bias, A, D, w_norm, W_out, K, headdim, d_state,
                       gate_mode=0, return_intermediates=False):
    """Forward of one RoM layer on a Mamba2-style block (reading in the module docstring).
    x[B,L,D_m]; W_in[E, 2D_e+2N+H, D_m]; w_conv[k, D_e+2N]; dt_bias, A, D [H]; w_norm[D_e]; W_out[E,D_m,D_e]."""
    x = np.asarray(x, dtype=F64)
    Bsz, L, Dm = x.shape
    T = Bsz * L
    xt = x.reshape(T, Dm)
    E = np.asarray(W_r).shape[0]
    De = np.asarray(W_out).shape[2]
    N = d_state
    H = De // headdim
    idx, gate, P, logit = R.route(xt, W_r, b_r, K, gate_mode)
    counts, offsets, perm, inv = R.permutation_tables(idx, E)
    zx = expert_in_proj(xt, W_in, idx)
    z = zx[:, :De]
    xbc = conv_silu(zx[:, De:2 * De + 2 * N].reshape(Bsz, L, De + 2 * N), w_conv, b_conv)
    xs, Bm, Cm = xbc[..., :De], xbc[..., De:De + N], xbc[..., De + N:]
    dt_raw = zx[:, 2 * De + 2 * N:].reshape(Bsz, L, H)
    dt = R.softplus(dt_raw + (0.0 if dt_bias is None else np.asarray(dt_bias, dtype=F64)[None, None, :]))
    y, h_last = ssd_scan(xs.reshape(Bsz, L, H, headdim), dt, A, Bm, Cm, D)
    yn = gated_rmsnorm(y.reshape(T, De), z, w_norm)
    out = R.expert_out_proj(yn, W_out, idx, gate).reshape(Bsz, L, Dm)
    if not return_intermediates:
        return out
    return out, dict(idx=idx, gate=gate, counts=counts, offsets=offsets, perm=perm, inv_perm=inv, zx=zx,
                     xs=xs.reshape(T, De), Bm=Bm.reshape(T, N), Cm=Cm.reshape(T, N), dt=dt.reshape(T, H),
                     y=y.reshape(T, De), yn=yn, h_last=h_last)
