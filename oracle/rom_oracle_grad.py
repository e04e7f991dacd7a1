"""CPU oracle for the backward pass of one Routing-Mamba (RoM) layer.

TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64 numpy.  Every function here is the reverse of one
forward function of `rom_oracle.py` (same name + `_backward`), written out by the chain rule from
the forward definition: no automatic differentiation, no blocking, no fusion.  Only tests, the smoke
check and the benchmark's cpu-baseline leg may import this package; the CUDA path shares no code
with it.

What is differentiated (Section 5.1 trains the layer end to end; Appendix A.3 trains the router
through the gate): the layer output O of Section 4.2 with respect to the input X, every expert
matrix (Conv Proj | Gate Proj, Out Proj), the shared Conv1D, x Proj, dt Proj, A, D, the biases and the
router weights.  Readings taken where the paper is silent:
  * The top-K indicator 1[i in TopK(P)] is piecewise constant: it is held fixed, and the router
    receives gradient only through the gate values R_i = P_i (gate_mode 0) or P_i / sum of the
    selected P (gate_mode 1).  The Conv/Gate projections carry the indicator only (no gate), so
    they send nothing to the router.  Jitter noise and SparseMixer (Appendix A.3) are training-time
    stochastic estimators and stay out.
  * Only the shared x Proj / dt Proj wiring (Section 4.3) is differentiated here.

Pins (tests/test_oracle_grad_pins.py): central finite differences of the forward oracle on tiny
shapes for every tensor; E = K = 1 against torch.autograd on an independently written dense Mamba;
the adjoint identity <dY, scan(U)> = <scan_backward(dY).dU, U> (the scan is linear in U); K = E
with a zero router (uniform gates): all experts receive gate 1/E and db_r sums to zero; planted
mistakes fail the finite-difference pin.
"""
from __future__ import annotations

import numpy as np

from . import rom_oracle as F

F64 = np.float64


def sigmoid(v):
    v = np.asarray(v, dtype=F64)
    return 1.0 / (1.0 + np.exp(-v))


def silu_grad(v):
    """d/dv [v sigmoid(v)] = sigmoid(v) (1 + v (1 - sigmoid(v)))."""
    s = sigmoid(v)
    return s * (1.0 + np.asarray(v, dtype=F64) * (1.0 - s))


# --------------------------------------------------------------------------- S10/S11 reversed
def expert_out_proj_backward(dOut, Yg, W_out, idx, gate):
    """Reverse of O_t = sum_k gate[t,k] * W_out[idx[t,k]] Yg_t (Section 4.2, output equation).
    Returns dYg[T,D_e], dW_out[E,D_m,D_e], dgate[T,K]."""
    dOut = np.asarray(dOut, dtype=F64)
    Yg = np.asarray(Yg, dtype=F64)
    W_out = np.asarray(W_out, dtype=F64)
    T, De = Yg.shape
    E = W_out.shape[0]
    K = idx.shape[1]
    dYg = np.zeros((T, De), dtype=F64)
    dW_out = np.zeros_like(W_out)
    dgate = np.zeros((T, K), dtype=F64)
    for k in range(K):
        for e in range(E):
            tok = np.nonzero(idx[:, k] == e)[0]
            if tok.size == 0:
                continue
            back = dOut[tok] @ W_out[e]                     # W_out,e applied in reverse: [n, D_e]
            dYg[tok] += gate[tok, k][:, None] * back
            dgate[tok, k] = np.sum(back * Yg[tok], axis=1)
            dW_out[e] += (gate[tok, k][:, None] * dOut[tok]).T @ Yg[tok]
    return dYg, dW_out, dgate


def gated_backward(dYg, Y, Zpre):
    """Reverse of Yg = Y * SiLU(Zpre).  Returns dY, dZpre."""
    dYg = np.asarray(dYg, dtype=F64)
    return dYg * F.silu(Zpre), dYg * np.asarray(Y, dtype=F64) * silu_grad(Zpre)


# --------------------------------------------------------------------------- S7 reversed
def selective_scan_backward(dY, U, Delta, A, Bm, Cm, D=None, h0=None, disc_mode=0, dh_last=None):
    """Reverse of the recurrence of Section 3.1, h_t = A-bar_t h_{t-1} + B-bar_t U_t, Y_t = C_t h_t (+ D U_t).

    The forward states are recomputed and kept; then, walking t = L-1 .. 0 with
    g = dLoss/dh_t (all later steps already folded in):
        g      += C_t dY_t                      dC_t   = sum_c dY_t,c h_t,c
        dA-bar  = g h_{t-1}                     dB-bar = g U_t            dU_t = sum_n g B-bar
        with x = Delta A:  A-bar = exp(x);  zero-order hold B-bar = expm1(x)/A * B,  else B-bar = Delta B
        g      <- A-bar g                       (gradient w.r.t. h_{t-1})
    Returns dict(dU, dDelta, dA, dBm, dCm, dD, dh0).  dh_last: gradient arriving at the final state."""
    dY = np.asarray(dY, dtype=F64)
    U = np.asarray(U, dtype=F64)
    Delta = np.asarray(Delta, dtype=F64)
    A = np.asarray(A, dtype=F64)
    Bm = np.asarray(Bm, dtype=F64)
    Cm = np.asarray(Cm, dtype=F64)
    Bsz, L, De = U.shape
    N = A.shape[1]
    hs = np.zeros((L + 1, Bsz, De, N), dtype=F64)          # hs[t] = state before step t
    if h0 is not None:
        hs[0] = np.asarray(h0, dtype=F64)
    for t in range(L):
        x = Delta[:, t, :, None] * A[None]
        if disc_mode == 0:
            Bbar = np.expm1(x) / A[None] * Bm[:, t, None, :]
        else:
            Bbar = Delta[:, t, :, None] * Bm[:, t, None, :]
        hs[t + 1] = np.exp(x) * hs[t] + Bbar * U[:, t, :, None]
    dU = np.zeros_like(U)
    dDelta = np.zeros_like(Delta)
    dA = np.zeros_like(A)
    dBm = np.zeros_like(Bm)
    dCm = np.zeros_like(Cm)
    g = np.zeros((Bsz, De, N), dtype=F64) if dh_last is None else np.array(dh_last, dtype=F64)
    for t in range(L - 1, -1, -1):
        g = g + Cm[:, t, None, :] * dY[:, t, :, None]
        dCm[:, t, :] = np.sum(dY[:, t, :, None] * hs[t + 1], axis=1)
        x = Delta[:, t, :, None] * A[None]
        ex = np.exp(x)
        ut = U[:, t, :, None]
        bt = Bm[:, t, None, :]
        dx = g * hs[t] * ex                                 # through A-bar = exp(x)
        if disc_mode == 0:
            em1 = np.expm1(x)
            dx = dx + g * ut * bt * ex / A[None]            # through expm1(x)
            dA += np.sum(g * ut * bt * (-em1) / (A[None] ** 2), axis=0)
            dBm[:, t, :] = np.sum(g * ut * em1 / A[None], axis=1)
            dU[:, t, :] = np.sum(g * em1 / A[None] * bt, axis=2)
            dDelta[:, t, :] = np.sum(dx * A[None], axis=2)
        else:
            dl = Delta[:, t, :, None]
            dBm[:, t, :] = np.sum(g * ut * dl, axis=1)
            dU[:, t, :] = np.sum(g * dl * bt, axis=2)
            dDelta[:, t, :] = np.sum(dx * A[None], axis=2) + np.sum(g * ut * bt, axis=2)
        dA += np.sum(dx * Delta[:, t, :, None], axis=0)
        g = g * ex
    dD = None
    if D is not None:
        dU = dU + np.asarray(D, dtype=F64)[None, None, :] * dY
        dD = np.sum(dY * U, axis=(0, 1))
    return dict(dU=dU, dDelta=dDelta, dA=dA, dBm=dBm, dCm=dCm, dD=dD, dh0=g)


# --------------------------------------------------------------------------- S5/S6 reversed
def small_proj_backward(dBm, dCm, dDelta, U, W_x, W_dt, b_dt, dt_rank, d_state):
    """Reverse of (delta, B, C) = U W_x, Delta = softplus(delta W_dt + b_dt) (shared layers, Section 4.3).
    Returns dU[T,D_e] (the part through x Proj), dW_x, dW_dt, db_dt."""
    U = np.asarray(U, dtype=F64)
    W_x = np.asarray(W_x, dtype=F64)
    W_dt = np.asarray(W_dt, dtype=F64)
    R, N = dt_rank, d_state
    delta = U @ W_x[:R].T
    pre = delta @ W_dt.T
    if b_dt is not None:
        pre = pre + np.asarray(b_dt, dtype=F64)[None, :]
    dpre = np.asarray(dDelta, dtype=F64) * sigmoid(pre)     # softplus' = sigmoid
    dW_dt = dpre.T @ delta
    db_dt = np.sum(dpre, axis=0)
    ddelta = dpre @ W_dt
    dxdbl = np.concatenate([ddelta, np.asarray(dBm, dtype=F64), np.asarray(dCm, dtype=F64)], axis=1)
    return dxdbl @ W_x, dxdbl.T @ U, dW_dt, db_dt


# --------------------------------------------------------------------------- S4 reversed
def conv_silu_backward(dU, H, w_conv, b_conv=None):
    """Reverse of U = SiLU(b + sum_j w[j] H[t - (k-1-j)]) (causal depthwise conv, Section 3.1).
    Returns dH[B,L,D_e], dw_conv[k,D_e], db_conv[D_e]."""
    H = np.asarray(H, dtype=F64)
    w = np.asarray(w_conv, dtype=F64)
    Bsz, L, De = H.shape
    k = w.shape[0]
    pre = np.zeros((Bsz, L, De), dtype=F64)
    if b_conv is not None:
        pre += np.asarray(b_conv, dtype=F64)[None, None, :]
    for j in range(k):
        shift = (k - 1) - j
        if shift < L:
            pre[:, shift:, :] += w[j][None, None, :] * H[:, :L - shift, :]
    dpre = np.asarray(dU, dtype=F64) * silu_grad(pre)
    dH = np.zeros_like(H)
    dw = np.zeros_like(w)
    for j in range(k):
        shift = (k - 1) - j
        if shift < L:
            dH[:, :L - shift, :] += w[j][None, None, :] * dpre[:, shift:, :]
            dw[j] = np.sum(dpre[:, shift:, :] * H[:, :L - shift, :], axis=(0, 1))
    return dH, dw, np.sum(dpre, axis=(0, 1))


# --------------------------------------------------------------------------- S3 reversed
def expert_in_proj_backward(dH, dZ, x, W_inz, idx):
    """Reverse of H_t = sum_i 1_i X_t W_in,i, Z_t = sum_i 1_i X_t W_g,i (indicator only).
    Returns dx[T,D_m], dW_inz[E,2D_e,D_m]."""
    x = np.asarray(x, dtype=F64)
    W_inz = np.asarray(W_inz, dtype=F64)
    dHZ = np.concatenate([np.asarray(dH, dtype=F64), np.asarray(dZ, dtype=F64)], axis=1)
    E = W_inz.shape[0]
    dx = np.zeros_like(x)
    dW = np.zeros_like(W_inz)
    for k in range(idx.shape[1]):
        for e in range(E):
            tok = np.nonzero(idx[:, k] == e)[0]
            if tok.size == 0:
                continue
            dx[tok] += dHZ[tok] @ W_inz[e]
            dW[e] += dHZ[tok].T @ x[tok]
    return dx, dW


# --------------------------------------------------------------------------- S1 reversed
def route_backward(dgate, x, W_r, P, idx, gate, gate_mode=0):
    """Reverse of the gate values with the selected set held fixed: gate_mode 0, gate_k = P[idx_k];
    gate_mode 1, gate_k = P[idx_k] / sum_j P[idx_j]; P = softmax(x W_r^T + b_r).
    Returns dx[T,D_m], dW_r[E,D_m], db_r[E]."""
    x = np.asarray(x, dtype=F64)
    W_r = np.asarray(W_r, dtype=F64)
    P = np.asarray(P, dtype=F64)
    dgate = np.asarray(dgate, dtype=F64)
    T, E = P.shape
    rows = np.arange(T)
    dP = np.zeros((T, E), dtype=F64)
    if gate_mode == 0:
        dsel = dgate
    else:
        S = np.sum(P[rows[:, None], idx], axis=1, keepdims=True)
        dsel = (dgate - np.sum(dgate * gate, axis=1, keepdims=True)) / S
    for k in range(idx.shape[1]):
        np.add.at(dP, (rows, idx[:, k]), dsel[:, k])
    dlogit = P * (dP - np.sum(dP * P, axis=1, keepdims=True))
    return dlogit @ W_r, dlogit.T @ x, np.sum(dlogit, axis=0)


# --------------------------------------------------------------------------- the layer
def rom_layer_backward(dOut, x, W_r, b_r, W_inz, w_conv, b_conv, W_x, W_dt, b_dt, A, D, W_out,
                       K, dt_rank, gate_mode=0, disc_mode=0):
    """Gradients of sum(dOut * O) for the layer of `rom_oracle.rom_layer_forward` (shared small layers).
    Returns a dict: dx, dW_r, db_r, dW_inz, dw_conv, db_conv, dW_x, dW_dt, db_dt, dA, dD, dW_out."""
    x = np.asarray(x, dtype=F64)
    Bsz, L, Dm = x.shape
    T = Bsz * L
    xt = x.reshape(T, Dm)
    A = np.asarray(A, dtype=F64)
    N = A.shape[1]
    _, im = F.rom_layer_forward(x, W_r, b_r, W_inz, w_conv, b_conv, W_x, W_dt, b_dt, A, D, W_out, K, dt_rank,
                                gate_mode, disc_mode, return_intermediates=True)
    idx, gate = im["idx"], im["gate"]
    De = im["H"].shape[1]
    dYg, dW_out, dgate = expert_out_proj_backward(np.asarray(dOut, dtype=F64).reshape(T, Dm), im["Yg"], W_out, idx, gate)
    dY, dZpre = gated_backward(dYg, im["Y"], im["Zpre"])
    sc = selective_scan_backward(dY.reshape(Bsz, L, De), im["U"].reshape(Bsz, L, De), im["Delta"].reshape(Bsz, L, De), A,
                                 im["Bm"].reshape(Bsz, L, N), im["Cm"].reshape(Bsz, L, N), D, None, disc_mode)
    dU_x, dW_x, dW_dt, db_dt = small_proj_backward(sc["dBm"].reshape(T, N), sc["dCm"].reshape(T, N), sc["dDelta"].reshape(T, De),
                                                   im["U"], W_x, W_dt, b_dt, dt_rank, N)
    dU = sc["dU"].reshape(T, De) + dU_x
    dH, dw_conv, db_conv = conv_silu_backward(dU.reshape(Bsz, L, De), im["H"].reshape(Bsz, L, De), w_conv, b_conv)
    dx_in, dW_inz = expert_in_proj_backward(dH.reshape(T, De), dZpre, xt, W_inz, idx)
    dx_r, dW_r, db_r = route_backward(dgate, xt, W_r, im["P"], idx, gate, gate_mode)
    return dict(dx=(dx_in + dx_r).reshape(Bsz, L, Dm), dW_r=dW_r, db_r=db_r, dW_inz=dW_inz, dw_conv=dw_conv, db_conv=db_conv,
                dW_x=dW_x, dW_dt=dW_dt, db_dt=db_dt, dA=sc["dA"], dD=sc["dD"], dW_out=dW_out)
