"""Pins of the backward oracle (oracle/rom_oracle_grad.py) against things other than itself: central finite
differences of the forward oracle, torch.autograd on an independently written dense Mamba layer, the adjoint
identity of the scan, closed-form special cases, and planted mistakes.  CPU only."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import rom_oracle as O
from oracle import rom_oracle_grad as G

from test_oracle_pins import small_layer

NAMES = ("x", "W_r", "b_r", "W_inz", "w_conv", "b_conv", "W_x", "W_dt", "b_dt", "A", "D", "W_out")
GRAD_OF = {n: "d" + n for n in NAMES}


def layer_args(p):
    return [p[n] for n in NAMES]


def forward(p, K, R, **kw):
    return O.rom_layer_forward(*layer_args(p), K=K, dt_rank=R, **kw)


def backward(dOut, p, K, R, **kw):
    return G.rom_layer_backward(dOut, *layer_args(p), K=K, dt_rank=R, **kw)


def case(seed, **kw):
    p, s = small_layer(seed, **kw)
    g = np.random.default_rng(seed + 1000)
    p["b_r"] = g.normal(size=(s["E"],)) * 0.3
    dOut = g.normal(size=p["x"].shape)
    return p, s, dOut


# ------------------------------------------------------------------------------------------ finite differences
@pytest.mark.parametrize("K,gate_mode,disc_mode", [(1, 0, 0), (2, 0, 0), (2, 1, 0), (2, 0, 1), (3, 1, 1)])
def test_layer_gradients_match_central_differences(K, gate_mode, disc_mode):
    """For every tensor, the directional derivative of loss = sum(dOut * O) along a random direction, taken by
    central differences of the forward oracle, equals <gradient, direction>.  The step is small enough that no
    top-K decision flips (checked), so the piecewise-constant indicator does not enter."""
    p, s, dOut = case(11 + K, B=2, L=9, Dm=6, De=8, N=3, k=4, R=2, E=3)
    kw = dict(gate_mode=gate_mode, disc_mode=disc_mode)
    grads = backward(dOut, p, K, s["R"], **kw)
    _, im0 = forward(p, K, s["R"], return_intermediates=True, **kw)
    g = np.random.default_rng(5)
    eps = 1e-6
    for n in NAMES:
        d = g.normal(size=np.shape(p[n]))
        outs = []
        for sgn in (+1, -1):
            q = dict(p)
            q[n] = p[n] + sgn * eps * d
            o, im = forward(q, K, s["R"], return_intermediates=True, **kw)
            assert np.array_equal(im["idx"], im0["idx"])
            outs.append(np.sum(dOut * o))
        fd = (outs[0] - outs[1]) / (2 * eps)
        an = float(np.sum(grads[GRAD_OF[n]] * d))
        assert abs(fd - an) <= 2e-6 * max(1.0, abs(fd)), (n, fd, an)


def test_every_entry_of_small_tensors_by_central_differences():
    """Entry-by-entry check (not only a random direction) of the tensors where an index mistake would hide in a
    projection: conv taps, A, D, the biases and the router."""
    p, s, dOut = case(21, B=1, L=7, Dm=4, De=4, N=2, k=3, R=2, E=3)
    K = 2
    grads = backward(dOut, p, K, s["R"])
    eps = 1e-6
    for n in ("w_conv", "b_conv", "A", "D", "b_dt", "W_r", "b_r"):
        num = np.zeros_like(p[n])
        it = np.nditer(p[n], flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            vals = []
            for sgn in (+1, -1):
                q = dict(p); a = p[n].copy(); a[i] += sgn * eps; q[n] = a
                vals.append(np.sum(dOut * forward(q, K, s["R"])))
            num[i] = (vals[0] - vals[1]) / (2 * eps)
        np.testing.assert_allclose(grads[GRAD_OF[n]], num, rtol=2e-5, atol=2e-7, err_msg=n)


# ------------------------------------------------------------------------------------------ library autograd
def dense_mamba_autograd(p, R, disc_mode):
    """Dense Mamba (Section 3.1) typed with torch ops on leaf tensors; gradients by torch.autograd."""
    t = {n: torch.tensor(np.asarray(p[n]), dtype=torch.float64, requires_grad=True) for n in NAMES if n not in ("W_r", "b_r")}
    x = t["x"]; Bsz, L, _ = x.shape
    W_inz = t["W_inz"][0]; De = W_inz.shape[0] // 2
    H = x @ W_inz[:De].T; Z = x @ W_inz[De:].T
    k = t["w_conv"].shape[0]
    conv = F.conv1d(H.transpose(1, 2), t["w_conv"].T.reshape(De, 1, k), t["b_conv"], padding=k - 1, groups=De)[..., :L]
    U = F.silu(conv).transpose(1, 2)
    xdbl = U @ t["W_x"].T
    N = t["A"].shape[1]
    delta, Bm, Cm = xdbl[..., :R], xdbl[..., R:R + N], xdbl[..., R + N:]
    Delta = F.softplus(delta @ t["W_dt"].T + t["b_dt"])
    dA = torch.einsum("blc,cn->blcn", Delta, t["A"])
    Abar = torch.exp(dA)
    Bbar = ((Abar - 1.0) / dA if disc_mode == 0 else 1.0) * torch.einsum("blc,bln->blcn", Delta, Bm)
    h = torch.zeros(Bsz, De, N, dtype=torch.float64)
    ys = []
    for i in range(L):
        h = Abar[:, i] * h + Bbar[:, i] * U[:, i, :, None]
        ys.append(torch.einsum("bcn,bn->bc", h, Cm[:, i]))
    Y = torch.stack(ys, dim=1) + t["D"] * U
    out = (Y * F.silu(Z)) @ t["W_out"][0].T
    return out, t


@pytest.mark.parametrize("disc_mode", [0, 1])
def test_single_expert_gradients_equal_autograd_of_dense_mamba(disc_mode):
    p, s, dOut = case(31, E=1)
    grads = backward(dOut, p, 1, s["R"], disc_mode=disc_mode)
    out, t = dense_mamba_autograd(p, s["R"], disc_mode)
    # E = 1: the gate is softmax over one expert = 1, so the layer is the dense layer and the router gets no gradient
    np.testing.assert_allclose(out.detach().numpy(), forward(p, 1, s["R"], disc_mode=disc_mode), rtol=1e-10, atol=1e-12)
    (out * torch.tensor(dOut)).sum().backward()
    for n, v in t.items():
        np.testing.assert_allclose(grads[GRAD_OF[n]], v.grad.numpy(), rtol=1e-8, atol=1e-10, err_msg=n)
    assert np.abs(grads["dW_r"]).max() < 1e-12 and np.abs(grads["db_r"]).max() < 1e-12


# ------------------------------------------------------------------------------------------ scan adjoint
@pytest.mark.parametrize("disc_mode", [0, 1])
def test_scan_backward_is_the_adjoint_of_the_scan(disc_mode):
    """With Delta, A, B, C fixed the scan is linear in (U, h0): <dY, Y> + <dh, h_last> = <dU, U> + <dh0, h0>."""
    g = np.random.default_rng(3)
    B, L, De, N = 2, 11, 5, 4
    U = g.normal(size=(B, L, De)); Dl = np.exp(g.normal(size=(B, L, De)) - 2.0)
    A = -np.exp(g.normal(size=(De, N))); Bm = g.normal(size=(B, L, N)); Cm = g.normal(size=(B, L, N))
    D = g.normal(size=(De,)); h0 = g.normal(size=(B, De, N))
    dY = g.normal(size=(B, L, De)); dh = g.normal(size=(B, De, N))
    Y, hl = O.selective_scan(U, Dl, A, Bm, Cm, D, h0, disc_mode)
    r = G.selective_scan_backward(dY, U, Dl, A, Bm, Cm, D, h0, disc_mode, dh_last=dh)
    lhs = np.sum(dY * Y) + np.sum(dh * hl)
    rhs = np.sum(r["dU"] * U) + np.sum(r["dh0"] * h0)
    assert abs(lhs - rhs) <= 1e-10 * max(1.0, abs(lhs))


def test_scan_backward_one_step_closed_form():
    """L = 1, one channel, one state, zero-order hold: y = C (a h0 + (a - 1)/A B u), a = exp(Delta A)."""
    Dl, A, Bv, Cv, u, h0, dy = 0.3, -0.7, 1.3, -0.4, 0.9, 0.5, 2.0
    a = np.exp(Dl * A)
    r = G.selective_scan_backward(np.full((1, 1, 1), dy), np.full((1, 1, 1), u), np.full((1, 1, 1), Dl), np.full((1, 1), A),
                                  np.full((1, 1, 1), Bv), np.full((1, 1, 1), Cv), None, np.full((1, 1, 1), h0), 0)
    assert abs(r["dU"][0, 0, 0] - dy * Cv * (a - 1) / A * Bv) < 1e-14
    assert abs(r["dDelta"][0, 0, 0] - dy * Cv * (A * a * h0 + a * Bv * u)) < 1e-14
    assert abs(r["dCm"][0, 0, 0] - dy * (a * h0 + (a - 1) / A * Bv * u)) < 1e-14
    assert abs(r["dBm"][0, 0, 0] - dy * Cv * (a - 1) / A * u) < 1e-14
    assert abs(r["dh0"][0, 0, 0] - dy * Cv * a) < 1e-14
    assert abs(r["dA"][0, 0] - dy * Cv * (Dl * a * h0 + (Dl * a * A - (a - 1)) / A ** 2 * Bv * u)) < 1e-13


# ------------------------------------------------------------------------------------------ router
def test_uniform_router_with_all_experts_selected():
    """W_r = 0, b_r = 0, K = E: every gate is 1/E; db_r sums to zero (softmax is shift invariant) and, in gate
    mode 1 with K = E (gates are the full softmax renormalised by 1), equals the gate-mode-0 gradient."""
    p, s, dOut = case(41, E=3)
    p["W_r"] = np.zeros_like(p["W_r"]); p["b_r"] = np.zeros_like(p["b_r"])
    g0 = backward(dOut, p, 3, s["R"], gate_mode=0)
    g1 = backward(dOut, p, 3, s["R"], gate_mode=1)
    assert abs(np.sum(g0["db_r"])) < 1e-12
    np.testing.assert_allclose(g1["db_r"], g0["db_r"], rtol=1e-10, atol=1e-12)
    # dW_out of expert e is (1/E) dOut^T Yg over all tokens: the same matrix for every expert
    np.testing.assert_allclose(g0["dW_out"][0], g0["dW_out"][2], rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------------------------------ planted mistakes
def test_finite_difference_pin_catches_planted_mistakes(monkeypatch):
    p, s, dOut = case(51, B=1, L=6, Dm=4, De=4, N=2, k=3, R=2, E=2)
    K = 1
    g = np.random.default_rng(9)
    dirs = {n: g.normal(size=np.shape(p[n])) for n in NAMES}
    eps = 1e-6

    def mismatch():
        grads = backward(dOut, p, K, s["R"])
        worst = 0.0
        for n in NAMES:
            vals = []
            for sgn in (+1, -1):
                q = dict(p); q[n] = p[n] + sgn * eps * dirs[n]
                vals.append(np.sum(dOut * forward(q, K, s["R"])))
            fd = (vals[0] - vals[1]) / (2 * eps)
            worst = max(worst, abs(fd - float(np.sum(grads[GRAD_OF[n]] * dirs[n]))) / max(1.0, abs(fd)))
        return worst

    assert mismatch() < 1e-6
    orig_scan, orig_conv, orig_route = G.selective_scan_backward, G.conv_silu_backward, G.route_backward

    def scan_no_carry(dY, U, Dl, A, Bm, Cm, D=None, h0=None, m=0, dh_last=None):      # forgets the skip term's gradient
        r = orig_scan(dY, U, Dl, A, Bm, Cm, None, h0, m, dh_last); r["dD"] = np.zeros(U.shape[2]); return r
    with monkeypatch.context() as mp:
        mp.setattr(G, "selective_scan_backward", scan_no_carry)
        assert mismatch() > 1e-4
    with monkeypatch.context() as mp:                                                  # conv taps reversed in the backward
        mp.setattr(G, "conv_silu_backward", lambda dU, H, w, b=None: (lambda a, b_, c: (a, b_[::-1], c))(*orig_conv(dU, H, w, b)))
        assert mismatch() > 1e-4
    with monkeypatch.context() as mp:                                                  # softmax Jacobian without the mean term
        mp.setattr(G, "route_backward", lambda dg, x, W, P, idx, gate, gm=0: orig_route(dg, x, W, P * 0 + 1.0 / P.shape[1], idx, gate, gm))
        assert mismatch() > 1e-4
