"""Pins of the oracle for RoM on a Mamba2-style block (oracle/rom_mamba2_oracle.py) against things other than
itself: a dense Mamba2 block typed with library ops whose state-space part is the quadratic dual form (no
recurrence), a brute-force unrolled sum, the library RMS norm, closed forms and invariants.  CPU only."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import rom_mamba2_oracle as M


def case(seed, B=2, L=10, Dm=8, De=16, P=4, N=4, k=4, E=3, scale=0.5):
    g = np.random.default_rng(seed)
    H = De // P
    W = 2 * De + 2 * N + H
    p = dict(x=g.normal(size=(B, L, Dm)), W_r=g.normal(size=(E, Dm)), b_r=None,
             W_in=g.normal(size=(E, W, Dm)) * scale, w_conv=g.normal(size=(k, De + 2 * N)) * scale,
             b_conv=g.normal(size=(De + 2 * N,)) * 0.1, dt_bias=g.normal(size=(H,)) * 0.5 - 1.0,
             A=-np.exp(g.normal(size=(H,))), D=g.normal(size=(H,)), w_norm=1.0 + 0.1 * g.normal(size=(De,)),
             W_out=g.normal(size=(E, Dm, De)) * scale)
    return p, dict(B=B, L=L, Dm=Dm, De=De, P=P, N=N, k=k, E=E, H=H)


def run(p, s, K, **kw):
    return M.rom_mamba2_forward(p["x"], p["W_r"], p["b_r"], p["W_in"], p["w_conv"], p["b_conv"], p["dt_bias"], p["A"], p["D"],
                                p["w_norm"], p["W_out"], K=K, headdim=s["P"], d_state=s["N"], **kw)


def dense_mamba2_dual_form(x, W_in, w_conv, b_conv, dt_bias, A, D, w_norm, W_out, P, N):
    """A dense Mamba2 block with library ops; the state-space output is the masked, decay-weighted "attention"
    y_t = sum_{s<=t} (C_t . B_s) exp(sum_{r=s+1..t} dt_r A) dt_s x_s  computed with a cumulative sum and einsum."""
    x = torch.as_tensor(x); Bsz, L, Dm = x.shape
    De = W_out.shape[1]; H = De // P
    zx = x @ torch.as_tensor(W_in).T
    z, xbc_raw, dt_raw = zx[..., :De], zx[..., De:2 * De + 2 * N], zx[..., 2 * De + 2 * N:]
    k = w_conv.shape[0]
    C = De + 2 * N
    conv = F.conv1d(xbc_raw.transpose(1, 2), torch.as_tensor(w_conv).T.reshape(C, 1, k), torch.as_tensor(b_conv), padding=k - 1, groups=C)[..., :L]
    xbc = F.silu(conv).transpose(1, 2)
    xs, Bm, Cm = xbc[..., :De].reshape(Bsz, L, H, P), xbc[..., De:De + N], xbc[..., De + N:]
    dt = F.softplus(dt_raw + torch.as_tensor(dt_bias))                                  # [B,L,H]
    cs = torch.cumsum(dt * torch.as_tensor(A), dim=1)                                    # sum_{r<=t} dt_r A
    decay = torch.exp(cs[:, :, None, :] - cs[:, None, :, :])                             # [B,t,s,H] = exp(sum_{r=s+1..t})
    mask = torch.tril(torch.ones(L, L, dtype=torch.bool))[None, :, :, None]
    scores = torch.einsum("btn,bsn->bts", Cm, Bm)[..., None] * torch.where(mask, decay, torch.zeros_like(decay))
    y = torch.einsum("btsh,bsh,bshp->bthp", scores, dt, xs) + torch.as_tensor(D)[None, None, :, None] * xs
    g = y.reshape(Bsz, L, De) * F.silu(z)
    yn = F.rms_norm(g, (De,), torch.as_tensor(w_norm), eps=1e-5)
    return (yn @ torch.as_tensor(W_out).T).numpy()


def test_single_expert_equals_dense_mamba2_in_dual_form():
    p, s = case(1, E=1)
    ref = dense_mamba2_dual_form(p["x"], p["W_in"][0], p["w_conv"], p["b_conv"], p["dt_bias"], p["A"], p["D"], p["w_norm"], p["W_out"][0], s["P"], s["N"])
    np.testing.assert_allclose(run(p, s, K=1), ref, rtol=1e-9, atol=1e-11)


def test_recurrence_equals_bruteforce_unrolled_sum():
    g = np.random.default_rng(2)
    B, L, H, P, N = 1, 6, 2, 3, 2
    xh = g.normal(size=(B, L, H, P)); dt = np.exp(g.normal(size=(B, L, H)) - 1.0); A = -np.exp(g.normal(size=(H,)))
    Bm = g.normal(size=(B, L, N)); Cm = g.normal(size=(B, L, N)); h0 = g.normal(size=(B, H, P, N))
    y, hl = M.ssd_scan(xh, dt, A, Bm, Cm, None, h0)
    for t in range(L):
        for h in range(H):
            for pp in range(P):
                v = 0.0
                for n in range(N):
                    st = h0[0, h, pp, n] * np.prod([np.exp(dt[0, r, h] * A[h]) for r in range(t + 1)])
                    for s_ in range(t + 1):
                        st += np.prod([np.exp(dt[0, r, h] * A[h]) for r in range(s_ + 1, t + 1)]) * dt[0, s_, h] * xh[0, s_, h, pp] * Bm[0, s_, n]
                    v += Cm[0, t, n] * st
                assert abs(y[0, t, h, pp] - v) < 1e-12


def test_scan_in_two_halves_and_constant_input_series():
    g = np.random.default_rng(3)
    B, L, H, P, N = 2, 9, 2, 2, 3
    xh = g.normal(size=(B, L, H, P)); dt = np.exp(g.normal(size=(B, L, H)) - 1.0); A = -np.exp(g.normal(size=(H,)))
    Bm = g.normal(size=(B, L, N)); Cm = g.normal(size=(B, L, N)); D = g.normal(size=(H,))
    y, hl = M.ssd_scan(xh, dt, A, Bm, Cm, D)
    y1, h1 = M.ssd_scan(xh[:, :4], dt[:, :4], A, Bm[:, :4], Cm[:, :4], D)
    y2, h2 = M.ssd_scan(xh[:, 4:], dt[:, 4:], A, Bm[:, 4:], Cm[:, 4:], D, h1)
    np.testing.assert_allclose(np.concatenate([y1, y2], axis=1), y, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(h2, hl, rtol=1e-12, atol=1e-14)
    # constant dt, x, B: h_t = dt x B (1 - a^t) / (1 - a)
    d, a_, xv, bv = 0.3, -0.8, 1.7, -0.6
    yc, _ = M.ssd_scan(np.full((1, 7, 1, 1), xv), np.full((1, 7, 1), d), np.array([a_]), np.full((1, 7, 1), bv), np.ones((1, 7, 1)))
    a = np.exp(d * a_)
    np.testing.assert_allclose(yc[0, :, 0, 0], [d * xv * bv * (1 - a ** (t + 1)) / (1 - a) for t in range(7)], rtol=1e-12)


def test_gated_rmsnorm_equals_library_rms_norm():
    g = np.random.default_rng(4)
    y = g.normal(size=(5, 12)); z = g.normal(size=(5, 12)); w = g.normal(size=(12,))
    ref = F.rms_norm(torch.tensor(y) * F.silu(torch.tensor(z)), (12,), torch.tensor(w), eps=1e-5).numpy()
    np.testing.assert_allclose(M.gated_rmsnorm(y, z, w), ref, rtol=1e-12, atol=1e-14)


def test_all_experts_with_uniform_gates_is_the_dense_block_on_summed_and_mean_experts():
    p, s = case(5, E=3)
    p["W_r"] = np.zeros_like(p["W_r"])
    ref = dense_mamba2_dual_form(p["x"], p["W_in"].sum(axis=0), p["w_conv"], p["b_conv"], p["dt_bias"], p["A"], p["D"], p["w_norm"],
                                 p["W_out"].mean(axis=0), s["P"], s["N"])
    np.testing.assert_allclose(run(p, s, K=3), ref, rtol=1e-9, atol=1e-11)


@pytest.mark.parametrize("K", [1, 2])
def test_batch_permutation_invariance_and_causality(K):
    p, s = case(6, B=3)
    out, im = run(p, s, K=K, return_intermediates=True)
    pi = np.array([2, 0, 1])
    q = dict(p); q["x"] = p["x"][pi]
    out2, im2 = run(q, s, K=K, return_intermediates=True)
    np.testing.assert_allclose(out2, out[pi], rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(im2["counts"], im["counts"])
    r = dict(p); xr = p["x"].copy(); xr[1, 6] += 1.0; r["x"] = xr           # a later token of sequence 1 changes
    out3 = run(r, s, K=K)
    np.testing.assert_array_equal(out3[1, :6], out[1, :6])
    np.testing.assert_array_equal(out3[[0, 2]], out[[0, 2]])


def test_pins_catch_planted_mistakes(monkeypatch):
    p, s = case(7, E=1)
    ref = dense_mamba2_dual_form(p["x"], p["W_in"][0], p["w_conv"], p["b_conv"], p["dt_bias"], p["A"], p["D"], p["w_norm"], p["W_out"][0], s["P"], s["N"])
    orig_scan, orig_norm = M.ssd_scan, M.gated_rmsnorm

    def broken(name, fn):
        with monkeypatch.context() as m:
            m.setattr(M, name, fn)
            return np.abs(run(p, s, K=1) - ref).max()
    assert broken("ssd_scan", lambda xh, dt, A, B_, C_, D=None, h0=None: orig_scan(xh, dt, A, C_, B_, D, h0)) > 1e-6        # B / C swapped
    assert broken("ssd_scan", lambda xh, dt, A, B_, C_, D=None, h0=None: orig_scan(xh, dt, A, B_, C_, None, h0)) > 1e-6     # dropped D
    assert broken("ssd_scan", lambda xh, dt, A, B_, C_, D=None, h0=None: orig_scan(xh, np.ones_like(dt), A, B_, C_, D, h0)) > 1e-6   # dt ignored
    assert broken("gated_rmsnorm", lambda y, z, w, eps=1e-5: orig_norm(y, z, np.ones_like(w), eps)) > 1e-6                  # norm weight dropped
