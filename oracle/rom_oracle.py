"""CPU oracle for the forward pass of one Routing-Mamba (RoM) layer.

TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64 numpy; every function is the
paper's definition written out step by step, in the paper's order and notation.
Nothing here is blocked, fused or reordered, and nothing is shared with the
CUDA path (no common code, tables or helpers).  Only tests, the smoke check and
the benchmark's cpu-baseline leg may import this package.

Notation (Section 3.1 / 4.2):  X in R^{L x D_m} per sequence, D_e inner width,
D_s = N states, k conv taps, d_r = R dt rank, E experts, top-K.
Tensors are numpy float64 unless stated; "T" = B*L tokens in (b, t) order.

Readings taken where the paper is silent (each is a flag or an optional argument):
  * top-K is taken on the router logits (softmax is monotone); ties go to the
    lowest expert id; slot k holds the k-th largest.
  * gate_mode 0 = Eq. (R_i = P * indicator) literally, P the softmax over all E;
    gate_mode 1 = the sentence above it (renormalise over the selected K).
  * Conv Proj / Gate Proj sums over selected experts are NOT gate-weighted
    (Eq. for G and H_t carry only the indicator); only the Out Proj sum is.
  * (delta, B, C) = U W_x, Delta = softplus(delta W_dt + b_dt): the paper names
    "x Proj, dt Proj" without an equation; the split order delta|B|C is ours.
  * conv is causal with zero left padding per sequence; tap k-1 is the current token.
  * disc_mode 0 = zero-order hold exactly as printed (diagonal A);
    disc_mode 1 = B-bar = Delta * B.
  * D skip, conv bias, dt bias, router bias are optional (None = paper-literal).
  * per-expert x Proj / dt Proj (an ablation row of Section 5.3, no equation printed):
    indicator-only sums like H_t; each expert's delta passes through its own dt Proj.

Pins (tests/test_oracle_pins.py): dense-Mamba reduction (E=K=1), brute-force
unrolled SSM, K=E uniform gates = mean of experts, batch-permutation invariance,
identical experts, geometric-series closed form, exact ODE solution for ZOH,
identity conv tap + causality, permutation tables vs brute force and a stable
sort, gate sums, tie rule, two-half scan, parameter counts printed in the paper;
per-expert small projections: E=1 / identical experts reduce to the shared form, rows of
one expert equal the shared form with that expert's matrices, per-token brute force;
FFN-MoE with shared routing: library SwiGLU for E=1, per-token loops, identical experts with
gates summing to one = the dense FFN, linearity in the gates;
single-token step: a sequence fed token by token reproduces the full-sequence forward and its states.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------- elementwise
def silu(v):
    """SiLU(v) = v * sigmoid(v) (activation of Eq. for U and for G)."""
    v = np.asarray(v, dtype=F64)
    return v / (1.0 + np.exp(-v))


def softplus(v):
    """softplus(v) = log(1 + exp(v)), evaluated without overflow."""
    v = np.asarray(v, dtype=F64)
    return np.maximum(v, 0.0) + np.log1p(np.exp(-np.abs(v)))


# --------------------------------------------------------------------------- S1 router
def router_logits(x, W_r, b_r=None):
    """logit[t,e] = b_r[e] + sum_d x[t,d] * W_r[e,d], accumulated in ascending d.

    Section 4.2, P = Softmax(X_t . W_r) with W_r in R^{D_m x N}; W_r is stored
    transposed here ([E, D_m]).  The sum is taken strictly left to right so the
    result does not depend on a BLAS blocking order (the top-K decision below is
    compared bit for bit).
    """
    x = np.asarray(x, dtype=F64)
    W_r = np.asarray(W_r, dtype=F64)
    T, Dm = x.shape
    E = W_r.shape[0]
    logit = np.zeros((T, E), dtype=F64)
    if b_r is not None:
        logit += np.asarray(b_r, dtype=F64)[None, :]
    for d in range(Dm):
        logit = logit + x[:, d:d + 1] * W_r[None, :, d]
    return logit


def route(x, W_r, b_r, K, gate_mode=0):
    """Router of Section 4.2: P = softmax(logits) over all E experts; the K largest
    are selected (indicator 1_{i in TopK(P)}); R_i = P_i * indicator (gate_mode 0)
    or P_i / sum of the selected P (gate_mode 1).

    Returns (idx[T,K] int32, gate[T,K] f64, P[T,E] f64, logit[T,E] f64).
    """
    logit = router_logits(x, W_r, b_r)
    T, E = logit.shape
    if not (1 <= K <= E):
        raise ValueError("need 1 <= K <= E")
    m = np.max(logit, axis=1, keepdims=True)
    ex = np.exp(logit - m)
    P = ex / np.sum(ex, axis=1, keepdims=True)
    key = np.where(np.isnan(logit), -np.inf, logit).copy()
    idx = np.zeros((T, K), dtype=np.int32)
    rows = np.arange(T)
    taken = np.zeros((T, E), dtype=bool)
    for k in range(K):
        masked = np.where(taken, -np.inf, key)
        # first maximum among the experts not taken yet = lowest expert id on ties;
        # argmax over a masked copy could return a taken expert when all remaining
        # keys are -inf, so search the not-taken ones explicitly
        best = np.full(T, -1, dtype=np.int64)
        bestv = np.full(T, -np.inf)
        for e in range(E):
            cand = (~taken[:, e]) & ((best < 0) | (masked[:, e] > bestv))
            best = np.where(cand, e, best)
            bestv = np.where(cand, masked[:, e], bestv)
        idx[:, k] = best
        taken[rows, best] = True
    gate = P[rows[:, None], idx]
    if gate_mode == 1:
        gate = gate / np.sum(gate, axis=1, keepdims=True)
    elif gate_mode != 0:
        raise ValueError("gate_mode must be 0 or 1")
    return idx, gate, P, logit


# --------------------------------------------------------------------------- S2 permutation
def permutation_tables(idx, E):
    """Dropless grouping of the T*K (token, slot) assignments by expert.

    Assignment a = t*K + k goes to expert idx[t,k].  counts[e] = number of
    assignments of e; offsets = exclusive prefix sum (offsets[E] = T*K); inside an
    expert's segment assignments keep ascending a.  perm[r] = a, inv_perm[a] = r.
    (The paper only requires that no token is dropped and no capacity factor is
    used, Section 5.1; the order inside a segment is ours.)
    """
    idx = np.asarray(idx)
    flat = idx.reshape(-1)
    A = flat.shape[0]
    counts = np.zeros(E, dtype=np.int32)
    for a in range(A):
        counts[flat[a]] += 1
    offsets = np.zeros(E + 1, dtype=np.int32)
    for e in range(E):
        offsets[e + 1] = offsets[e] + counts[e]
    fill = np.zeros(E, dtype=np.int64)
    perm = np.zeros(A, dtype=np.int32)
    inv = np.zeros(A, dtype=np.int32)
    for a in range(A):
        e = flat[a]
        r = offsets[e] + fill[e]
        fill[e] += 1
        perm[r] = a
        inv[a] = r
    return counts, offsets, perm, inv


# --------------------------------------------------------------------------- S3 routed Conv/Gate Proj
def expert_in_proj(x, W_inz, idx):
    """H_t = sum_i 1_i X_t W_in,i and (pre-activation of G) Z_t = sum_i 1_i X_t W_g,i
    (Section 4.2, equations for H_t and G): indicator only, no gate weight.

    x[T,D_m]; W_inz[E, 2*D_e, D_m] with rows [0,D_e) = W_in,i^T and [D_e,2D_e) = W_g,i^T.
    Returns H[T,D_e], Zpre[T,D_e].
    """
    x = np.asarray(x, dtype=F64)
    W_inz = np.asarray(W_inz, dtype=F64)
    T = x.shape[0]
    E, twoDe, _ = W_inz.shape
    De = twoDe // 2
    H = np.zeros((T, De), dtype=F64)
    Z = np.zeros((T, De), dtype=F64)
    K = idx.shape[1]
    for k in range(K):
        for e in range(E):
            tok = np.nonzero(idx[:, k] == e)[0]
            if tok.size == 0:
                continue
            xz = x[tok] @ W_inz[e].T
            H[tok] += xz[:, :De]
            Z[tok] += xz[:, De:]
    return H, Z


# --------------------------------------------------------------------------- S4 short conv
def conv_silu(H, w_conv, b_conv=None):
    """U = SiLU(DWConv(H, W_conv)) (Section 3.1): depthwise, over the sequence
    dimension, causal; H[B,L,D_e], w_conv[k,D_e], tap k-1 on the current token.
    """
    H = np.asarray(H, dtype=F64)
    w = np.asarray(w_conv, dtype=F64)
    B, L, De = H.shape
    k = w.shape[0]
    pre = np.zeros((B, L, De), dtype=F64)
    if b_conv is not None:
        pre += np.asarray(b_conv, dtype=F64)[None, None, :]
    for j in range(k):
        shift = (k - 1) - j            # tap j looks `shift` tokens back
        if shift >= L:
            continue
        pre[:, shift:, :] += w[j][None, None, :] * H[:, :L - shift, :]
    return silu(pre)


# --------------------------------------------------------------------------- S5/S6 x Proj, dt Proj
def small_proj(U, W_x, W_dt, b_dt, dt_rank, d_state):
    """(delta, B, C) = U W_x ; Delta = softplus(delta W_dt + b_dt).  Shared across
    experts (Section 4.3).  U[T,D_e]; W_x[R+2N, D_e]; W_dt[D_e, R].
    Returns delta[T,R], Bm[T,N], Cm[T,N], Delta[T,D_e].
    """
    U = np.asarray(U, dtype=F64)
    W_x = np.asarray(W_x, dtype=F64)
    W_dt = np.asarray(W_dt, dtype=F64)
    R, N = dt_rank, d_state
    xdbl = U @ W_x.T
    delta = xdbl[:, :R]
    Bm = xdbl[:, R:R + N]
    Cm = xdbl[:, R + N:R + 2 * N]
    pre = delta @ W_dt.T
    if b_dt is not None:
        pre = pre + np.asarray(b_dt, dtype=F64)[None, :]
    return delta, Bm, Cm, softplus(pre)


def small_proj_routed(U, W_x, W_dt, b_dt, idx, dt_rank, d_state):
    """x Proj and dt Proj as per-expert layers under the shared routing decision: the ablation
    "RoM (Conv, Gate, dt, x, Out)" of Section 5.3 (Section 4.3 shares them by default).  The paper
    prints no equation for this variant; it is read in the pattern of the equations for H_t and G
    (indicator-only sums over the selected experts):
        (delta_i, B_i, C_i) = U_t W_x,i ,  B_t = sum_i 1_i B_i ,  C_t = sum_i 1_i C_i ,
        Delta_t = softplus( sum_i 1_i delta_i W_dt,i + b_dt ),
    each expert's delta_i going through that expert's own dt Proj; b_dt stays shared.
    U[T,D_e]; W_x[E, R+2N, D_e]; W_dt[E, D_e, R]; idx[T,K].  Returns Bm[T,N], Cm[T,N], Delta[T,D_e].
    """
    U = np.asarray(U, dtype=F64)
    W_x = np.asarray(W_x, dtype=F64)
    W_dt = np.asarray(W_dt, dtype=F64)
    R, N = dt_rank, d_state
    T, De = U.shape
    E = W_x.shape[0]
    Bm = np.zeros((T, N), dtype=F64)
    Cm = np.zeros((T, N), dtype=F64)
    pre = np.zeros((T, De), dtype=F64)
    K = idx.shape[1]
    for k in range(K):
        for e in range(E):
            tok = np.nonzero(idx[:, k] == e)[0]
            if tok.size == 0:
                continue
            xdbl = U[tok] @ W_x[e].T
            Bm[tok] += xdbl[:, R:R + N]
            Cm[tok] += xdbl[:, R + N:R + 2 * N]
            pre[tok] += xdbl[:, :R] @ W_dt[e].T
    if b_dt is not None:
        pre = pre + np.asarray(b_dt, dtype=F64)[None, :]
    return Bm, Cm, softplus(pre)


# --------------------------------------------------------------------------- S7 selective scan
def selective_scan(U, Delta, A, Bm, Cm, D=None, h0=None, disc_mode=0):
    """Linear recurrence of Section 3.1:  h_t = A-bar h_{t-1} + B-bar U_t,  Y_t = C h_t
    with A-bar = exp(Delta A) and (zero-order hold, diagonal A)
    B-bar = (Delta A)^-1 (exp(Delta A) - 1) Delta B = expm1(Delta A) / A * B
    (disc_mode 0) or B-bar = Delta B (disc_mode 1).  Optional skip D*U.

    U, Delta [B,L,D_e]; A[D_e,N] (negative); Bm, Cm [B,L,N]; D[D_e]; h0[B,D_e,N].
    Returns Y[B,L,D_e], h_last[B,D_e,N].
    """
    U = np.asarray(U, dtype=F64)
    Delta = np.asarray(Delta, dtype=F64)
    A = np.asarray(A, dtype=F64)
    Bm = np.asarray(Bm, dtype=F64)
    Cm = np.asarray(Cm, dtype=F64)
    Bsz, L, De = U.shape
    N = A.shape[1]
    h = np.zeros((Bsz, De, N), dtype=F64) if h0 is None else np.array(h0, dtype=F64)
    Y = np.zeros((Bsz, L, De), dtype=F64)
    for t in range(L):
        dA = Delta[:, t, :, None] * A[None, :, :]                  # [B,De,N]
        Abar = np.exp(dA)
        if disc_mode == 0:
            Bbar = np.expm1(dA) / A[None, :, :] * Bm[:, t, None, :]
        elif disc_mode == 1:
            Bbar = Delta[:, t, :, None] * Bm[:, t, None, :]
        else:
            raise ValueError("disc_mode must be 0 or 1")
        h = Abar * h + Bbar * U[:, t, :, None]
        Y[:, t, :] = np.sum(Cm[:, t, None, :] * h, axis=2)
    if D is not None:
        Y = Y + np.asarray(D, dtype=F64)[None, None, :] * U
    return Y, h


# --------------------------------------------------------------------------- S8..S11 gate, Out Proj, combine
def gated(Y, Zpre):
    """Y (.) G with G = SiLU(Zpre) (Section 3.1 output equation / Section 4.2 expert equation)."""
    return np.asarray(Y, dtype=F64) * silu(Zpre)


def expert_out_proj(Yg, W_out, idx, gate):
    """O_t = sum_i R_i(X_t) * (Y_t (.) G) W_out,i (Section 4.2): gate-weighted sum over
    the selected experts, slots added in ascending k.  Yg[T,D_e]; W_out[E,D_m,D_e].
    """
    Yg = np.asarray(Yg, dtype=F64)
    W_out = np.asarray(W_out, dtype=F64)
    T = Yg.shape[0]
    E, Dm, _ = W_out.shape
    out = np.zeros((T, Dm), dtype=F64)
    K = idx.shape[1]
    for k in range(K):
        for e in range(E):
            tok = np.nonzero(idx[:, k] == e)[0]
            if tok.size == 0:
                continue
            out[tok] += gate[tok, k][:, None] * (Yg[tok] @ W_out[e].T)
    return out


# --------------------------------------------------------------------------- the layer
def rom_layer_forward(x, W_r, b_r, W_inz, w_conv, b_conv, W_x, W_dt, b_dt, A, D, W_out,
                      K, dt_rank, gate_mode=0, disc_mode=0, return_intermediates=False):
    """Forward pass of one RoM layer (Section 4.2 with the shared small layers of 4.3).
    W_x[R+2N, D_e] and W_dt[D_e, R] are the shared x Proj / dt Proj; three-dimensional
    W_x[E, ...], W_dt[E, ...] select the per-expert variant (small_proj_routed).

    x[B,L,D_m].  Returns out[B,L,D_m] (and a dict of every intermediate if asked).
    """
    x = np.asarray(x, dtype=F64)
    Bsz, L, Dm = x.shape
    T = Bsz * L
    xt = x.reshape(T, Dm)
    E = np.asarray(W_r).shape[0]
    A = np.asarray(A, dtype=F64)
    N = A.shape[1]
    idx, gate, P, logit = route(xt, W_r, b_r, K, gate_mode)
    counts, offsets, perm, inv = permutation_tables(idx, E)
    H, Zpre = expert_in_proj(xt, W_inz, idx)
    De = H.shape[1]
    U = conv_silu(H.reshape(Bsz, L, De), w_conv, b_conv)
    if np.asarray(W_x).ndim == 3:          # per-expert x Proj / dt Proj (ablation of Section 5.3)
        delta = None
        Bm, Cm, Delta = small_proj_routed(U.reshape(T, De), W_x, W_dt, b_dt, idx, dt_rank, N)
    else:
        delta, Bm, Cm, Delta = small_proj(U.reshape(T, De), W_x, W_dt, b_dt, dt_rank, N)
    Y, h_last = selective_scan(U, Delta.reshape(Bsz, L, De), A, Bm.reshape(Bsz, L, N),
                               Cm.reshape(Bsz, L, N), D, None, disc_mode)
    Yg = gated(Y.reshape(T, De), Zpre)
    out = expert_out_proj(Yg, W_out, idx, gate).reshape(Bsz, L, Dm)
    if not return_intermediates:
        return out
    return out, dict(idx=idx, gate=gate, P=P, logit=logit, counts=counts, offsets=offsets,
                     perm=perm, inv_perm=inv, H=H, Zpre=Zpre, U=U.reshape(T, De), delta=delta,
                     Bm=Bm, Cm=Cm, Delta=Delta, Y=Y.reshape(T, De), Yg=Yg, h_last=h_last)


# --------------------------------------------------------------------------- single-token step (recurrent inference)
def rom_layer_step(x_t, conv_state, ssm_state, W_r, b_r, W_inz, w_conv, b_conv, W_x, W_dt, b_dt, A, D, W_out,
                   K, dt_rank, gate_mode=0, disc_mode=0):
    """One token per sequence through the RoM layer with the state carried between calls: the recurrent
    form of the same equations (Section 3.1: the state-space model as a linear recurrence, which is what
    gives constant cost per generated token; Section 4.2 routing and expert equations unchanged).

    x_t[B,D_m]: the new token of each sequence.
    conv_state[B,k-1,D_e]: H of the previous k-1 tokens, oldest first (zeros at a sequence start).
    ssm_state[B,D_e,N]: h_{t-1} (zeros at a sequence start).
    Returns out_t[B,D_m], new conv_state, new ssm_state.  Nothing here is shared with the full-sequence
    functions except the routed projections: the conv tap sum and the state update are written for one step.
    """
    x_t = np.asarray(x_t, dtype=F64)
    conv_state = np.asarray(conv_state, dtype=F64)
    h = np.array(ssm_state, dtype=F64)
    A = np.asarray(A, dtype=F64)
    w = np.asarray(w_conv, dtype=F64)
    Bsz = x_t.shape[0]
    k = w.shape[0]
    N = A.shape[1]
    idx, gate, _, _ = route(x_t, W_r, b_r, K, gate_mode)
    H_t, Zpre = expert_in_proj(x_t, W_inz, idx)                       # [B,D_e] each
    window = np.concatenate([conv_state, H_t[:, None, :]], axis=1)    # [B,k,D_e], oldest first, current last
    pre = np.zeros_like(H_t)
    if b_conv is not None:
        pre = pre + np.asarray(b_conv, dtype=F64)[None, :]
    for j in range(k):
        pre = pre + w[j][None, :] * window[:, j, :]
    U_t = silu(pre)
    if np.asarray(W_x).ndim == 3:
        Bm, Cm, Delta = small_proj_routed(U_t, W_x, W_dt, b_dt, idx, dt_rank, N)
    else:
        _, Bm, Cm, Delta = small_proj(U_t, W_x, W_dt, b_dt, dt_rank, N)
    dA = Delta[:, :, None] * A[None, :, :]
    if disc_mode == 0:
        Bbar = np.expm1(dA) / A[None, :, :] * Bm[:, None, :]
    else:
        Bbar = Delta[:, :, None] * Bm[:, None, :]
    h = np.exp(dA) * h + Bbar * U_t[:, :, None]
    Y_t = np.sum(Cm[:, None, :] * h, axis=2)
    if D is not None:
        Y_t = Y_t + np.asarray(D, dtype=F64)[None, :] * U_t
    out_t = expert_out_proj(gated(Y_t, Zpre), W_out, idx, gate)
    return out_t, window[:, 1:, :].copy(), h


# --------------------------------------------------------------------------- FFN-MoE with shared routing
def ffn_moe_shared_routing(x, W_gu, W_down, idx, gate):
    """Feed-forward SwiGLU mixture of experts that reuses the routing decision of the preceding RoM
    layer (Appendix A.2, the two equations of the hybrid "RoM + FFN-MoE" model):
        Y_t = sum_i R_i * E_i(X_t),   E_i(X_t) = 1[i in TopK] * f_i(X_t),
    with idx[T,K] (the selected experts) and gate[T,K] (R_i of the selected experts) taken from that
    layer's router, not recomputed.  The paper names f_i "the i-th feedforward SwiGLU expert" without
    writing it out; the usual bias-free form is taken:
        f_i(x) = W_down,i ( SiLU(W_gate,i x) * (W_up,i x) ).
    x[T,D_m]; W_gu[E, 2*D_ff, D_m], rows [0,D_ff) = W_gate,i and [D_ff,2D_ff) = W_up,i;
    W_down[E, D_m, D_ff].  Returns Y[T,D_m].
    """
    x = np.asarray(x, dtype=F64)
    W_gu = np.asarray(W_gu, dtype=F64)
    W_down = np.asarray(W_down, dtype=F64)
    gate = np.asarray(gate, dtype=F64)
    T, Dm = x.shape
    E, twoF, _ = W_gu.shape
    Dff = twoF // 2
    Y = np.zeros((T, Dm), dtype=F64)
    for k in range(idx.shape[1]):
        for e in range(E):
            tok = np.nonzero(idx[:, k] == e)[0]
            if tok.size == 0:
                continue
            gu = x[tok] @ W_gu[e].T
            hidden = silu(gu[:, :Dff]) * gu[:, Dff:]
            Y[tok] += gate[tok, k][:, None] * (hidden @ W_down[e].T)
    return Y


# --------------------------------------------------------------------------- wiring pin
def rom_param_count(n_layers, d_model, E, vocab, expand=2, d_state=16, d_conv=4, tie_embeddings=True):
    """Parameters of a stack of RoM layers wired as in Section 4.2/4.3: Conv Proj, Gate
    Proj and Out Proj replicated E times; router, conv1d, x Proj, dt Proj, A, D shared;
    d_e = expand * d_m, d_r = d_m / 16 (Section 3.1).  Pre-norm weight per layer plus a
    final norm; embedding counted once when tied.  Returns (total, active-with-top-1).
    """
    De = expand * d_model
    R = d_model // 16
    N = d_state
    routed = 2 * d_model * De + De * d_model                 # W_in + W_g + W_out of one expert
    shared = (d_conv * De + De) + De * (R + 2 * N) + (R * De + De) + De * N + De + d_model
    router = d_model * E if E > 1 else 0
    per_layer_total = E * routed + shared + router
    per_layer_active = routed + shared + router
    emb = vocab * d_model * (1 if tie_embeddings else 2)
    return n_layers * per_layer_total + emb + d_model, n_layers * per_layer_active + emb + d_model


# --------------------------------------------------------------------------- load-balance statistic
def load_balance_loss(P, idx, alpha=1e-3):
    """One layer's term of the auxiliary loss of Appendix A.3:
    alpha * N * sum_i F_i * mean_t P[t,i], F_i = fraction of tokens dispatched to expert i.
    """
    P = np.asarray(P, dtype=F64)
    T, E = P.shape
    F = np.zeros(E, dtype=F64)
    for e in range(E):
        F[e] = np.sum(idx == e) / float(T)
    return alpha * E * float(np.sum(F * P.mean(axis=0))), F
