"""CPU oracle for the compressed-sensing attention (CSAT) forward.  TEST INFRASTRUCTURE.

This file is test infrastructure: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it.  The product (the CUDA library and
its Python binding) never does, and this file imports nothing from the product.

Plain numpy in float64, one step per equation of the paper's "Mathematical
Framework" section, in the paper's order and notation (rows are tokens, so the
paper's column vectors alpha_i, Z_i, C_i appear here as 1 x d rows):

  compress           K~ = Phi K,  V~ = Phi V              (compression equation)
  compressed_scores  S  = Q K~^T / sqrt(d_k)              (approximate attention matrix)
  softmax_rows       A~ = softmax over the m measurements (same equation)
  compressed_output  Z  = A~ V~                           (compressed attention output)
  decoder_setup      S, B, theta of the LISTA recurrence, instantiated as ISTA
  ista               alpha^{t+1} = eta_theta(S alpha^t + B Z_i)   (LISTA recurrence, ISTA weights)
  lista              the same recurrence with supplied S, B and per-layer theta_t
  reconstruct        C^_i = Psi alpha^_i                  (reconstruction equation)
  project_qkv        Q = X W^Q, K = X W^K, V = X W^V      (projection equation, one set of d_k columns per head)
  csat_backward      gradients of the forward with respect to Q, K, V (chain rule through the equations above,
                     last to first; the paper trains through the unrolled decoder but prints no backward pass)

Reading of the decoder (the paper's "Z_i = Phi Psi alpha_i" with Phi in R^{m x n}
cannot multiply a d_k-vector): the sensing matrix of the decoder is a d x d matrix
D acting on the feature axis, by default the leading d x d block of the head's
Phi ("Phi_V reused"); M = D Psi; the recurrence is ISTA for
min_alpha 1/2 ||z - alpha M^T||^2 + lambda ||alpha||_1 with step mu = 1/L^,
L^ = max absolute row sum of M^T M; S = I - mu M^T M, B = mu M, theta = mu lambda;
alpha^0 = 0; T = 0 returns Z itself.  Parity with the paper's own (unstated)
decoder: parity unpinned.  Every function below is pinned by tests/test_oracle_pins.py.

A library matmul (numpy @) serves as the contraction step; nothing is blocked,
fused or reordered.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------
# input projections
# ----------------------------------------------------------------------------
def project_qkv(X: np.ndarray, W: np.ndarray, H: int, d: int):
    """Q = X W^Q, K = X W^K, V = X W^V for every head.  X [B,n,d_model]; W [d_model, 3*H*d] holds the projection
    matrices side by side: columns [0, H*d) are W^Q of heads 0..H-1 (d columns each), then W^K, then W^V.
    Returns Q, K, V, each [B,H,n,d]."""
    X = np.asarray(X, F64)
    W = np.asarray(W, F64)
    B, n, dm = X.shape
    assert W.shape == (dm, 3 * H * d)
    out = []
    for which in range(3):
        P = np.empty((B, H, n, d), dtype=F64)
        for h in range(H):
            Wh = W[:, (which * H + h) * d:(which * H + h + 1) * d]      # [d_model, d] of this head
            for b in range(B):
                P[b, h] = X[b] @ Wh
        out.append(P)
    return tuple(out)


# ----------------------------------------------------------------------------
# compression, scores, softmax, compressed output
# ----------------------------------------------------------------------------
def compress(Phi: np.ndarray, X: np.ndarray) -> np.ndarray:
    """X~ = Phi X for one (batch, head): Phi [m,n], X [n,d] -> [m,d]."""
    Phi = np.asarray(Phi, F64)
    X = np.asarray(X, F64)
    assert Phi.ndim == 2 and X.ndim == 2 and Phi.shape[1] == X.shape[0]
    return Phi @ X


def compressed_scores(Q: np.ndarray, Kt: np.ndarray, scale: float | None = None) -> np.ndarray:
    """S[i,r] = scale * <Q_i, K~_r>, scale = 1/sqrt(d_k) by default.  Q [n_q,d], K~ [m,d] -> [n_q,m]."""
    Q = np.asarray(Q, F64)
    Kt = np.asarray(Kt, F64)
    d = Q.shape[1]
    if scale is None:
        scale = 1.0 / np.sqrt(F64(d))
    return (Q @ Kt.T) * F64(scale)


def softmax_rows(S: np.ndarray) -> np.ndarray:
    """Row-wise softmax over the m measurements (last axis), max-subtracted."""
    S = np.asarray(S, F64)
    e = np.exp(S - S.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def compressed_output(A: np.ndarray, Vt: np.ndarray) -> np.ndarray:
    """Z = A~ V~ : [n_q,m] x [m,d] -> [n_q,d]."""
    return np.asarray(A, F64) @ np.asarray(Vt, F64)


# ----------------------------------------------------------------------------
# sparse decoder
# ----------------------------------------------------------------------------
def soft_threshold(x: np.ndarray, theta: float) -> np.ndarray:
    """eta_theta(x) = sign(x) * max(|x| - theta, 0), elementwise."""
    x = np.asarray(x, F64)
    return np.sign(x) * np.maximum(np.abs(x) - F64(theta), 0.0)


def decoder_setup(M: np.ndarray, lam: float, step: float | None = None):
    """ISTA instance of the LISTA weights for the model z = alpha M^T (M is p x q).

    Returns (S_dec [q,q], B_dec [p,q], theta, mu) with
      G = M^T M,  L^ = max_a sum_b |G[a,b]|,  mu = 1/L^ (unless `step` is given),
      S_dec = I - mu G,  B_dec = mu M,  theta = mu * lambda.
    """
    M = np.asarray(M, F64)
    G = M.T @ M
    if step is None or step == 0:
        L = np.abs(G).sum(axis=1).max()
        mu = 1.0 / L
    else:
        mu = F64(step)
    S_dec = np.eye(G.shape[0], dtype=F64) - mu * G
    B_dec = mu * M
    theta = mu * F64(lam)
    return S_dec, B_dec, theta, mu


def ista(Z: np.ndarray, S_dec: np.ndarray, B_dec: np.ndarray, theta: float, T: int,
         return_iterates: bool = False):
    """T iterations alpha^{t+1} = eta_theta(alpha^t S_dec + Z B_dec), alpha^0 = 0, row-wise.

    Z [rows,p], S_dec [q,q], B_dec [p,q] -> alpha [rows,q].
    """
    Z = np.asarray(Z, F64)
    c = Z @ B_dec
    alpha = np.zeros((Z.shape[0], S_dec.shape[0]), dtype=F64)
    its = [alpha]
    for _ in range(int(T)):
        alpha = soft_threshold(alpha @ S_dec + c, theta)
        if return_iterates:
            its.append(alpha)
    return (alpha, its) if return_iterates else alpha


def lista(Z: np.ndarray, S: np.ndarray, B: np.ndarray, thetas, return_iterates: bool = False):
    """LISTA recurrence with supplied ("learned") weights, row-wise:
    alpha^{t+1} = eta_{theta_t}(alpha^t S_t + Z B_t), t = 0 .. T-1, alpha^0 = 0, T = len(thetas).

    Z [rows,p]; thetas: sequence of T thresholds (one per layer) -> alpha [rows,q].
    S [q,q] and B [p,q] (the paper's S, B carry no layer index: shared over the T layers), or one matrix per
    layer, S [T,q,q] and B [T,p,q] (untied layers: layer t uses S[t], B[t]).
    """
    Z = np.asarray(Z, F64)
    S = np.asarray(S, F64)
    B = np.asarray(B, F64)
    thetas = list(thetas)
    if S.ndim != B.ndim:
        raise ValueError("S and B are both shared over the layers or both per layer")
    if S.ndim == 3 and not (S.shape[0] == B.shape[0] == len(thetas)):
        raise ValueError("per-layer weights need one S, one B and one threshold per layer")
    alpha = np.zeros((Z.shape[0], S.shape[-1]), dtype=F64)
    its = [alpha]
    for t, th in enumerate(thetas):
        S_t = S[t] if S.ndim == 3 else S
        B_t = B[t] if B.ndim == 3 else B
        alpha = soft_threshold(alpha @ S_t + Z @ B_t, th)
        if return_iterates:
            its.append(alpha)
    return (alpha, its) if return_iterates else alpha


def reconstruct(alpha: np.ndarray, Psi: np.ndarray | None) -> np.ndarray:
    """C^_i = Psi alpha^_i, row-wise: out = alpha Psi^T (Psi = I when None)."""
    if Psi is None:
        return np.asarray(alpha, F64)
    return np.asarray(alpha, F64) @ np.asarray(Psi, F64).T


def default_decoder_matrix(Phi_h: np.ndarray, d: int) -> np.ndarray:
    """D = leading d x d block of the head's measurement matrix (rows 0..d-1, columns 0..d-1)."""
    Phi_h = np.asarray(Phi_h, F64)
    assert Phi_h.shape[0] >= d and Phi_h.shape[1] >= d, "default decoder matrix needs m >= d and n >= d"
    return Phi_h[:d, :d].copy()


# ----------------------------------------------------------------------------
# the whole forward
# ----------------------------------------------------------------------------
def csat_forward_head(Q, K, V, Phi_h, *, T, lam, Psi=None, D=None, step=None, scale=None,
                      stages: dict | None = None, weights=None, Phi_v_h=None) -> np.ndarray:
    """CSAT forward for one (batch, head).  Q [n_q,d], K,V [n,d], Phi_h [m,n] -> [n_q,d].
    Phi_v_h: separate measurement matrix for the values (the paper's Phi_V; Phi_h is then Phi_K).  The decoder's
    default D is taken from Phi_V (the paper decodes with the values' measurement matrix).
    weights = (S, B, thetas [T]) with S, B [d,d] or per layer [T,d,d] replaces the ISTA-derived decoder by
    supplied LISTA weights (lam, D and step are then unused)."""
    Q = np.asarray(Q, F64)
    d = Q.shape[1]
    Phi_v = Phi_h if Phi_v_h is None else Phi_v_h
    Kt = compress(Phi_h, K)
    Vt = compress(Phi_v, V)
    S = compressed_scores(Q, Kt, scale)
    A = softmax_rows(S)
    Z = compressed_output(A, Vt)
    if stages is not None:
        stages.update(Kt=Kt, Vt=Vt, Z=Z)
    if int(T) == 0:
        return Z
    if weights is not None:
        S_w, B_w, thetas = weights
        assert len(thetas) == int(T)
        alpha = lista(Z, S_w, B_w, thetas)
        if stages is not None:
            stages.update(alpha=alpha)
        return reconstruct(alpha, Psi)
    if D is None:
        D = default_decoder_matrix(Phi_v, d)
    D = np.asarray(D, F64)
    M = D if Psi is None else D @ np.asarray(Psi, F64)
    S_dec, B_dec, theta, mu = decoder_setup(M, lam, step)
    alpha = ista(Z, S_dec, B_dec, theta, T)
    if stages is not None:
        stages.update(alpha=alpha, S_dec=S_dec, B_dec=B_dec, theta=theta, mu=mu)
    return reconstruct(alpha, Psi)


def csat_forward(Q, K, V, Phi, *, T, lam, Psi=None, D=None, step=None, scale=None,
                 stages: list | None = None, weights=None, Phi_V=None) -> np.ndarray:
    """CSAT forward.  Q [B,H,n_q,d], K,V [B,H,n,d], Phi [H,m,n] (one per head, shared over the
    batch, Phi_K = Phi_V), Psi None | [d,d] | [H,d,d], D None | [H,d,d]  ->  out [B,H,n_q,d]."""
    Q = np.asarray(Q)
    B, H, nq, d = Q.shape
    out = np.empty((B, H, nq, d), dtype=F64)
    for b in range(B):
        for h in range(H):
            psi_h = None if Psi is None else (Psi if np.ndim(Psi) == 2 else Psi[h])
            D_h = None if D is None else D[h]
            st = {} if stages is not None else None
            # weights = (S, B, thetas [T,H]) with S, B [H,d,d] (shared over the layers) or [T,H,d,d] (per layer)
            w_h = None
            if weights is not None:
                per_layer = np.ndim(weights[0]) == 4
                w_h = (np.asarray(weights[0])[:, h] if per_layer else weights[0][h],
                       np.asarray(weights[1])[:, h] if per_layer else weights[1][h], [th[h] for th in weights[2]])
            out[b, h] = csat_forward_head(Q[b, h], K[b, h], V[b, h], Phi[h], T=T, lam=lam,
                                          Psi=psi_h, D=D_h, step=step, scale=scale, stages=st, weights=w_h,
                                          Phi_v_h=None if Phi_V is None else Phi_V[h])
            if stages is not None:
                stages.append(st)
    return out


# ----------------------------------------------------------------------------
# backward: d out / d (Q, K, V), chain rule through the forward's equations in reverse order
# ----------------------------------------------------------------------------
def csat_backward_head(Q, K, V, Phi_h, G, *, T, lam, Psi=None, D=None, step=None, scale=None, weights=None,
                       Phi_v_h=None, stages: dict | None = None, masks=None):
    """Vector-Jacobian product of csat_forward_head for one (batch, head): given G = dL/d out [n_q,d], returns
    (dL/dQ [n_q,d], dL/dK [n,d], dL/dV [n,d]).  Phi is a constant.
    The shrinkage eta_theta(x) = x - theta sign(x) where |x| > theta and 0 elsewhere; its derivative with respect
    to x is 1 where |x| > theta and 0 elsewhere (0 is taken at |x| = theta), with respect to theta it is -sign(x)
    where |x| > theta.
    masks (optional, bool [T,n_q,d]): the decisions |x_t| > theta_t taken elsewhere.  The derivative of eta is
    discontinuous, so an implementation in lower precision may decide an entry within rounding distance of its
    threshold the other way; both sides of a comparison then have to use the same decisions.  With masks given,
    layer t differentiates alpha^{t+1} = masks[t] o (x_t - theta_t sign(x_t)); the forward values stay this
    function's own.
    stages (optional dict) receives: xs [T,n_q,d] (the pre-activations x_t), masks [T,n_q,d] (this function's own
    decisions), min_margin [n_q] = min over layers and columns of | |x_t| - theta_t |, dZ, A, Z, and the gradients
    with respect to the decoder's parameters as used in layer t: dS [T,d,d], dB [T,d,d], dtheta [T] (with weights
    shared by the layers the gradient of the shared matrix is the sum over t) and dPsi [d,d] of the
    reconstruction out = alpha Psi^T (None without a dictionary); and dPhi_K = dK~ K^T, dPhi_V = dV~ V^T [m,n], the
    gradients with respect to the measurement matrices through the compression K~ = Phi K, V~ = Phi_V V with the
    decoder's matrices held fixed (a Phi shared by keys and values receives their sum)."""
    Q = np.asarray(Q, F64)
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    G = np.asarray(G, F64)
    Phi_h = np.asarray(Phi_h, F64)
    d = Q.shape[1]
    Phi_v = Phi_h if Phi_v_h is None else np.asarray(Phi_v_h, F64)
    sc = (1.0 / np.sqrt(d)) if scale is None else float(scale)
    # forward, keeping what the backward needs
    Kt = compress(Phi_h, K)
    Vt = compress(Phi_v, V)
    A = softmax_rows(compressed_scores(Q, Kt, scale))
    Z = compressed_output(A, Vt)
    margin = np.full(Q.shape[0], np.inf)
    T = int(T)
    if T == 0:
        dZ = G.copy()
        if stages is not None:
            stages.update(xs=np.zeros((0,) + Z.shape), masks=np.zeros((0,) + Z.shape, dtype=bool),
                          dS=np.zeros((0, d, d)), dB=np.zeros((0, d, d)), dtheta=np.zeros(0), dPsi=None)
    else:
        if weights is not None:
            S_w, B_w, thetas = weights
            S_w, B_w = np.asarray(S_w, F64), np.asarray(B_w, F64)
            S_l = [S_w[t] if S_w.ndim == 3 else S_w for t in range(T)]
            B_l = [B_w[t] if B_w.ndim == 3 else B_w for t in range(T)]
            thetas = [float(th) for th in thetas]
        else:
            Dm = default_decoder_matrix(Phi_v, d) if D is None else np.asarray(D, F64)
            M = Dm if Psi is None else Dm @ np.asarray(Psi, F64)
            S_dec, B_dec, theta, _ = decoder_setup(M, lam, step)
            S_l, B_l, thetas = [S_dec] * T, [B_dec] * T, [float(theta)] * T
        alpha = np.zeros_like(Z)
        alphas, xs = [], []
        for t in range(T):
            x = alpha @ S_l[t] + Z @ B_l[t]
            alphas.append(alpha)
            xs.append(x)
            margin = np.minimum(margin, np.abs(np.abs(x) - thetas[t]).min(axis=1))
            alpha = soft_threshold(x, thetas[t])
        own_masks = np.stack([np.abs(xs[t]) > thetas[t] for t in range(T)])
        use = own_masks if masks is None else np.asarray(masks, dtype=bool)
        assert use.shape == own_masks.shape
        # out = alpha Psi^T  ->  d alpha = G Psi, d Psi = G^T alpha
        d_alpha = G if Psi is None else G @ np.asarray(Psi, F64)
        dPsi = None if Psi is None else G.T @ alpha
        dZ = np.zeros_like(Z)
        dS, dB, dth = np.zeros((T, d, d)), np.zeros((T, d, d)), np.zeros(T)
        for t in range(T - 1, -1, -1):
            dx = d_alpha * use[t]                                # through eta_theta, with respect to x_t
            dth[t] = -(dx * np.sign(xs[t])).sum()                # ... and with respect to theta_t
            dS[t] = alphas[t].T @ dx                             # x_t = alpha_t S_t + Z B_t
            dB[t] = Z.T @ dx
            dZ += dx @ B_l[t].T
            d_alpha = dx @ S_l[t].T
        if stages is not None:
            stages.update(xs=np.stack(xs), masks=own_masks, dS=dS, dB=dB, dtheta=dth, dPsi=dPsi)
    if stages is not None:
        stages.update(min_margin=margin, dZ=dZ, A=A, Z=Z)
    # Z = A~ V~
    dA = dZ @ Vt.T
    dVt = A.T @ dZ
    # A~ = softmax(S) row-wise:  dS = A o (dA - rowsum(dA o A))
    dS_scores = A * (dA - (dA * A).sum(axis=1, keepdims=True))
    # S = sc Q K~^T
    dQ = sc * (dS_scores @ Kt)
    dKt = sc * (dS_scores.T @ Q)
    # K~ = Phi K, V~ = Phi_V V
    dK = Phi_h.T @ dKt
    dV = Phi_v.T @ dVt
    if stages is not None:
        # ... and with respect to the measurement matrices themselves (a learned Phi), the decoder's matrices held
        # fixed: d Phi_K = dK~ K^T, d Phi_V = dV~ V^T, each [m,n]; one shared Phi receives their sum
        stages.update(dPhi_K=dKt @ K.T, dPhi_V=dVt @ V.T)
    return dQ, dK, dV


def csat_backward(Q, K, V, Phi, G, *, T, lam, Psi=None, D=None, step=None, scale=None, weights=None, Phi_V=None,
                  stages: list | None = None, masks=None):
    """Vector-Jacobian product of csat_forward: G [B,H,n_q,d] -> (dQ [B,H,n_q,d], dK [B,H,n,d], dV [B,H,n,d]).
    masks (optional, bool [B,H,T,n_q,d]): shrinkage decisions to differentiate with, see csat_backward_head."""
    Q = np.asarray(Q)
    B, H, nq, d = Q.shape
    n = np.asarray(K).shape[2]
    dQ = np.empty((B, H, nq, d), dtype=F64)
    dK = np.empty((B, H, n, d), dtype=F64)
    dV = np.empty((B, H, n, d), dtype=F64)
    for b in range(B):
        for h in range(H):
            psi_h = None if Psi is None else (Psi if np.ndim(Psi) == 2 else Psi[h])
            D_h = None if D is None else D[h]
            w_h = None
            if weights is not None:
                per_layer = np.ndim(weights[0]) == 4
                w_h = (np.asarray(weights[0])[:, h] if per_layer else weights[0][h],
                       np.asarray(weights[1])[:, h] if per_layer else weights[1][h], [th[h] for th in weights[2]])
            st = {} if stages is not None else None
            dQ[b, h], dK[b, h], dV[b, h] = csat_backward_head(
                Q[b, h], K[b, h], V[b, h], Phi[h], G[b, h], T=T, lam=lam, Psi=psi_h, D=D_h, step=step, scale=scale,
                weights=w_h, Phi_v_h=None if Phi_V is None else Phi_V[h], stages=st,
                masks=None if masks is None else np.asarray(masks)[b, h])
            if stages is not None:
                stages.append(st)
    return dQ, dK, dV
