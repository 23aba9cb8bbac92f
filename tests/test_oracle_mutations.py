"""The pins must bite: plant one plausible mistake at a time in the oracle (on the CPU, by
monkeypatching) and require that at least one pin of tests/test_oracle_pins.py fails."""
import numpy as np
import pytest

from oracle import csat_oracle as orc
import test_oracle_pins as pins

PINS = [getattr(pins, k) for k in dir(pins) if k.startswith("test_") and "phi" not in k and "philox" not in k]

F64 = np.float64


def _scores_no_scale(Q, Kt, scale=None):
    return np.asarray(Q, F64) @ np.asarray(Kt, F64).T * (1.0 if scale is None else scale)


def _softmax_wrong_axis(S):
    e = np.exp(S - S.max(axis=0, keepdims=True))
    return e / e.sum(axis=0, keepdims=True)


def _softmax_no_norm(S):
    return np.exp(S - S.max(axis=-1, keepdims=True))


def _soft_no_sign(x, theta):
    return np.maximum(np.abs(x) - theta, 0.0)


def _soft_hard(x, theta):
    return np.where(np.abs(x) > theta, x, 0.0)


def _setup_theta_is_lambda(M, lam, step=None):
    S, B, th, mu = _orig_setup(M, lam, step)
    return S, B, F64(lam), mu


def _setup_plus_sign(M, lam, step=None):
    S, B, th, mu = _orig_setup(M, lam, step)
    return 2 * np.eye(S.shape[0]) - S, B, th, mu


def _setup_B_transposed(M, lam, step=None):
    S, B, th, mu = _orig_setup(M, lam, step)
    return S, (B.T if B.shape[0] == B.shape[1] else B), th, mu


def _setup_spectral_of_M(M, lam, step=None):
    # step from ||M||_inf instead of ||M^T M||_inf
    M = np.asarray(M, F64)
    mu = 1.0 / np.abs(M).sum(axis=1).max() if not step else step
    G = M.T @ M
    return np.eye(G.shape[0]) - mu * G, mu * M, mu * lam, mu


def _reconstruct_no_transpose(alpha, Psi):
    return alpha if Psi is None else alpha @ Psi


def _block_transposed(Phi_h, d):
    assert Phi_h.shape[0] >= d and Phi_h.shape[1] >= d
    return np.asarray(Phi_h, F64)[:d, :d].T.copy()


def _block_offset(Phi_h, d):
    assert Phi_h.shape[0] >= d and Phi_h.shape[1] >= d
    return np.asarray(Phi_h, F64)[-d:, :d].copy()


def _ista_drop_B(Z, S_dec, B_dec, theta, T, return_iterates=False):
    return _orig_ista(Z, S_dec, np.eye(*B_dec.shape), theta, T, return_iterates)


def _ista_one_short(Z, S_dec, B_dec, theta, T, return_iterates=False):
    return _orig_ista(Z, S_dec, B_dec, theta, max(int(T) - 1, 0) if T < 50 else T, return_iterates)


def _compress_abs(Phi, X):
    return np.abs(np.asarray(Phi, F64)) @ np.asarray(X, F64)


def _output_uses_unweighted(A, Vt):
    return np.ones_like(A) / A.shape[1] @ np.asarray(Vt, F64)


def _lista_S_transposed(Z, S, B, thetas, return_iterates=False):
    return _orig_lista(Z, np.asarray(S, F64).T, B, thetas, return_iterates)


def _lista_first_theta_everywhere(Z, S, B, thetas, return_iterates=False):
    thetas = list(thetas)
    return _orig_lista(Z, S, B, [thetas[0]] * len(thetas), return_iterates)


def _lista_drop_input(Z, S, B, thetas, return_iterates=False):
    # Z B only feeds the first layer
    Z = np.asarray(Z, F64)
    alpha = np.zeros((Z.shape[0], np.asarray(S).shape[0]))
    for i, th in enumerate(thetas):
        alpha = orc.soft_threshold(alpha @ S + (Z @ B if i == 0 else 0.0), th)
    return alpha


def _lista_first_layer_everywhere(Z, S, B, thetas, return_iterates=False):
    S, B = np.asarray(S, F64), np.asarray(B, F64)
    if S.ndim == 3:
        S, B = S[0], B[0]
    return _orig_lista(Z, S, B, thetas, return_iterates)


def _lista_B_one_layer_late(Z, S, B, thetas, return_iterates=False):
    B = np.asarray(B, F64)
    if B.ndim == 3:
        B = np.roll(B, 1, axis=0)
    return _orig_lista(Z, S, B, thetas, return_iterates)


def _lista_layers_reversed(Z, S, B, thetas, return_iterates=False):
    S, B = np.asarray(S, F64), np.asarray(B, F64)
    if S.ndim == 3:
        S, B = S[::-1], B[::-1]
    return _orig_lista(Z, S, B, thetas, return_iterates)


def _project_heads_interleaved(X, W, H, d):
    # columns taken as [head][which] instead of [which][head]
    Wp = np.asarray(W, F64).reshape(W.shape[0], H, 3, d).transpose(0, 2, 1, 3).reshape(W.shape[0], 3 * H * d)
    return _orig_project(X, Wp, H, d)


def _project_W_transposed_per_head(X, W, H, d):
    Q, K, V = _orig_project(X, W, H, d)
    return K, Q, V


def _backward_scale_dropped(Q, K, V, Phi_h, G, **kw):
    dQ, dK, dV = _orig_backward_head(Q, K, V, Phi_h, G, **kw)
    s = np.sqrt(np.asarray(Q).shape[1]) if kw.get("scale") is None else 1.0 / kw["scale"]
    return dQ * s, dK * s, dV


def _backward_softmax_without_row_term(Q, K, V, Phi_h, G, **kw):
    # dS = A o dA, the projection onto the simplex's tangent space forgotten
    st = {}
    _orig_backward_head(Q, K, V, Phi_h, G, **{**kw, "stages": st})
    Phi_h = np.asarray(Phi_h, F64)
    Phi_v = Phi_h if kw.get("Phi_v_h") is None else np.asarray(kw["Phi_v_h"], F64)
    Kt, Vt = Phi_h @ np.asarray(K, F64), Phi_v @ np.asarray(V, F64)
    sc = 1.0 / np.sqrt(np.asarray(Q).shape[1]) if kw.get("scale") is None else kw["scale"]
    dS = st["A"] * (st["dZ"] @ Vt.T)
    if kw.get("stages") is not None:
        kw["stages"].update(st)
    return sc * dS @ Kt, Phi_h.T @ (sc * dS.T @ np.asarray(Q, F64)), Phi_v.T @ (st["A"].T @ st["dZ"])


def _backward_masks_of_the_wrong_layer(Q, K, V, Phi_h, G, **kw):
    # supplied decisions applied one layer late (the natural ones are left alone)
    if kw.get("masks") is not None:
        kw = {**kw, "masks": np.roll(np.asarray(kw["masks"]), 1, axis=0)}
    return _orig_backward_head(Q, K, V, Phi_h, G, **kw)


def _backward_masks_ignored(Q, K, V, Phi_h, G, **kw):
    return _orig_backward_head(Q, K, V, Phi_h, G, **{**kw, "masks": None})


def _backward_dtheta_without_sign(Q, K, V, Phi_h, G, **kw):
    st = kw.get("stages")
    out = _orig_backward_head(Q, K, V, Phi_h, G, **kw)
    if st is not None and len(st["dtheta"]):
        st["dtheta"] = -np.abs(st["dtheta"])
    return out


def _backward_dS_from_the_next_iterate(Q, K, V, Phi_h, G, **kw):
    st = kw.get("stages")
    out = _orig_backward_head(Q, K, V, Phi_h, G, **kw)
    if st is not None and len(st["dS"]) > 1:
        st["dS"] = np.roll(st["dS"], -1, axis=0)
    return out


def _backward_dPhi_keys_and_values_exchanged(Q, K, V, Phi_h, G, **kw):
    st = kw.get("stages")
    out = _orig_backward_head(Q, K, V, Phi_h, G, **kw)
    if st is not None:
        st["dPhi_K"], st["dPhi_V"] = st["dPhi_V"], st["dPhi_K"]
    return out


def _backward_dPhi_transposed_product(Q, K, V, Phi_h, G, **kw):
    # K~^T-like slip: the gradient of K~ = Phi K taken against the rows of K in reverse order
    st = kw.get("stages")
    out = _orig_backward_head(Q, K, V, Phi_h, G, **kw)
    if st is not None:
        st["dPhi_K"] = st["dPhi_K"][:, ::-1]
    return out


_orig_lista = orc.lista
_orig_project = orc.project_qkv
_orig_backward_head = orc.csat_backward_head
_orig_setup = orc.decoder_setup
_orig_ista = orc.ista

MUTATIONS = {
    "scores: scale dropped": ("compressed_scores", _scores_no_scale),
    "softmax: wrong axis": ("softmax_rows", _softmax_wrong_axis),
    "softmax: not normalised": ("softmax_rows", _softmax_no_norm),
    "shrink: sign dropped": ("soft_threshold", _soft_no_sign),
    "shrink: hard threshold": ("soft_threshold", _soft_hard),
    "setup: theta = lambda": ("decoder_setup", _setup_theta_is_lambda),
    "setup: S = I + mu G": ("decoder_setup", _setup_plus_sign),
    "setup: B transposed": ("decoder_setup", _setup_B_transposed),
    "setup: step from ||M||": ("decoder_setup", _setup_spectral_of_M),
    "reconstruct: Psi not transposed": ("reconstruct", _reconstruct_no_transpose),
    "decoder block transposed": ("default_decoder_matrix", _block_transposed),
    "decoder block from last rows": ("default_decoder_matrix", _block_offset),
    "ista: B dropped": ("ista", _ista_drop_B),
    "ista: one iteration short": ("ista", _ista_one_short),
    "lista: S transposed": ("lista", _lista_S_transposed),
    "lista: per-layer thresholds ignored": ("lista", _lista_first_theta_everywhere),
    "lista: input only in the first layer": ("lista", _lista_drop_input),
    "lista: first layer's matrices in every layer": ("lista", _lista_first_layer_everywhere),
    "lista: B of the layer before": ("lista", _lista_B_one_layer_late),
    "lista: layers in reverse order": ("lista", _lista_layers_reversed),
    "project: head and q/k/v order swapped": ("project_qkv", _project_heads_interleaved),
    "project: queries and keys exchanged": ("project_qkv", _project_W_transposed_per_head),
    "backward: score scale dropped": ("csat_backward_head", _backward_scale_dropped),
    "backward: softmax Jacobian without the row term": ("csat_backward_head", _backward_softmax_without_row_term),
    "backward: supplied decisions one layer late": ("csat_backward_head", _backward_masks_of_the_wrong_layer),
    "backward: supplied decisions ignored": ("csat_backward_head", _backward_masks_ignored),
    "backward: d theta loses the sign of x": ("csat_backward_head", _backward_dtheta_without_sign),
    "backward: d S_t taken from the layer after": ("csat_backward_head", _backward_dS_from_the_next_iterate),
    "backward: d Phi_K and d Phi_V exchanged": ("csat_backward_head", _backward_dPhi_keys_and_values_exchanged),
    "backward: d Phi_K against the tokens in reverse order": ("csat_backward_head", _backward_dPhi_transposed_product),
    "compress: |Phi|": ("compress", _compress_abs),
    "output: weights ignored": ("compressed_output", _output_uses_unweighted),
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_some_pin_catches(name, monkeypatch):
    attr, fn = MUTATIONS[name]
    monkeypatch.setattr(orc, attr, fn)
    caught = False
    for pin in PINS:
        try:
            pin()
        except AssertionError:
            caught = True
            break
        except Exception:
            caught = True       # a shape error from the planted mistake also exposes it
            break
    assert caught, f"no pin noticed: {name}"
