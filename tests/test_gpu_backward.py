"""GPU parity of csat_backward (gradients with respect to Q, K, V) against the float64 oracle.

The derivative of the shrinkage is discontinuous at |x| = theta, so an entry whose pre-activation x_t lies within
rounding distance of its threshold may be decided the other way on the GPU.  The comparison therefore has two
parts, as for any result where floating point takes a discrete decision:
  1. the decisions: the library exports the ones it took (CSAT_KEEP_MASKS, csat_get_backward_masks); wherever they
     differ from the oracle's, the oracle's x_t must lie within the forward's own error bar of the threshold
     (the parity tolerance times max |x_t|), and such entries must be few;
  2. the gradients: the oracle differentiates with the library's decisions (its forward values stay its own) and
     every gradient is compared element by element, max |gpu - oracle| / max |oracle| <= the forward's tolerance
     (2e-2 with bf16 storage; float32: 2e-5, measured ~1e-6).
The output gradient G is random.  dK~ and dV~ are sums over the query rows, so with an unlucky draw the column sums
of dZ cancel far below their typical 1/sqrt(n_q) of the sum of magnitudes; the gradient is then a difference of
nearly equal terms and magnifies the bf16 rounding of its operands (one of ten draws did for the sparse case: 1 %
cancellation, 4 % error from rounding P alone in float64 emulation, 0.3-0.9 % for the other nine).  The test
asserts, from the oracle alone, that the draw's cancellation is typical, so that the bar measures the kernel and
not the draw."""
import numpy as np
import pytest
import torch

from oracle import csat_oracle as orc
from paper_2507_02957_b200 import binding, workloads as wl
from gpu_util import TOL, device_inputs, make_ctx, rel_err, to_dev, to_np

pytestmark = pytest.mark.gpu
C = wl.CONFIGS


CASES = {
    "c1_fp32": lambda: C["c1"],
    "fp32_T0": lambda: wl.shrink(C["c1"], n=96, n_q=40, m=32, T=0),
    "fp32_cross_d32": lambda: wl.shrink(C["c1"], B=2, H=2, n=100, n_q=37, m=40, d=32, T=6),
    "bf16_d64": lambda: wl.shrink(C["c2"], B=2, H=3, n_q=150, lam=0.01),
    "bf16_d64_sparse": lambda: wl.shrink(C["c2"], B=2, H=3, n_q=150),
    "bf16_d128": lambda: wl.shrink(C["c5"], B=1, H=2, n=512, n_q=200, m=160, T=8, lam=0.002),
}


BWD_TOL = {"bf16": 2e-2, "fp32": 2e-5}
G_SEED = 103


@pytest.mark.parametrize("name", sorted(CASES))
@pytest.mark.parametrize("variant", ["default", "psi_separate_untied"])
def test_backward_matches_oracle(name, variant):
    w = CASES[name]()
    if variant != "default" and w.T == 0:
        pytest.skip("no decoder without recovery layers")
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    binding.csat_set_i64(ctx.h, binding.CSAT_KEEP_MASKS, 1)
    r = np.random.default_rng(97)
    d, H, T = w.d, w.H, w.T
    kw = dict(T=T, lam=w.lam)
    if variant == "psi_separate_untied":
        Psi = wl.round_to_storage((np.eye(d) + 0.3 * r.standard_normal((d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        ctx.set_dictionary(to_dev(Psi, w.dtype))
        ctx.set(separate_phi=True)
        S = wl.round_to_storage((0.6 * np.eye(d) + 0.4 * r.standard_normal((T, H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        Bm = wl.round_to_storage((r.standard_normal((T, H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        st0 = []
        orc.csat_forward(inp["Q"][:1], inp["K"][:1], inp["V"][:1], to_np(ctx.get_phi())[:H], T=0, lam=0.0, stages=st0)
        th0 = float(np.median(np.abs(st0[0]["Z"] @ Bm[0, 0].astype(np.float64))))
        thetas = (th0 * r.uniform(0.2, 1.5, size=(T, H))).astype(np.float32)
        ctx.set_lista_layer_weights(to_dev(S, w.dtype), to_dev(Bm, w.dtype), torch.from_numpy(thetas).cuda())
        kw.update(Psi=Psi.astype(np.float64), weights=(S.astype(np.float64), Bm.astype(np.float64), list(thetas.astype(np.float64))))
    phi = to_np(ctx.get_phi())
    if variant == "psi_separate_untied":
        kw.update(Phi_V=phi[H:])
        phi = phi[:H]
    G = wl.round_to_storage(np.random.default_rng(G_SEED).standard_normal(inp["Q"].shape).astype(np.float32), w.dtype)
    got = ctx.backward(Q, K, V, to_dev(G, w.dtype))
    assert binding.csat_last_launch_count(ctx.h) >= 4
    tol = BWD_TOL[w.dtype]
    masks = None
    if T > 0:
        # part 1: the decisions
        words = ctx.backward_masks().cpu().numpy().astype(np.uint32)                 # [B,H,n_q,d]
        masks = np.stack([(words >> t) & 1 for t in range(T)], axis=2).astype(bool)    # [B,H,T,n_q,d]
        stages = []
        orc.csat_backward(inp["Q"], inp["K"], inp["V"], phi, G, stages=stages, **kw)
        own = np.stack([s["masks"] for s in stages]).reshape(masks.shape)
        xs = np.stack([s["xs"] for s in stages]).reshape(masks.shape)
        if "weights" in kw:
            th = np.asarray(kw["weights"][2], dtype=np.float64).T[None, :, :, None, None]      # [1,H,T,1,1]
        else:
            st1 = []
            orc.csat_forward(inp["Q"][:1], inp["K"][:1], inp["V"][:1], phi, T=1, lam=w.lam, stages=st1)
            th = np.asarray([s["theta"] for s in st1])[None, :, None, None, None]
        for st in stages:                     # the draw of G is not a degenerate one (see the file header)
            col_abs = np.abs(st["dZ"]).sum(axis=0).max()
            if col_abs > 0:
                assert np.abs(st["dZ"].sum(axis=0)).max() / col_abs >= 0.25 / np.sqrt(w.n_q), (name, variant)
        differ = masks != own
        assert differ.mean() <= (2e-2 if w.dtype == "bf16" else 1e-4), (name, variant, differ.mean())
        bar = TOL[w.dtype] * np.abs(xs).max(axis=(3, 4), keepdims=True)               # per (b, h, layer)
        dist = np.abs(np.abs(xs) - th)
        assert (dist[differ] <= np.broadcast_to(bar, dist.shape)[differ]).all(), (name, variant)
    # part 2: the gradients, with the library's decisions
    ref = orc.csat_backward(inp["Q"], inp["K"], inp["V"], phi, G, masks=masks, **kw)
    for nm, g, rf in zip(("dQ", "dK", "dV"), got, ref):
        g = to_np(g)
        assert np.isfinite(g).all()
        assert np.abs(rf).max() > 0
        err = rel_err(g, rf)
        assert err <= tol, (name, variant, nm, err)
    # deterministic (no atomics)
    again = ctx.backward(Q, K, V, to_dev(G, w.dtype))
    for a, b in zip(got, again):
        assert torch.equal(a, b)
    ctx.close()


def test_backward_masks_need_the_key():
    ctx = binding.Csat(64, 16, 8, 1, 0, dtype="fp32", T=2)
    x = torch.zeros(1, 1, 64, 8, device="cuda")
    ctx.backward(x, x, x, x)
    with pytest.raises(binding.CsatError) as ei:
        ctx.backward_masks()
    assert ei.value.code == 6
    binding.csat_set_i64(ctx.h, binding.CSAT_KEEP_MASKS, 1)
    ctx.backward(x, x, x, x)
    assert ctx.backward_masks().shape == (1, 1, 64, 8)
    ctx.close()


def test_backward_refuses_what_it_does_not_cover():
    ctx = binding.Csat(64, 16, 8, 1, 0, dtype="fp32", T=33)
    x = torch.zeros(1, 1, 64, 8, device="cuda")
    with pytest.raises(binding.CsatError) as ei:
        ctx.backward(x, x, x, x)
    assert ei.value.code == 5
    ctx.set(T=2)
    ctx.backward(x, x, x, x)                     # the context stays usable
    ctx.close()


def test_backward_tensor_core_path_takes_more_than_32_layers():
    """The tensor-core path keeps its decisions per layer, so CSAT_T is not bounded by a word's 32 bits there.  With
    lambda = 0 every decision is |x| > 0, the same on both sides, so the oracle needs no decisions supplied."""
    w = wl.shrink(C["c2"], B=1, H=2, n_q=150, T=40, lam=0.0)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    phi = to_np(ctx.get_phi())
    G = wl.round_to_storage(np.random.default_rng(G_SEED).standard_normal(inp["Q"].shape).astype(np.float32), w.dtype)
    got = ctx.backward(Q, K, V, to_dev(G, w.dtype))
    ref = orc.csat_backward(inp["Q"], inp["K"], inp["V"], phi, G, T=w.T, lam=0.0)
    for nm, g, rf in zip(("dQ", "dK", "dV"), got, ref):
        assert rel_err(to_np(g), rf) <= BWD_TOL["bf16"], nm
    binding.csat_set_i64(ctx.h, binding.CSAT_KEEP_MASKS, 1)          # one word per entry: 32 layers at most
    with pytest.raises(binding.CsatError) as ei:
        ctx.backward(Q, K, V, to_dev(G, w.dtype))
    assert ei.value.code == 5
    ctx.close()


EDGE = {
    # (workload, tied LISTA weights with one threshold per layer?)
    "one_layer": (wl.shrink(C["c2"], B=1, H=2, n_q=130, T=1, lam=0.01), False),
    "thirty_two_layers": (wl.shrink(C["c2"], B=1, H=1, n_q=64, T=32, lam=0.01), False),
    "zero_threshold": (wl.shrink(C["c2"], B=1, H=2, n_q=77, T=3, lam=0.0), False),
    "single_query_d128": (wl.shrink(C["c5"], B=1, H=2, n=256, n_q=1, m=128, T=4, lam=0.002), False),
    "per_layer_thresholds_d128": (wl.shrink(C["c5"], B=2, H=1, n=320, n_q=129, m=192, T=5, lam=0.002), True),
}


@pytest.mark.parametrize("name", sorted(EDGE))
def test_backward_edge_cases_on_the_tensor_core_path(name):
    """Depths 1 and 32, a zero threshold (eta is the identity: every decision is 1), a single query, 129 queries (a
    second tile with one live row), and supplied tied weights with one threshold per layer: all bf16 with d in
    {64, 128}, i.e. the tensor-core kernels.  Same two-part comparison as above."""
    w, per_layer = EDGE[name]
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    binding.csat_set_i64(ctx.h, binding.CSAT_KEEP_MASKS, 1)
    r = np.random.default_rng(11)
    d, H, T = w.d, w.H, w.T
    kw = dict(T=T, lam=w.lam)
    phi = to_np(ctx.get_phi())
    if per_layer:
        S = wl.round_to_storage((0.6 * np.eye(d) + 0.4 * r.standard_normal((H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        Bm = wl.round_to_storage((r.standard_normal((H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        st0 = []
        orc.csat_forward(inp["Q"][:1], inp["K"][:1], inp["V"][:1], phi, T=0, lam=0.0, stages=st0)
        th0 = float(np.median(np.abs(st0[0]["Z"] @ Bm[0].astype(np.float64))))
        thetas = (th0 * r.uniform(0.2, 1.5, size=(T, H))).astype(np.float32)
        ctx.set_lista_weights(to_dev(S, w.dtype), to_dev(Bm, w.dtype), torch.from_numpy(thetas).cuda())
        kw.update(weights=(S.astype(np.float64), Bm.astype(np.float64), list(thetas.astype(np.float64))))
    G = wl.round_to_storage(np.random.default_rng(G_SEED).standard_normal(inp["Q"].shape).astype(np.float32), w.dtype)
    got = ctx.backward(Q, K, V, to_dev(G, w.dtype))
    words = ctx.backward_masks().cpu().numpy().astype(np.uint32)
    masks = np.stack([(words >> t) & 1 for t in range(T)], axis=2).astype(bool)
    stages = []
    orc.csat_backward(inp["Q"], inp["K"], inp["V"], phi, G, stages=stages, **kw)
    own = np.stack([s["masks"] for s in stages]).reshape(masks.shape)
    xs = np.stack([s["xs"] for s in stages]).reshape(masks.shape)
    differ = masks != own
    if name == "zero_threshold":
        assert masks.all()
    assert differ.mean() <= 2e-2, (name, differ.mean())
    if "weights" in kw:
        th = np.asarray(kw["weights"][2], dtype=np.float64).T[None, :, :, None, None]
    else:
        st1 = []
        orc.csat_forward(inp["Q"][:1], inp["K"][:1], inp["V"][:1], phi, T=1, lam=w.lam, stages=st1)
        th = np.asarray([s["theta"] for s in st1])[None, :, None, None, None]
    bar = TOL[w.dtype] * np.abs(xs).max(axis=(3, 4), keepdims=True)
    dist = np.abs(np.abs(xs) - th)
    assert (dist[differ] <= np.broadcast_to(bar, dist.shape)[differ]).all(), name
    ref = orc.csat_backward(inp["Q"], inp["K"], inp["V"], phi, G, masks=masks, **kw)
    for nm, g, rf in zip(("dQ", "dK", "dV"), got, ref):
        assert np.abs(rf).max() > 0
        err = rel_err(to_np(g), rf)
        assert err <= BWD_TOL[w.dtype], (name, nm, err)
    ctx.close()


def _random_backward_shapes():
    """Seeded random shapes for both backward paths (bf16 with d in {64, 128}: tensor cores; the rest: FFMA kernels):
    query, token and measurement counts that are no multiples of any tile, lambda = 0 so that every decision is
    |x| > 0 on both sides and the oracle needs no decisions supplied."""
    r = np.random.default_rng(4048)
    out = []
    for i in range(10):
        tc = i % 2 == 0
        dtype = "bf16" if tc else "fp32"
        d = (64, 128)[(i // 2) % 2] if tc else int(r.choice([8, 24, 40]))
        m = int(r.integers(d, 2 * d + 70))
        n = int(r.integers(m, m + 400))
        out.append(wl.Workload(f"bwrand{i}", int(r.integers(1, 3)), int(r.integers(1, 4)), n, int(r.integers(1, 300)), d, m,
                               dtype, int(r.integers(0, 5)), 0.0, "iid", 700 + i))
    return out


@pytest.mark.parametrize("w", _random_backward_shapes(), ids=lambda w: f"{w.name}_{w.dtype}_B{w.B}H{w.H}_n{w.n}_nq{w.n_q}_d{w.d}_m{w.m}_T{w.T}")
def test_backward_random_shapes_match_oracle(w):
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    phi = to_np(ctx.get_phi())
    G = wl.round_to_storage(np.random.default_rng(G_SEED + 1).standard_normal(inp["Q"].shape).astype(np.float32), w.dtype)
    got = ctx.backward(Q, K, V, to_dev(G, w.dtype))
    ref = orc.csat_backward(inp["Q"], inp["K"], inp["V"], phi, G, T=w.T, lam=0.0)
    for nm, g, rf in zip(("dQ", "dK", "dV"), got, ref):
        g = to_np(g)
        assert np.isfinite(g).all()
        assert rel_err(g, rf) <= BWD_TOL[w.dtype], (w, nm, rel_err(g, rf))
    ctx.close()


WGRAD_CASES = {
    "bf16_d64": lambda: wl.shrink(C["c2"], B=2, H=3, n_q=150, lam=0.01),
    "bf16_d64_T1": lambda: wl.shrink(C["c2"], B=1, H=2, n_q=77, T=1, lam=0.01),
    "bf16_d128": lambda: wl.shrink(C["c5"], B=2, H=2, n=512, n_q=200, m=160, T=8, lam=0.002),
}


@pytest.mark.parametrize("name", sorted(WGRAD_CASES))
@pytest.mark.parametrize("with_psi", [False, True], ids=["identity", "dictionary"])
def test_weight_gradients_match_oracle(name, with_psi):
    """Gradients with respect to the decoder's S, B, thresholds and dictionary (CSAT_WEIGHT_GRADS), against the oracle's
    per-layer gradients summed over the layers (one S, B for all layers) and over the batch, with the library's own
    shrinkage decisions (the same protocol as for dQ, dK, dV) and the same tolerance."""
    w = WGRAD_CASES[name]()
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    binding.csat_set_i64(ctx.h, binding.CSAT_KEEP_MASKS, 1)
    binding.csat_set_i64(ctx.h, binding.CSAT_WEIGHT_GRADS, 1)
    d, H, T, B = w.d, w.H, w.T, w.B
    kw = dict(T=T, lam=w.lam)
    if with_psi:
        r = np.random.default_rng(97)
        Psi = wl.round_to_storage((np.eye(d) + 0.3 * r.standard_normal((d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        ctx.set_dictionary(to_dev(Psi, w.dtype))
        kw.update(Psi=Psi.astype(np.float64))
    phi = to_np(ctx.get_phi())
    G = wl.round_to_storage(np.random.default_rng(G_SEED).standard_normal(inp["Q"].shape).astype(np.float32), w.dtype)
    got_in = ctx.backward(Q, K, V, to_dev(G, w.dtype))
    words = ctx.backward_masks().cpu().numpy().astype(np.uint32)
    masks = np.stack([(words >> t) & 1 for t in range(T)], axis=2).astype(bool)
    stages = []
    ref_in = orc.csat_backward(inp["Q"], inp["K"], inp["V"], phi, G, masks=masks, stages=stages, **kw)
    assert len(stages) == B * H
    dS = np.zeros((H, d, d)); dB = np.zeros((H, d, d)); dth = np.zeros((T, H)); dPsi = np.zeros((d, d))
    for b in range(B):
        for h in range(H):
            st = stages[b * H + h]
            dS[h] += st["dS"].sum(axis=0)
            dB[h] += st["dB"].sum(axis=0)
            dth[:, h] += st["dtheta"]
            if with_psi:
                dPsi += st["dPsi"]
    gS, gB, gth, gPsi = (x.cpu().numpy().astype(np.float64) for x in ctx.weight_grads())
    tol = BWD_TOL[w.dtype]
    for nm, g, rf in (("dS", gS, dS), ("dB", gB, dB), ("dtheta", gth, dth)) + ((("dPsi", gPsi, dPsi),) if with_psi else ()):
        assert np.isfinite(g).all()
        if T == 1 and nm == "dS":                 # alpha^0 = 0: the only layer has no input iterate
            assert np.abs(rf).max() == 0.0 and np.abs(g).max() == 0.0
            continue
        assert np.abs(rf).max() > 0, nm
        assert rel_err(g, rf) <= tol, (name, with_psi, nm, rel_err(g, rf))
    if not with_psi:
        assert np.abs(gPsi).max() == 0.0
    # the input gradients are what they are without the key
    for g, rf in zip(got_in, ref_in):
        assert rel_err(to_np(g), rf) <= tol
    # bit-identical on a second run (fixed-order sums)
    ctx.backward(Q, K, V, to_dev(G, w.dtype))
    for a, b_ in zip((gS, gB, gth, gPsi), ctx.weight_grads()):
        assert np.array_equal(a, b_.cpu().numpy().astype(np.float64))
    ctx.close()


def test_weight_gradients_need_the_key_and_the_tensor_core_path():
    ctx = binding.Csat(64, 16, 8, 1, 0, dtype="fp32", T=2)
    x = torch.zeros(1, 1, 64, 8, device="cuda")
    ctx.backward(x, x, x, x)
    with pytest.raises(binding.CsatError) as ei:
        ctx.weight_grads()
    assert ei.value.code == 6
    binding.csat_set_i64(ctx.h, binding.CSAT_WEIGHT_GRADS, 1)
    with pytest.raises(binding.CsatError) as ei:
        ctx.backward(x, x, x, x)                # float32 context: FFMA kernels
    assert ei.value.code == 5
    ctx.close()


PHIGRAD_CASES = {
    "bf16_d64": lambda: wl.shrink(C["c2"], B=2, H=3, n_q=150, lam=0.01),                            # n = 197: ragged, odd
    "bf16_d128": lambda: wl.shrink(C["c5"], B=2, H=2, n=520, n_q=200, m=160, T=8, lam=0.002),       # m, n ragged tiles
    "bf16_d64_T0": lambda: wl.shrink(C["c2"], B=1, H=2, n=300, n_q=77, m=130, T=0),
}


@pytest.mark.parametrize("name", sorted(PHIGRAD_CASES))
@pytest.mark.parametrize("separate", [False, True], ids=["shared_phi", "separate_phi"])
def test_measurement_matrix_gradient_matches_oracle(name, separate):
    """csat_backward_phi (d Phi = sum over the batch of dK~ K^T + dV~ V^T, decoder held fixed) against the oracle's
    dPhi_K, dPhi_V summed the same way, with the library's shrinkage decisions; element by element, the tolerance of
    every other gradient."""
    w = PHIGRAD_CASES[name]()
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    if separate:
        ctx.set(separate_phi=True)
    binding.csat_set_i64(ctx.h, binding.CSAT_KEEP_MASKS, 1)
    H, T, B = w.H, w.T, w.B
    phi = to_np(ctx.get_phi())
    kw = dict(T=T, lam=w.lam)
    if separate:
        kw.update(Phi_V=phi[H:])
        phi = phi[:H]
    G = wl.round_to_storage(np.random.default_rng(G_SEED).standard_normal(inp["Q"].shape).astype(np.float32), w.dtype)
    ctx.backward(Q, K, V, to_dev(G, w.dtype))
    masks = None
    if T > 0:
        words = ctx.backward_masks().cpu().numpy().astype(np.uint32)
        masks = np.stack([(words >> t) & 1 for t in range(T)], axis=2).astype(bool)
    got = ctx.backward_phi(K, V).cpu().numpy().astype(np.float64)
    stages = []
    orc.csat_backward(inp["Q"], inp["K"], inp["V"], phi, G, masks=masks, stages=stages, **kw)
    ref = np.zeros_like(got)
    for b in range(B):
        for h in range(H):
            st = stages[b * H + h]
            if separate:
                ref[h] += st["dPhi_K"]
                ref[H + h] += st["dPhi_V"]
            else:
                ref[h] += st["dPhi_K"] + st["dPhi_V"]
    assert got.shape == ((2 * H if separate else H), w.m, w.n)
    assert np.isfinite(got).all() and np.abs(ref).max() > 0
    assert rel_err(got, ref) <= BWD_TOL[w.dtype], (name, separate, rel_err(got, ref))
    assert torch.equal(ctx.backward_phi(K, V), torch.from_numpy(got.astype(np.float32)).cuda())
    ctx.close()


def test_measurement_matrix_gradient_needs_a_backward_first():
    w = wl.shrink(C["c2"], B=1, H=1, n_q=64, T=2)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    with pytest.raises(binding.CsatError) as ei:
        ctx.backward_phi(K, V)
    assert ei.value.code == 6
    ctx.close()


@pytest.mark.parametrize("T", [1, 2, 3, 5])
@pytest.mark.parametrize("with_psi", [False, True], ids=["identity", "dictionary"])
def test_backward_with_per_layer_weights_small_depths(T, with_psi):
    """One S_t, B_t per layer on the tensor-core path at the depths where its two-stage ring of layer matrices starts,
    wraps and ends (1, 2, 3, 5 layers), with and without a dictionary; the usual two-part comparison."""
    w = wl.shrink(C["c2"], B=1, H=2, n_q=100, T=T, lam=0.01)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    binding.csat_set_i64(ctx.h, binding.CSAT_KEEP_MASKS, 1)
    r = np.random.default_rng(11 + T)
    d, H = w.d, w.H
    kw = dict(T=T, lam=w.lam)
    if with_psi:
        Psi = wl.round_to_storage((np.eye(d) + 0.3 * r.standard_normal((d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        ctx.set_dictionary(to_dev(Psi, w.dtype))
        kw.update(Psi=Psi.astype(np.float64))
    S = wl.round_to_storage((0.6 * np.eye(d) + 0.4 * r.standard_normal((T, H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
    Bm = wl.round_to_storage((r.standard_normal((T, H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
    phi = to_np(ctx.get_phi())
    st0 = []
    orc.csat_forward(inp["Q"][:1], inp["K"][:1], inp["V"][:1], phi, T=0, lam=0.0, stages=st0)
    th0 = float(np.median(np.abs(st0[0]["Z"] @ Bm[0, 0].astype(np.float64))))
    thetas = (th0 * r.uniform(0.2, 1.5, size=(T, H))).astype(np.float32)
    ctx.set_lista_layer_weights(to_dev(S, w.dtype), to_dev(Bm, w.dtype), torch.from_numpy(thetas).cuda())
    kw.update(weights=(S.astype(np.float64), Bm.astype(np.float64), list(thetas.astype(np.float64))))
    G = wl.round_to_storage(np.random.default_rng(G_SEED).standard_normal(inp["Q"].shape).astype(np.float32), w.dtype)
    got = ctx.backward(Q, K, V, to_dev(G, w.dtype))
    # the six tensor-core kernels and the mask export, plus the operand set-up on the first call
    assert binding.csat_last_launch_count(ctx.h) in (7, 8)
    words = ctx.backward_masks().cpu().numpy().astype(np.uint32)
    masks = np.stack([(words >> t) & 1 for t in range(T)], axis=2).astype(bool)
    stages = []
    ref = orc.csat_backward(inp["Q"], inp["K"], inp["V"], phi, G, masks=masks, stages=stages, **kw)
    own = np.stack([s["masks"] for s in stages]).reshape(masks.shape)
    assert (masks != own).mean() <= 2e-2
    for nm, g, rf in zip(("dQ", "dK", "dV"), got, ref):
        assert rel_err(to_np(g), rf) <= BWD_TOL[w.dtype], (T, with_psi, nm, rel_err(to_np(g), rf))
    ctx.close()


@pytest.mark.parametrize("name", ["bf16_d64", "bf16_d128"])
@pytest.mark.parametrize("weights", ["ista", "per_layer"])
def test_forward_that_saves_for_the_backward(name, weights):
    """CSAT_SAVE_FOR_BACKWARD: the forward's output still matches the oracle, the backward that follows skips its own
    compression and forward pass (two launches fewer) and returns the same bits as a backward that recomputes, a second
    backward still does, and a setter in between makes the backward recompute again."""
    w = CASES[name]()
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    kw = dict(T=w.T, lam=w.lam)
    if weights == "per_layer":
        r = np.random.default_rng(5)
        d, H, T = w.d, w.H, w.T
        S = wl.round_to_storage((0.6 * np.eye(d) + 0.4 * r.standard_normal((T, H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        Bm = wl.round_to_storage((r.standard_normal((T, H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        thetas = np.full((T, H), 0.02, dtype=np.float32)
        ctx.set_lista_layer_weights(to_dev(S, w.dtype), to_dev(Bm, w.dtype), torch.from_numpy(thetas).cuda())
        kw.update(weights=(S.astype(np.float64), Bm.astype(np.float64), list(thetas.astype(np.float64))))
    G = to_dev(wl.round_to_storage(np.random.default_rng(G_SEED).standard_normal(inp["Q"].shape).astype(np.float32), w.dtype), w.dtype)
    ctx.forward(Q, K, V)                                          # (sets up the decoder's operands)
    plain = ctx.backward(Q, K, V, G)
    n_plain = binding.csat_last_launch_count(ctx.h)
    binding.csat_set_i64(ctx.h, binding.CSAT_SAVE_FOR_BACKWARD, 1)
    out = to_np(ctx.forward(Q, K, V))
    ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], to_np(ctx.get_phi()), **kw)
    assert rel_err(out, ref) <= TOL[w.dtype]
    saved = ctx.backward(Q, K, V, G)
    assert binding.csat_last_launch_count(ctx.h) == n_plain - 2
    again = ctx.backward(Q, K, V, G)
    for a, b, c_ in zip(plain, saved, again):
        assert torch.equal(a, b) and torch.equal(a, c_)
    ctx.set(lam=w.lam)                                            # any setter drops what was saved
    recomputed = ctx.backward(Q, K, V, G)
    assert binding.csat_last_launch_count(ctx.h) >= n_plain
    for a, b in zip(plain, recomputed):
        assert torch.equal(a, b)
    if weights == "ista":
        # the decoder's gradients too: the saving forward then also keeps the iterates
        binding.csat_set_i64(ctx.h, binding.CSAT_WEIGHT_GRADS, 1)
        binding.csat_set_i64(ctx.h, binding.CSAT_SAVE_FOR_BACKWARD, 0)
        ctx.backward(Q, K, V, G)
        wg_plain = [x.clone() for x in ctx.weight_grads()]
        n_wg = binding.csat_last_launch_count(ctx.h)
        binding.csat_set_i64(ctx.h, binding.CSAT_SAVE_FOR_BACKWARD, 1)
        ctx.forward(Q, K, V)
        ctx.backward(Q, K, V, G)
        assert binding.csat_last_launch_count(ctx.h) == n_wg - 2          # no compression, no forward pass
        for a, b in zip(wg_plain, ctx.weight_grads()):
            assert torch.equal(a, b)
    ctx.close()


@pytest.mark.parametrize("name", ["bf16_d64", "bf16_d128"])
@pytest.mark.parametrize("with_psi", [False, True], ids=["identity", "dictionary"])
def test_per_layer_weight_gradients_match_oracle(name, with_psi):
    """CSAT_WEIGHT_GRADS with one S_t, B_t per layer: dS, dB [T,H,d,d] layer by layer (no sum over the layers), dtheta
    [T,H], dPsi, against the oracle's per-layer gradients summed over the batch, with the library's decisions."""
    w = WGRAD_CASES[name]()
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    binding.csat_set_i64(ctx.h, binding.CSAT_KEEP_MASKS, 1)
    binding.csat_set_i64(ctx.h, binding.CSAT_WEIGHT_GRADS, 1)
    d, H, T, B = w.d, w.H, w.T, w.B
    r = np.random.default_rng(23)
    kw = dict(T=T, lam=w.lam)
    if with_psi:
        Psi = wl.round_to_storage((np.eye(d) + 0.3 * r.standard_normal((d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        ctx.set_dictionary(to_dev(Psi, w.dtype))
        kw.update(Psi=Psi.astype(np.float64))
    S = wl.round_to_storage((0.6 * np.eye(d) + 0.4 * r.standard_normal((T, H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
    Bm = wl.round_to_storage((r.standard_normal((T, H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
    phi = to_np(ctx.get_phi())
    st0 = []
    orc.csat_forward(inp["Q"][:1], inp["K"][:1], inp["V"][:1], phi, T=0, lam=0.0, stages=st0)
    th0 = float(np.median(np.abs(st0[0]["Z"] @ Bm[0, 0].astype(np.float64))))
    thetas = (th0 * r.uniform(0.2, 1.5, size=(T, H))).astype(np.float32)
    ctx.set_lista_layer_weights(to_dev(S, w.dtype), to_dev(Bm, w.dtype), torch.from_numpy(thetas).cuda())
    kw.update(weights=(S.astype(np.float64), Bm.astype(np.float64), list(thetas.astype(np.float64))))
    G = wl.round_to_storage(np.random.default_rng(G_SEED).standard_normal(inp["Q"].shape).astype(np.float32), w.dtype)
    ctx.backward(Q, K, V, to_dev(G, w.dtype))
    words = ctx.backward_masks().cpu().numpy().astype(np.uint32)
    masks = np.stack([(words >> t) & 1 for t in range(T)], axis=2).astype(bool)
    stages = []
    orc.csat_backward(inp["Q"], inp["K"], inp["V"], phi, G, masks=masks, stages=stages, **kw)
    dS = np.zeros((T, H, d, d)); dB = np.zeros((T, H, d, d)); dth = np.zeros((T, H)); dPsi = np.zeros((d, d))
    for b in range(B):
        for h in range(H):
            st = stages[b * H + h]
            dS[:, h] += st["dS"]
            dB[:, h] += st["dB"]
            dth[:, h] += st["dtheta"]
            if with_psi:
                dPsi += st["dPsi"]
    gS, gB, gth, gPsi = (x.cpu().numpy().astype(np.float64) for x in ctx.weight_grads())
    assert gS.shape == (T, H, d, d) and gB.shape == (T, H, d, d)
    assert np.abs(gS[0]).max() == 0.0                          # alpha^0 = 0
    tol = BWD_TOL[w.dtype]
    for nm, g, rf in (("dS", gS, dS), ("dB", gB, dB), ("dtheta", gth, dth)) + ((("dPsi", gPsi, dPsi),) if with_psi else ()):
        assert np.isfinite(g).all() and np.abs(rf).max() > 0
        assert rel_err(g, rf) <= tol, (name, with_psi, nm, rel_err(g, rf))
    # every layer on its own scale too
    for t in range(1, T):
        assert rel_err(gS[t], dS[t]) <= 2 * tol and rel_err(gB[t], dB[t]) <= 2 * tol, t
    ctx.close()


def test_saving_forward_without_recovery_layers():
    """CSAT_SAVE_FOR_BACKWARD at T = 0 (the output is Z itself: nothing but Z and the softmax statistics to keep)."""
    w = wl.shrink(C["c2"], B=2, H=2, n_q=150, T=0)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    G = to_dev(wl.round_to_storage(np.random.default_rng(G_SEED).standard_normal(inp["Q"].shape).astype(np.float32), w.dtype), w.dtype)
    plain = ctx.backward(Q, K, V, G)
    binding.csat_set_i64(ctx.h, binding.CSAT_SAVE_FOR_BACKWARD, 1)
    out = ctx.forward(Q, K, V)
    ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], to_np(ctx.get_phi()), T=0, lam=w.lam)
    assert rel_err(to_np(out), ref) <= TOL[w.dtype]
    saved = ctx.backward(Q, K, V, G)
    for a, b in zip(plain, saved):
        assert torch.equal(a, b)
    ctx.close()
