"""GPU parity: libcsat (through its C-ABI binding) against the float64 CPU oracle, element by element,
on the same seeded inputs and the library's exported Phi.

Bar: max|gpu - oracle| / max|oracle| <= 2e-2 for bf16 storage with fp32 accumulation, <= 1e-4 for the
fp32 path.  Several workloads give an all-zero output at their own (T, lambda) (everything is shrunk
away), so every case is also checked with recovery disabled (T = 0, out = Z), at lambda = 0 and at a
lambda that keeps about half of the coefficients.
"""
import numpy as np
import pytest
import torch

from oracle import csat_oracle as orc
from oracle import phi_oracle as pho
from paper_2507_02957_b200 import binding, workloads as wl
from gpu_util import TOL, device_inputs, make_ctx, rel_err, to_dev, to_np

pytestmark = pytest.mark.gpu

C = wl.CONFIGS

SMALL_CASES = {
    "c1_full_fp32": C["c1"],
    "c1_as_bf16": wl.shrink(C["c1"], dtype="bf16"),
    "c2_vit_B2_H3": wl.shrink(C["c2"], B=2, H=3),
    "c3_video_B1_H2": wl.shrink(C["c3"], B=1, H=2),
    "c3_video_B3_H1_odd_batch": wl.shrink(C["c3"], B=3, H=1, n=392, n_q=200, m=200),
    "c4_cross_B2_H2": wl.shrink(C["c4"], B=2, H=2),
    "c5_long_n2048_nq700": wl.shrink(C["c5"], B=1, H=2, n=2048, n_q=700, m=128),
    "c5_long_n4096_m256": wl.shrink(C["c5"], B=1, H=1, n=4096, n_q=1000, m=256),
    "ragged_fp32_d72": wl.Workload("ragged", 2, 2, 203, 37, 72, 75, "fp32", 5, 0.02, "iid", 77),
    "ragged_bf16_d40": wl.Workload("ragged16", 1, 3, 131, 67, 40, 41, "bf16", 4, 0.02, "iid", 78),
}


def oracle_all(w, inp, phi, T, lam, stages=None):
    return orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=T, lam=lam, Psi=inp["Psi"], stages=stages)


def median_lambda(w, inp, phi):
    """lambda that shrinks about half of the first-iteration coefficients (from the oracle only)."""
    st = []
    orc.csat_forward(inp["Q"][:1, :1], inp["K"][:1, :1], inp["V"][:1, :1], phi[:1], T=1, lam=0.0,
                     Psi=inp["Psi"], stages=st)
    s = st[0]
    return float(np.median(np.abs(s["Z"] @ s["B_dec"])) / s["mu"])


@pytest.mark.parametrize("name", sorted(SMALL_CASES))
def test_forward_matches_oracle(name):
    w = SMALL_CASES[name]
    inp = wl.make_inputs(w)
    Q, K, V, Psi = device_inputs(w, inp)
    ctx = make_ctx(w)
    if Psi is not None:
        ctx.set_dictionary(Psi)
    phi = to_np(ctx.get_phi())
    tol = TOL[w.dtype]
    lam_med = median_lambda(w, inp, phi)
    for T, lam in [(0, w.lam), (w.T, w.lam), (w.T, 0.0), (w.T, lam_med), (1, lam_med)]:
        ctx.set(T=T, lam=lam)
        out = to_np(ctx.forward(Q, K, V))
        stages = []
        ref = oracle_all(w, inp, phi, T, lam, stages)
        if np.abs(ref).max() == 0.0:
            theta = max(s["theta"] for s in stages)
            assert np.abs(out).max() <= theta * tol, (name, T, lam)
        else:
            err = rel_err(out, ref)
            assert err <= tol, (name, T, lam, err)
        assert ctx.launches >= 2
    # compression stage on its own: K~, V~ as left in the workspace
    kt, vt = (to_np(t) for t in ctx.get_compressed())
    kt_ref = np.stack([[s["Kt"]] for s in stages]).reshape(kt.shape)
    vt_ref = np.stack([[s["Vt"]] for s in stages]).reshape(vt.shape)
    assert rel_err(kt, kt_ref) <= (4e-3 if w.dtype == "bf16" else 2e-6)
    assert rel_err(vt, vt_ref) <= (4e-3 if w.dtype == "bf16" else 2e-6)
    ctx.close()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_identity_measurement_is_softmax_attention(dtype):
    """m = n, Phi = I: recovery disabled gives standard attention; T >= 1 gives soft(Attn, lambda)."""
    w = wl.shrink(C["c1"], m=256, dtype=dtype)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w, T=0)
    ctx.set_phi(to_dev(np.eye(w.n, dtype=np.float32)[None], dtype))
    Qd, Kd, Vd = (inp[k][0, 0].astype(np.float64) for k in "QKV")
    A = np.exp(Qd @ Kd.T / 8.0 - (Qd @ Kd.T / 8.0).max(axis=1, keepdims=True))
    attn = (A / A.sum(axis=1, keepdims=True)) @ Vd
    out = to_np(ctx.forward(Q, K, V))[0, 0]
    assert rel_err(out, attn) <= TOL[dtype]
    ctx.set(T=3, lam=0.1)
    out = to_np(ctx.forward(Q, K, V))[0, 0]
    shr = np.sign(attn) * np.maximum(np.abs(attn) - 0.1, 0.0)
    assert rel_err(out, shr) <= TOL[dtype]
    ctx.close()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_phi_matches_oracle_generator(dtype):
    for (H, m, n, seed) in [(1, 64, 256, 0), (3, 20, 197, 0xDEADBEEF12345678), (2, 7, 64, 5)]:
        ctx = binding.Csat(n, m, 8, H, seed, dtype=dtype)
        got = to_np(ctx.get_phi())
        exact = pho.phi_gaussian(H, m, n, seed)
        ref = wl.round_to_storage(exact.astype(np.float32), dtype).astype(np.float64)
        if dtype == "fp32":
            # float32 transcendentals vs float64: a few ulp, plus cancellation near sin/cos zeros
            assert np.all(np.abs(got - exact) <= 4e-6 * np.abs(exact) + 2e-7 / np.sqrt(m))
        else:
            bad = got != ref
            assert bad.mean() <= 1e-3
            assert np.all(np.abs(got - ref)[bad] <= np.abs(ref[bad]) * 2.0 ** -7)   # one bf16 ulp
        ctx.close()


def test_decoder_matrices_match_oracle():
    w = wl.shrink(C["c4"], B=1, H=3, n=392, m=98)
    inp = wl.make_inputs(w)
    ctx = make_ctx(w)
    Psi = to_dev(inp["Psi"], w.dtype)
    phi = to_np(ctx.get_phi())
    for psi_dev, psi_np in ((None, None), (Psi, inp["Psi"].astype(np.float64))):
        ctx.set_dictionary(psi_dev)
        for step in (0.0, 0.3):
            ctx.set(step=step)
            S, Bm, th, mu = (to_np(t) for t in ctx.get_decoder())
            for h in range(w.H):
                D = phi[h, :w.d, :w.d]
                M = D if psi_np is None else D @ psi_np
                S_ref, B_ref, th_ref, mu_ref = orc.decoder_setup(M, w.lam, step)
                assert np.abs(S[h] - S_ref).max() <= 1e-6
                assert np.abs(Bm[h] - B_ref).max() <= 1e-6 * max(1.0, np.abs(B_ref).max())
                assert abs(th[h] - th_ref) <= 1e-6 * th_ref and abs(mu[h] - mu_ref) <= 1e-6 * mu_ref
    # a caller-supplied decoder matrix replaces the Phi block
    r = np.random.default_rng(3)
    Dn = wl.round_to_storage((np.eye(w.d) + 0.1 * r.standard_normal((w.H, w.d, w.d))).astype(np.float32), w.dtype)
    ctx.set_dictionary(None)
    ctx.set(step=0.0)
    ctx.set_decoder_matrix(to_dev(Dn, w.dtype))
    S, Bm, th, mu = (to_np(t) for t in ctx.get_decoder())
    for h in range(w.H):
        S_ref, B_ref, _, _ = orc.decoder_setup(Dn[h].astype(np.float64), w.lam)
        assert np.abs(S[h] - S_ref).max() <= 1e-6 and np.abs(Bm[h] - B_ref).max() <= 1e-6
    Q, K, V, _ = device_inputs(w, inp)
    out = to_np(ctx.forward(Q, K, V))
    ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=w.T, lam=w.lam, D=Dn.astype(np.float64))
    assert rel_err(out, ref) <= TOL[w.dtype]
    ctx.close()


def test_edge_shapes():
    """Single query, single measurement (needs a supplied D), tiny ragged sizes, huge lambda."""
    r = np.random.default_rng(11)
    for dtype in ("fp32", "bf16"):
        for (B, H, n, nq, d, m) in [(1, 1, 8, 1, 8, 1), (2, 1, 9, 3, 8, 9), (1, 2, 300, 5, 16, 2), (1, 1, 64, 129, 64, 64)]:
            w = wl.Workload("edge", B, H, n, nq, d, m, dtype, 3, 0.01, "iid", 5)
            inp = wl.make_inputs(w)
            Q, K, V, _ = device_inputs(w, inp)
            ctx = make_ctx(w)
            Dn = wl.round_to_storage((np.eye(d) + 0.2 * r.standard_normal((H, d, d))).astype(np.float32), dtype)
            ctx.set_decoder_matrix(to_dev(Dn, dtype))
            phi = to_np(ctx.get_phi())
            for T, lam in [(0, 0.0), (3, 0.01), (2, 1e6)]:
                ctx.set(T=T, lam=lam)
                out = to_np(ctx.forward(Q, K, V))
                ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=T, lam=lam, D=Dn.astype(np.float64))
                if lam == 1e6:
                    assert np.all(out == 0.0) and np.all(ref == 0.0)
                else:
                    assert rel_err(out, ref) <= TOL[dtype], (dtype, B, H, n, nq, d, m, T)
            ctx.close()


def test_abi_errors_and_determinism():
    w = wl.shrink(C["c2"], B=1, H=2)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w, lam=0.0)
    out1 = ctx.forward(Q, K, V).clone()
    out2 = ctx.forward(Q, K, V)
    assert torch.equal(out1, out2)                                    # bit-identical run to run
    lib = binding.load()
    s = torch.cuda.current_stream().cuda_stream
    p = lambda t: t.data_ptr()
    assert lib.csat_forward(ctx.h, None, p(K), p(V), p(out2), s) == 1
    assert lib.csat_forward(ctx.h, p(Q) + 2, p(K), p(V), p(out2), s) == 1     # misaligned
    assert lib.csat_forward(ctx.h, p(Q), p(K), p(V), p(Q), s) == 1            # out aliases Q
    assert "overlap" in binding.csat_last_error(ctx.h)
    big = torch.empty(2 * Q.numel(), dtype=Q.dtype, device="cuda")
    big[: Q.numel()].copy_(Q.reshape(-1))
    shifted = big[64: 64 + Q.numel()]                                         # 128 bytes into the copy of Q
    assert lib.csat_forward(ctx.h, p(big), p(K), p(V), p(shifted), s) == 1    # out overlaps Q without equal pointers
    assert "overlap" in binding.csat_last_error(ctx.h)
    assert lib.csat_set_i64(ctx.h, 99, 1) == 1
    assert lib.csat_set_i64(ctx.h, binding.CSAT_T, -1) == 1
    assert lib.csat_set_f64(ctx.h, binding.CSAT_LAMBDA, -0.5) == 1
    assert lib.csat_set_i64(ctx.h, binding.CSAT_BATCH, 0) == 2
    assert binding.csat_get_i64(ctx.h, binding.CSAT_T) == w.T
    assert binding.csat_get_f64(ctx.h, binding.CSAT_LAMBDA) == 0.0
    assert ctx.workspace_bytes > 0
    torch.cuda.synchronize()
    assert torch.equal(ctx.forward(Q, K, V), out1)                    # failed calls left the context usable
    ctx.close()
    # default decoder matrix needs m >= d
    small = binding.Csat(64, 8, 64, 1, 0, dtype="fp32", T=2)
    q = torch.zeros(1, 1, 64, 64, device="cuda")
    with pytest.raises(binding.CsatError) as ei:
        small.forward(q, q.clone(), q.clone())
    assert ei.value.code == 2
    small.set(T=0)
    small.forward(q, q.clone(), q.clone())                            # recovery disabled: legal
    small.close()
    with pytest.raises(binding.CsatError):
        c = binding.Csat(64, 8, 64, 1, 0)
        try:
            binding.csat_get_compressed(c.h, q, q)                    # before any forward
        finally:
            c.close()


def test_forward_host_equals_forward():
    w = wl.shrink(C["c3"], B=1, H=2, n=392, n_q=392, m=64)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    out = ctx.forward(Q, K, V)
    Qh, Kh, Vh = (t.cpu().pin_memory() for t in (Q, K, V))
    oh = torch.empty_like(Qh).pin_memory()
    ctx.forward_host(Qh, Kh, Vh, oh)
    assert torch.equal(oh, out.cpu())
    ctx.close()


@pytest.mark.parametrize("name", ["c1_full_fp32", "c3_video_B1_H2", "c5_long_n2048_nq700", "ragged_bf16_d40"])
def test_supplied_lista_weights_match_oracle(name):
    """Caller-supplied S, B (non-symmetric, random) with one threshold for all layers and with per-layer
    thresholds; then ISTA's own weights supplied through the same call reproduce the default decoder."""
    w = SMALL_CASES[name]
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    phi = to_np(ctx.get_phi())
    r = np.random.default_rng(31)
    d, H, T = w.d, w.H, w.T
    S = wl.round_to_storage((0.6 * np.eye(d) + 0.4 * r.standard_normal((H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
    Bm = wl.round_to_storage((r.standard_normal((H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
    st = []
    orc.csat_forward(inp["Q"][:1], inp["K"][:1], inp["V"][:1], phi, T=0, lam=0.0, stages=st)
    th0 = float(np.median(np.abs(st[0]["Z"] @ Bm[0].astype(np.float64))))           # about half survive layer 0
    tied = np.full((1, H), th0, dtype=np.float32)
    per_layer = (th0 * r.uniform(0.2, 1.5, size=(T, H))).astype(np.float32)
    for thetas in (tied, per_layer):
        ctx.set_lista_weights(to_dev(S, w.dtype), to_dev(Bm, w.dtype), torch.from_numpy(thetas).cuda())
        out = to_np(ctx.forward(Q, K, V))
        th_list = [thetas[t if thetas.shape[0] > 1 else 0].astype(np.float64) for t in range(T)]
        ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=T, lam=0.0,
                               weights=(S.astype(np.float64), Bm.astype(np.float64), th_list))
        assert np.abs(ref).max() > 0
        err = rel_err(out, ref)
        assert err <= TOL[w.dtype], (name, thetas.shape, err)
    # wrong number of layers is refused, and the context stays usable
    ctx.set_lista_weights(to_dev(S, w.dtype), to_dev(Bm, w.dtype), torch.from_numpy(per_layer[:-1].copy()).cuda())
    if T > 2:
        with pytest.raises(binding.CsatError) as ei:
            ctx.forward(Q, K, V)
        assert ei.value.code == 6
    # back to the derived decoder; ISTA's weights supplied by hand give the same output as the default path
    ctx.set_lista_weights(None)
    ctx.set(lam=th0)
    base = to_np(ctx.forward(Q, K, V))
    S_d, B_d, th_d, _ = ctx.get_decoder()
    if w.dtype == "fp32":
        ctx.set_lista_weights(S_d, B_d, th_d)
        again = to_np(ctx.forward(Q, K, V))
        assert rel_err(again, base) <= 1e-5
    ctx.close()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_rademacher_ensemble_is_bit_exact_and_runs(dtype):
    """Integer work: the library's Rademacher Phi equals the oracle's bit for bit; a forward with it matches
    the oracle; switching back restores the Gaussian matrix."""
    for (H, m, n, seed) in [(1, 64, 256, 0), (3, 20, 197, 0xDEADBEEF12345678), (2, 7, 4099, 5), (2, 9, 4104, 6), (5, 33, 1568, 1)]:
        ctx = binding.Csat(n, m, 8, H, seed, dtype=dtype)
        gauss = ctx.get_phi().clone()
        ctx.set(ensemble="rademacher")
        got = to_np(ctx.get_phi())
        ref = wl.round_to_storage(pho.phi_rademacher(H, m, n, seed).astype(np.float32), dtype).astype(np.float64)
        assert np.array_equal(got, ref)
        ctx.set(ensemble="gaussian")
        assert torch.equal(ctx.get_phi(), gauss)
        ctx.close()
    w = wl.shrink(C["c3"], B=1, H=2, n=784, n_q=300, m=128) if dtype == "bf16" else C["c1"]
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    ctx.set(ensemble="rademacher")
    phi = to_np(ctx.get_phi())
    assert np.array_equal(np.abs(phi), np.full_like(phi, np.abs(phi[0, 0, 0])))
    for T, lam in [(0, 0.0), (w.T, w.lam)]:
        ctx.set(T=T, lam=lam)
        out = to_np(ctx.forward(Q, K, V))
        ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=T, lam=lam)
        assert rel_err(out, ref) <= TOL[dtype], (dtype, T)
    ctx.close()


def test_bounded_wait_reports_a_timeout_and_the_context_recovers():
    """A wait that can never complete (nothing arrives at its barrier) gives up after its limit, the status
    word turns every later forward into CSAT_ERR_TIMEOUT, and clearing it restores the context."""
    w = wl.shrink(C["c2"], B=1, H=2)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w, lam=0.0)
    good = ctx.forward(Q, K, V).clone()
    assert binding.csat_selftest_wait_timeout(ctx.h, 1000) == 7          # 1 ms limit
    assert "gave up" in binding.csat_last_error(ctx.h)
    with pytest.raises(binding.CsatError) as ei:
        ctx.forward(Q, K, V)
    assert ei.value.code == 7
    assert binding.csat_clear_status(ctx.h) == 999                        # the self-test's code
    assert binding.csat_clear_status(ctx.h) == 0
    assert torch.equal(ctx.forward(Q, K, V), good)
    ctx.close()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_hadamard_ensemble_is_bit_exact_and_runs(dtype):
    for (H, m, n, seed) in [(1, 64, 256, 0), (3, 20, 197, 0xDEADBEEF12345678), (2, 9, 4104, 6), (4, 33, 1568, 1)]:
        ctx = binding.Csat(n, m, 8, H, seed, dtype=dtype)
        ctx.set(ensemble="hadamard")
        got = to_np(ctx.get_phi())
        ref = wl.round_to_storage(pho.phi_hadamard(H, m, n, seed).astype(np.float32), dtype).astype(np.float64)
        assert np.array_equal(got, ref), (H, m, n)
        ctx.close()
    w = wl.shrink(C["c3"], B=1, H=2, n=784, n_q=300, m=128) if dtype == "bf16" else C["c1"]
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    ctx.set(ensemble="hadamard")
    phi = to_np(ctx.get_phi())
    for T, lam in [(0, 0.0), (w.T, w.lam)]:
        ctx.set(T=T, lam=lam)
        out = to_np(ctx.forward(Q, K, V))
        ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=T, lam=lam)
        assert rel_err(out, ref) <= TOL[dtype], (dtype, T)
    ctx.close()


@pytest.mark.parametrize("name", ["c1_full_fp32", "c3_video_B1_H2", "c5_long_n2048_nq700", "c4_cross_B2_H2", "ragged_bf16_d40"])
def test_separate_key_and_value_matrices(name):
    """CSAT_SEPARATE_PHI: K~ = Phi_K K, V~ = Phi_V V with Phi_V drawn as heads H .. 2H-1 of the same generator;
    the decoder's default matrix is the block of Phi_V."""
    w = SMALL_CASES[name]
    inp = wl.make_inputs(w)
    Q, K, V, Psi = device_inputs(w, inp)
    ctx = make_ctx(w)
    if Psi is not None:
        ctx.set_dictionary(Psi)
    shared = ctx.get_phi().clone()
    ctx.set(separate_phi=True)
    both = ctx.get_phi()
    assert both.shape[0] == 2 * w.H and torch.equal(both[:w.H], shared)       # Phi_K is the shared matrix
    assert not torch.equal(both[w.H:], both[:w.H])
    phi = to_np(both)
    for T, lam in [(0, w.lam), (w.T, w.lam), (w.T, 0.0)]:
        ctx.set(T=T, lam=lam)
        out = to_np(ctx.forward(Q, K, V))
        stages = []
        ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi[:w.H], T=T, lam=lam, Psi=inp["Psi"],
                               Phi_V=phi[w.H:], stages=stages)
        if np.abs(ref).max() == 0.0:
            assert np.abs(out).max() <= max(s["theta"] for s in stages) * TOL[w.dtype]
        else:
            assert rel_err(out, ref) <= TOL[w.dtype], (name, T, lam)
    kt, vt = (to_np(t) for t in ctx.get_compressed())
    vt_ref = np.stack([[s["Vt"]] for s in stages]).reshape(vt.shape)
    assert rel_err(vt, vt_ref) <= (4e-3 if w.dtype == "bf16" else 2e-6)
    # Rademacher: both halves bit-exact against the oracle's 2H-head generator
    ctx.set(ensemble="rademacher")
    ref = wl.round_to_storage(pho.phi_rademacher(2 * w.H, w.m, w.n, w.phi_seed).astype(np.float32), w.dtype)
    assert np.array_equal(to_np(ctx.get_phi()), ref.astype(np.float64))
    # back to one matrix per head
    ctx.set(ensemble="gaussian")
    ctx.set(separate_phi=False)
    assert torch.equal(ctx.get_phi(), shared)
    ctx.close()


def test_tensor_core_edge_shapes():
    """Shapes that stress the tcgen05 kernels' tails: partial query tiles and measurement chunks at d = 128,
    a single query, fewer measurements than one chunk, a dictionary with one iteration, many iterations."""
    r = np.random.default_rng(17)
    cases = [  # B, H, n, n_q, d, m, T, with_psi
        (3, 2, 200, 130, 128, 136, 3, False),
        (1, 1, 128, 1, 128, 128, 2, True),
        (2, 1, 300, 257, 128, 9, 1, True),
        (1, 2, 90, 40, 64, 1, 4, False),
        (2, 3, 520, 513, 64, 200, 1, True),
        (1, 1, 256, 100, 128, 192, 60, False),
    ]
    for (B, H, n, nq, d, m, T, with_psi) in cases:
        w = wl.Workload("tc_edge", B, H, n, nq, d, m, "bf16", T, 0.02, "iid", 5)
        inp = wl.make_inputs(w)
        Q, K, V, _ = device_inputs(w, inp)
        ctx = make_ctx(w)
        Dn = wl.round_to_storage((np.eye(d) + 0.1 * r.standard_normal((H, d, d))).astype(np.float32), "bf16")
        ctx.set_decoder_matrix(to_dev(Dn, "bf16"))           # m may be smaller than d
        psi = None
        if with_psi:
            psi = wl.orthonormal_basis(d, 99 + d)
            psi = wl.round_to_storage(psi, "bf16")
            ctx.set_dictionary(to_dev(psi, "bf16"))
        phi = to_np(ctx.get_phi())
        for T_run, lam in [(0, 0.0), (T, 0.02), (T, 0.0)]:
            ctx.set(T=T_run, lam=lam)
            out = ctx.forward(Q, K, V)
            assert torch.isfinite(out).all()
            ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=T_run, lam=lam, D=Dn.astype(np.float64),
                                   Psi=None if psi is None else psi.astype(np.float64))
            assert np.abs(ref).max() > 0
            err = rel_err(to_np(out), ref)
            assert err <= TOL["bf16"], (B, H, n, nq, d, m, T_run, lam, err)
        ctx.close()


def test_values_with_b_folded_in_edge_shapes():
    """Jobs long enough for the library to form V~ B first (at least 8 query tiles per SM at d = 64, 2 at d = 128): ragged measurement counts,
    a dictionary, separate Phi_K / Phi_V, both head sizes, a ragged last query tile; sampled (batch, head) pairs against
    the oracle, and the exported V~ is still Phi V (V~ B lives beside it)."""
    cases = [  # B, H, n, n_q, d, m, T, with_psi, separate
        (2, 5, 600, 15400, 64, 200, 3, True, False),
        (1, 10, 512, 15900, 128, 136, 2, False, True),
        (1, 10, 384, 16000, 128, 129, 5, False, False),
    ]
    for (B, H, n, nq, d, m, T, with_psi, separate) in cases:
        w = wl.Workload("folded_edge", B, H, n, nq, d, m, "bf16", T, 0.004, "iid", 9)
        inp = wl.make_inputs(w)
        Q, K, V, _ = device_inputs(w, inp)
        ctx = make_ctx(w)
        psi = None
        if with_psi:
            psi = wl.round_to_storage(wl.orthonormal_basis(d, 7 + d), "bf16")
            ctx.set_dictionary(to_dev(psi, "bf16"))
        if separate:
            ctx.set(separate_phi=True)
        phi = to_np(ctx.get_phi())
        out = ctx.forward(Q, K, V)
        assert ctx.launches >= 3 and torch.isfinite(out).all()
        assert torch.equal(out, ctx.forward(Q, K, V))
        kt, vt = (to_np(t) for t in ctx.get_compressed())
        for (b, h) in [(0, 0), (B - 1, H - 1)]:
            st = {}
            ref = orc.csat_forward_head(inp["Q"][b, h], inp["K"][b, h], inp["V"][b, h], phi[h], T=T, lam=w.lam,
                                        Psi=None if psi is None else psi.astype(np.float64),
                                        Phi_v_h=phi[H + h] if separate else None, stages=st)
            assert np.abs(ref).max() > 0
            assert rel_err(to_np(out[b, h]), ref) <= TOL["bf16"], (B, H, n, nq, d, m, T, b, h)
            assert rel_err(vt[b, h], st["Vt"]) <= 4e-3
        ctx.close()


@pytest.mark.parametrize("d", [64, 128])
def test_pipelined_host_forward_is_bit_identical(d):
    """csat_forward_host cuts the job into chunks of heads of one batch element (here 2 + 2 + 1 heads per batch
    element) on its own streams; the result must equal csat_forward on device buffers bit for bit, twice in a row,
    and with a caller stream other than the default one."""
    w = wl.Workload("host_pipe", 2, 5, 448, 300, d, 128, "bf16", 3, 0.01, "iid", 41)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    ref = ctx.forward(Q, K, V).cpu()
    Qh, Kh, Vh = (t.cpu().pin_memory() for t in (Q, K, V))
    for rep in range(2):
        oh = torch.full_like(Qh, float("nan")).pin_memory()
        ctx.forward_host(Qh, Kh, Vh, oh)
        assert torch.equal(oh, ref), rep
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        oh = torch.full_like(Qh, float("nan")).pin_memory()
        ctx.forward_host(Qh, Kh, Vh, oh)
    assert torch.equal(oh, ref)
    ctx.set(T=0)
    ref0 = ctx.forward(Q, K, V).cpu()
    oh = torch.empty_like(Qh).pin_memory()
    ctx.forward_host(Qh, Kh, Vh, oh)
    assert torch.equal(oh, ref0)
    ctx.close()


def test_forward_can_be_captured_in_a_cuda_graph():
    """csat_forward only enqueues work (no allocation, no synchronisation), so a stream capture records it; replays
    with new input values in the same buffers give the same output as eager calls."""
    w = wl.shrink(C["c2"], B=2, H=3)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w, lam=0.0)
    out = torch.empty_like(Q)
    ctx.forward(Q, K, V, out)                     # first call: derives the decoder matrices outside the capture
    torch.cuda.synchronize()
    eager1 = out.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx.forward(Q, K, V, out)
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager1)
    Q.copy_(torch.flip(Q, dims=[2]))              # new values, same buffers
    graph.replay()
    torch.cuda.synchronize()
    replayed = out.clone()
    assert torch.equal(ctx.forward(Q, K, V), replayed)
    assert not torch.equal(replayed, eager1)
    ctx.close()


@pytest.mark.parametrize("name", ["c1_fp32", "c2_bf16_d64", "c5_bf16_d128", "c3_bf16_psi"])
def test_untied_lista_layers_match_oracle(name):
    """One S_t, B_t and theta_t per layer (random, non-symmetric): FFMA path in fp32, per-layer tensor-core kernel
    in bf16 (head dimension 64 and 128, ragged query tiles, with and without a dictionary)."""
    if name == "c1_fp32":
        w = C["c1"]
    elif name == "c2_bf16_d64":
        w = wl.shrink(C["c2"], B=2, H=3, n_q=300)
    elif name == "c5_bf16_d128":
        w = wl.shrink(C["c5"], B=1, H=2, n=1024, n_q=700, m=192)
    else:
        w = wl.shrink(C["c3"], B=2, H=2, n=784, n_q=257, m=100)
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    phi = to_np(ctx.get_phi())
    r = np.random.default_rng(41)
    d, H = w.d, w.H
    Psi = None
    if name == "c3_bf16_psi":
        Psi = wl.round_to_storage((np.eye(d) + 0.3 * r.standard_normal((d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        ctx.set_dictionary(to_dev(Psi, w.dtype))
    st = []
    orc.csat_forward(inp["Q"][:1], inp["K"][:1], inp["V"][:1], phi, T=0, lam=0.0, stages=st)
    for T in sorted({1, 2, w.T}):
        ctx.set(T=T)
        S = wl.round_to_storage((0.6 * np.eye(d) + 0.4 * r.standard_normal((T, H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        Bm = wl.round_to_storage((r.standard_normal((T, H, d, d)) / np.sqrt(d)).astype(np.float32), w.dtype)
        th0 = float(np.median(np.abs(st[0]["Z"] @ Bm[0, 0].astype(np.float64))))
        thetas = (th0 * r.uniform(0.2, 1.5, size=(T, H))).astype(np.float32)
        thetas[T // 2, 0] = 0.0                                    # a layer without shrinkage
        ctx.set_lista_layer_weights(to_dev(S, w.dtype), to_dev(Bm, w.dtype), torch.from_numpy(thetas).cuda())
        out = to_np(ctx.forward(Q, K, V))
        ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=T, lam=0.0, Psi=None if Psi is None else Psi.astype(np.float64),
                               weights=(S.astype(np.float64), Bm.astype(np.float64), list(thetas.astype(np.float64))))
        assert np.abs(ref).max() > 0
        err = rel_err(out, ref)
        assert err <= TOL[w.dtype], (name, T, err)
        if w.dtype == "bf16":
            # the FFMA path reads the same per-layer weights
            ctx.set(force_simt=1)
            err = rel_err(to_np(ctx.forward(Q, K, V)), ref)
            ctx.set(force_simt=0)
            assert err <= TOL[w.dtype], (name, T, "ffma", err)
    # csat_get_decoder returns layer 0
    S_d, B_d, th_d, _ = ctx.get_decoder()
    assert np.array_equal(to_np(S_d), S[0].astype(np.float64)) and np.array_equal(to_np(B_d), Bm[0].astype(np.float64))
    assert np.array_equal(to_np(th_d), thetas[0].astype(np.float64))
    # another depth than the weights' is refused; tied weights and the derived decoder come back afterwards
    ctx.set(T=T + 1)
    with pytest.raises(binding.CsatError) as ei:
        ctx.forward(Q, K, V)
    assert ei.value.code == 6
    ctx.set(T=T)
    tied_th = torch.from_numpy(thetas[:1].copy()).cuda()
    ctx.set_lista_weights(to_dev(S[0], w.dtype), to_dev(Bm[0], w.dtype), tied_th)
    tied = to_np(ctx.forward(Q, K, V))
    same = np.stack([S[0]] * T), np.stack([Bm[0]] * T), np.repeat(thetas[:1], T, axis=0)
    ctx.set_lista_layer_weights(to_dev(same[0], w.dtype), to_dev(same[1], w.dtype), torch.from_numpy(same[2].copy()).cuda())
    again = to_np(ctx.forward(Q, K, V))
    assert rel_err(again, tied) <= TOL[w.dtype]
    ctx.set_lista_weights(None)
    ctx.set(lam=w.lam)
    ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=T, lam=w.lam, Psi=None if Psi is None else Psi.astype(np.float64))
    assert rel_err(to_np(ctx.forward(Q, K, V)), ref) <= TOL[w.dtype]
    ctx.close()


def test_output_aligned_to_16_bytes_only_gives_the_same_result():
    """The tensor-core kernel's output stores (TMA stores of whole boxes in the plain forward, 32 or 16 bytes per lane
    in the recording variants) need no more than 16-byte alignment: an output that starts 16 bytes into an
    allocation must come out bit-identical."""
    for w in (wl.shrink(C["c2"], B=2, H=3, n_q=300), wl.shrink(C["c5"], B=1, H=2, n=1024, n_q=700, m=192)):
        inp = wl.make_inputs(w)
        Q, K, V, _ = device_inputs(w, inp)
        ctx = make_ctx(w)
        ref = ctx.forward(Q, K, V)
        flat = torch.zeros(Q.numel() + 8, dtype=Q.dtype, device="cuda")
        out = flat[8:].view(Q.shape)
        assert out.data_ptr() % 32 == 16 and out.is_contiguous()
        ctx.forward(Q, K, V, out)
        torch.cuda.synchronize()
        assert torch.equal(out, ref)
        assert float(flat[:8].abs().max()) == 0.0
        ctx.close()


def test_output_stores_stay_inside_the_tensor():
    """Query counts that end inside a warp's 32 rows, a tile's 128 or an item's 256: the output boxes are clipped at
    n_q, so guard rows before and after the tensor keep their sentinel and every row of the tensor is written."""
    for d, nqs in ((128, (1, 33, 129, 255, 257)), (64, (31, 160, 385))):
        for nq in nqs:
            w = wl.shrink(C["c5"] if d == 128 else C["c2"], B=1, H=2, n=512, n_q=nq, m=192, T=2, lam=0.0)
            inp = wl.make_inputs(w)
            Q, K, V, _ = device_inputs(w, inp)
            ctx = make_ctx(w)
            guard = 256 * d
            flat = torch.full((Q.numel() + 2 * guard,), 7.0, dtype=Q.dtype, device="cuda")
            out = flat[guard:guard + Q.numel()].view(Q.shape)
            ctx.forward(Q, K, V, out)
            torch.cuda.synchronize()
            assert float((flat[:guard] - 7.0).abs().max()) == 0.0 and float((flat[guard + Q.numel():] - 7.0).abs().max()) == 0.0
            ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], to_np(ctx.get_phi()), T=w.T, lam=w.lam)
            assert np.abs(ref).max() > 0 and rel_err(to_np(out), ref) <= TOL["bf16"], (d, nq)
            ctx.close()


@pytest.mark.parametrize("case", ["bf16_d64_self", "bf16_d128_self", "bf16_d64_cross", "bf16_ragged_k", "fp32", "bf16_ffma"])
def test_project_qkv_matches_oracle(case):
    """Q = X W^Q, K = X W^K, V = X W^V for all heads, in the layout csat_forward reads: tensor-core kernel over
    several 128 x 256 tiles with ragged tokens, columns and reduction length; cross-attention (two launches);
    the FFMA kernel for float32 and for forced bf16."""
    r = np.random.default_rng(71)
    cfg = {
        "bf16_d64_self":  dict(dtype="bf16", B=2, H=3, d=64, n=197, n_q=197, dm=192),
        "bf16_d128_self": dict(dtype="bf16", B=1, H=3, d=128, n=300, n_q=300, dm=256),
        "bf16_d64_cross": dict(dtype="bf16", B=2, H=5, d=64, n=260, n_q=77, dm=128),
        "bf16_ragged_k":  dict(dtype="bf16", B=1, H=2, d=64, n=130, n_q=130, dm=72),
        "fp32":           dict(dtype="fp32", B=2, H=2, d=32, n=50, n_q=20, dm=40),
        "bf16_ffma":      dict(dtype="bf16", B=1, H=2, d=64, n=70, n_q=70, dm=64),
    }[case]
    dt, B, H, d, n, nq, dm = (cfg[k] for k in ("dtype", "B", "H", "d", "n", "n_q", "dm"))
    ctx = binding.Csat(n, 16, d, H, 3, B=B, n_q=nq, dtype=dt, T=0)
    if case == "bf16_ffma":
        ctx.set(force_simt=1)
    X = wl.round_to_storage(r.standard_normal((B, nq, dm)).astype(np.float32), dt)
    Xkv = X if nq == n else wl.round_to_storage(r.standard_normal((B, n, dm)).astype(np.float32), dt)
    W = wl.round_to_storage((r.standard_normal((dm, 3 * H * d)) / np.sqrt(dm)).astype(np.float32), dt)
    Xd, Wd = to_dev(X, dt), to_dev(W, dt)
    Xkvd = Xd if nq == n else to_dev(Xkv, dt)
    Q, K, V = ctx.project_qkv(Xd, Wd, None if nq == n else Xkvd)
    HD = H * d
    Qr = orc.project_qkv(X, W, H, d)[0]
    _, Kr, Vr = orc.project_qkv(Xkv, W, H, d)
    for name, got, ref in (("Q", Q, Qr), ("K", K, Kr), ("V", V, Vr)):
        err = rel_err(to_np(got), ref)
        assert err <= (1e-5 if dt == "fp32" else 8e-3), (case, name, err)     # bf16: output rounding, 2^-8 of max
    assert binding.csat_last_launch_count(ctx.h) == (1 if nq == n else 2)
    # the projected tensors feed the forward as they are
    out = to_np(ctx.forward(Q, K, V))
    ref = orc.csat_forward(to_np(Q), to_np(K), to_np(V), to_np(ctx.get_phi()), T=0, lam=0.0)
    assert rel_err(out, ref) <= TOL[dt]
    ctx.close()


FWHT_CASES = {
    "bf16_d64_n4096_m1024": wl.Workload("fwht_a", 2, 2, 4096, 300, 64, 1024, "bf16", 3, 0.01, "iid", 71),
    "bf16_d64_ragged_n197": wl.Workload("fwht_b", 2, 3, 197, 197, 64, 64, "bf16", 3, 0.01, "iid", 72),
    "fp32_d72_n1000": wl.Workload("fwht_c", 1, 2, 1000, 100, 72, 250, "fp32", 2, 0.01, "iid", 73),
    "bf16_d128_n5000": wl.Workload("fwht_d", 1, 2, 5000, 200, 128, 320, "bf16", 2, 0.01, "iid", 74),
    "bf16_d64_n16384": wl.Workload("fwht_e", 1, 1, 16384, 256, 64, 1024, "bf16", 0, 0.0, "iid", 75),
}


@pytest.mark.parametrize("name", sorted(FWHT_CASES))
@pytest.mark.parametrize("separate", [False, True])
def test_hadamard_fast_transform_matches_oracle_and_dense_product(name, separate):
    """CSAT_HADAMARD_TRANSFORM: K~, V~ by a fast Walsh-Hadamard transform and a gather of the selected rows.  The
    reference is the oracle's compression with the dense matrix the library exports for the same ensemble; the dense
    tensor-core / FFMA product of the same context must agree as well, and so must the whole forward."""
    w = FWHT_CASES[name]
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    ctx.set(ensemble="hadamard")
    if separate:
        ctx.set(separate_phi=True)
    phi = to_np(ctx.get_phi())
    phi_k, phi_v = phi[:w.H], (phi[w.H:] if separate else phi[:w.H])
    dense_out = ctx.forward(Q, K, V).clone()
    kt_d, vt_d = (to_np(t) for t in ctx.get_compressed())
    ctx.set(hadamard_transform=True)
    assert binding.csat_get_i64(ctx.h, binding.CSAT_HADAMARD_TRANSFORM) == 1
    fast_out = ctx.forward(Q, K, V)
    kt_f, vt_f = (to_np(t) for t in ctx.get_compressed())
    kt_ref = np.stack([[orc.compress(phi_k[h], inp["K"][b, h]) for h in range(w.H)] for b in range(w.B)])
    vt_ref = np.stack([[orc.compress(phi_v[h], inp["V"][b, h]) for h in range(w.H)] for b in range(w.B)])
    tol_kv = 4e-3 if w.dtype == "bf16" else 2e-6
    assert rel_err(kt_f, kt_ref) <= tol_kv and rel_err(vt_f, vt_ref) <= tol_kv, name
    assert rel_err(kt_f, kt_d) <= 2 * tol_kv and rel_err(vt_f, vt_d) <= 2 * tol_kv, name
    ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi_k, T=w.T, lam=w.lam, Phi_V=phi_v if separate else None)
    assert rel_err(to_np(fast_out), ref) <= TOL[w.dtype], name
    assert rel_err(to_np(fast_out), to_np(dense_out)) <= TOL[w.dtype], name
    assert torch.equal(fast_out, ctx.forward(Q, K, V))               # deterministic
    # a supplied matrix has no structure to transform: the dense product takes over again
    ctx.set_phi(ctx.get_phi())
    assert torch.equal(ctx.forward(Q, K, V), dense_out)
    ctx.close()


def _random_shapes():
    """Seeded random shapes: both kernel families (bf16 with d in {64, 128} on the tensor cores, everything else on
    the FFMA kernels), token / query / measurement counts that are no multiples of any tile, odd batches."""
    r = np.random.default_rng(2024)
    out = []
    for i in range(16):
        tc = i % 2 == 0
        dtype = "bf16" if (tc or i % 4 == 1) else "fp32"
        d = int(r.choice([64, 128])) if tc else int(r.choice([8, 16, 24, 40, 72]))
        m = int(r.integers(d, 3 * d + 40))
        n = int(r.integers(m, m + 600))
        nq = int(r.integers(1, 420))
        out.append(wl.Workload(f"rand{i}", int(r.integers(1, 4)), int(r.integers(1, 4)), n, nq, d, m, dtype,
                               int(r.integers(0, 6)), float(r.choice([0.0, 0.005, 0.02])), "iid", 500 + i))
    return out


@pytest.mark.parametrize("w", _random_shapes(), ids=lambda w: f"{w.name}_{w.dtype}_B{w.B}H{w.H}_n{w.n}_nq{w.n_q}_d{w.d}_m{w.m}_T{w.T}")
def test_random_shapes_match_oracle(w):
    inp = wl.make_inputs(w)
    Q, K, V, _ = device_inputs(w, inp)
    ctx = make_ctx(w)
    phi = to_np(ctx.get_phi())
    out = to_np(ctx.forward(Q, K, V))
    stages = []
    ref = orc.csat_forward(inp["Q"], inp["K"], inp["V"], phi, T=w.T, lam=w.lam, stages=stages)
    assert np.isfinite(out).all()
    if np.abs(ref).max() == 0.0:
        assert np.abs(out).max() <= max(s["theta"] for s in stages) * TOL[w.dtype]
    else:
        assert rel_err(out, ref) <= TOL[w.dtype], w
    # the host-buffer entry point runs the same kernels over sub-ranges of (batch, head) pairs
    Qh, Kh, Vh = (t.cpu().pin_memory() for t in (Q, K, V))
    oh = torch.empty_like(Qh).pin_memory()
    ctx.forward_host(Qh, Kh, Vh, oh)
    assert torch.equal(oh, ctx.forward(Q, K, V).cpu())
    ctx.close()
