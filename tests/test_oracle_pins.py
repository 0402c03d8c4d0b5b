"""Pins that hold the CPU oracle to the paper and to the mathematics (no GPU).

Each test checks the oracle against something other than itself: a hand-worked example, a library attention
routine in float64, dense linear algebra on the brute-force mixing matrix, structural invariants the paper
states, finite differences.  A dropped term, a wrong sign or index, a transposed operand, or a softmax over the
wrong axis fails at least one of them.
"""
import math
import os

import numpy as np
import pytest
import torch

from paper_2508_12594_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _np(inp):
    f = lambda t: None if t is None else t.double().numpy()
    return f(inp.Q), f(inp.K), f(inp.V), (None if inp.key_mask is None else inp.key_mask.numpy()), f(inp.dY)


def _sdpa_f64(Q, K, V, scale):
    """The mixer through a library attention routine (two calls, float64, CPU): encode, then decode with
    queries and keys swapped and the latent sequence as values (Section 3.2)."""
    Qt = torch.from_numpy(Q)                               # [H,M,D]
    Kt = torch.from_numpy(K).permute(0, 2, 1, 3)           # [B,H,N,D]
    Vt = torch.from_numpy(V).permute(0, 2, 1, 3)
    Qb = Qt.unsqueeze(0).expand(Kt.shape[0], -1, -1, -1)
    sdpa = torch.nn.functional.scaled_dot_product_attention
    Z = sdpa(Qb, Kt, Vt, scale=scale)
    Y = sdpa(Kt, Qb, Z, scale=scale)
    return Z.numpy(), Y.permute(0, 2, 1, 3).numpy()


def test_closed_form_two_tokens(oracle):
    vals = {}
    for line in open(os.path.join(GOLDEN, "closed_form_two_tokens.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        vals[k] = float(v)
    Q = np.array([[[0.0], [1.0]]])                          # H=1, M=2, D=1
    K = np.array([0.0, math.log(3.0)]).reshape(1, 2, 1, 1)
    V = np.array([4.0, 8.0]).reshape(1, 2, 1, 1)
    out = oracle.forward(Q, K, V)
    got = dict(z0=out["Z"][0, 0, 0, 0], z1=out["Z"][0, 0, 1, 0], y0=out["Y"][0, 0, 0, 0], y1=out["Y"][0, 1, 0, 0],
               lse_enc0=out["lse_enc"][0, 0, 0], lse_enc1=out["lse_enc"][0, 0, 1],
               lse_dec0=out["lse_dec"][0, 0, 0], lse_dec1=out["lse_dec"][0, 1, 0])
    for k, v in vals.items():
        assert got[k] == pytest.approx(v, rel=1e-14, abs=1e-14), k


@pytest.mark.parametrize("scale", [1.0, 0.25])
@pytest.mark.parametrize("shape", [(2, 3, 50, 7, 4), (1, 2, 200, 16, 16), (2, 1, 33, 1, 8)])
def test_matches_library_attention(oracle, shape, scale):
    B, H, N, M, D = shape
    Q, K, V, _, _ = _np(workloads.make_random(B, H, N, M, D, seed=11))
    out = oracle.forward(Q, K, V, scale=scale)
    Z_ref, Y_ref = _sdpa_f64(Q, K, V, scale)
    np.testing.assert_allclose(out["Z"], Z_ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(out["Y"], Y_ref, rtol=1e-12, atol=1e-13)


def test_brute_force_mixing_matrix(oracle):
    """Y_h = (W_dec W_enc) V_h with the N x N matrix formed explicitly; rows stochastic; rank <= M."""
    B, H, N, M, D = 2, 2, 96, 5, 8
    Q, K, V, _, _ = _np(workloads.make_random(B, H, N, M, D, seed=3))
    out = oracle.forward(Q, K, V)
    for b in range(B):
        for h in range(H):
            We, Wd, W = oracle.mixing_matrices(Q, K, b, h)
            assert (We >= 0).all() and (Wd >= 0).all() and (W >= 0).all()
            np.testing.assert_allclose(We.sum(1), 1.0, rtol=0, atol=1e-13)
            np.testing.assert_allclose(Wd.sum(1), 1.0, rtol=0, atol=1e-13)
            np.testing.assert_allclose(W.sum(1), 1.0, rtol=0, atol=1e-13)
            np.testing.assert_allclose(W, Wd @ We, rtol=1e-13, atol=1e-15)
            np.testing.assert_allclose(out["Y"][b, :, h, :], W @ V[b, :, h, :], rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(out["Z"][b, h], We @ V[b, :, h, :], rtol=1e-12, atol=1e-13)
            sv = np.linalg.svd(W, compute_uv=False)
            assert (sv > 1e-10 * sv[0]).sum() <= M
            # both softmaxes come from ONE exponentiated score matrix A (spectral appendix):
            A = np.exp(Q[h] @ K[b, :, h, :].T)
            np.testing.assert_allclose(We, A / A.sum(1, keepdims=True), rtol=1e-12)
            np.testing.assert_allclose(Wd, (A / A.sum(0, keepdims=True)).T, rtol=1e-12)


def test_constant_values_and_convexity(oracle):
    B, H, N, M, D = 1, 2, 64, 6, 4
    Q, K, V, _, _ = _np(workloads.make_random(B, H, N, M, D, seed=5))
    Yc = oracle.forward(Q, K, np.full_like(V, 2.5))["Y"]
    np.testing.assert_allclose(Yc, 2.5, rtol=1e-14)
    Y = oracle.forward(Q, K, V)["Y"]
    lo = V.min(axis=1, keepdims=True) - 1e-12
    hi = V.max(axis=1, keepdims=True) + 1e-12
    assert (Y >= lo).all() and (Y <= hi).all()


def test_single_latent(oracle):
    """M = 1: every token receives the same row, the softmax-weighted average of V; with q = 0 the plain mean."""
    B, H, N, M, D = 2, 3, 40, 1, 4
    Q, K, V, _, _ = _np(workloads.make_random(B, H, N, M, D, seed=7))
    Y = oracle.forward(Q, K, V)["Y"]
    for b in range(B):
        for h in range(H):
            s = K[b, :, h, :] @ Q[h, 0]
            w = np.exp(s - s.max()); w /= w.sum()
            row = w @ V[b, :, h, :]
            np.testing.assert_allclose(Y[b, :, h, :], np.broadcast_to(row, (N, D)), rtol=1e-12, atol=1e-14)
    Y0 = oracle.forward(np.zeros_like(Q), K, V)["Y"]
    np.testing.assert_allclose(Y0, np.broadcast_to(V.mean(axis=1, keepdims=True), V.shape), rtol=1e-12, atol=1e-14)


def test_heads_independent(oracle):
    B, H, N, M, D = 1, 3, 32, 4, 4
    Q, K, V, _, _ = _np(workloads.make_random(B, H, N, M, D, seed=9))
    Y = oracle.forward(Q, K, V)["Y"]
    Q2, K2, V2 = Q.copy(), K.copy(), V.copy()
    Q2[1] += 1.0; K2[:, :, 1, :] *= -2.0; V2[:, :, 1, :] += 3.0
    Y2 = oracle.forward(Q2, K2, V2)["Y"]
    np.testing.assert_array_equal(Y[:, :, [0, 2], :], Y2[:, :, [0, 2], :])
    assert np.abs(Y[:, :, 1, :] - Y2[:, :, 1, :]).max() > 1e-3


def test_permutation_equivariance(oracle):
    B, H, N, M, D = 1, 2, 48, 5, 4
    Q, K, V, _, _ = _np(workloads.make_random(B, H, N, M, D, seed=13))
    Y = oracle.forward(Q, K, V)["Y"]
    rng = np.random.default_rng(0)
    pt = rng.permutation(N)
    Yp = oracle.forward(Q, K[:, pt], V[:, pt])["Y"]
    np.testing.assert_allclose(Yp, Y[:, pt], rtol=1e-12, atol=1e-14)
    pl = rng.permutation(M)
    Yl = oracle.forward(Q[:, pl], K, V)["Y"]
    np.testing.assert_allclose(Yl, Y, rtol=1e-12, atol=1e-14)


def test_mask_equals_deleting_tokens(oracle):
    B, H, N, M, D = 2, 2, 60, 4, 4
    inp = workloads.make_random(B, H, N, M, D, seed=17, masked_fraction=0.3)
    Q, K, V, mask, _ = _np(inp)
    out = oracle.forward(Q, K, V, key_mask=mask)
    for b in range(B):
        keep = mask[b].astype(bool)
        assert 0 < keep.sum() < N
        sub = oracle.forward(Q, K[b:b + 1, keep], V[b:b + 1, keep])
        np.testing.assert_allclose(out["Z"][b], sub["Z"][0], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(out["lse_enc"][b], sub["lse_enc"][0], rtol=1e-12)
        np.testing.assert_allclose(out["Y"][b, keep], sub["Y"][0], rtol=1e-12, atol=1e-14)
    # a batch item with no valid token: Z = 0, lse_enc = -inf, Y = 0
    mask0 = mask.copy(); mask0[0] = 0
    o0 = oracle.forward(Q, K, V, key_mask=mask0)
    assert (o0["Z"][0] == 0).all() and np.isneginf(o0["lse_enc"][0]).all() and (o0["Y"][0] == 0).all()
    np.testing.assert_array_equal(o0["Y"][1], out["Y"][1])


def test_lse_definitions(oracle):
    B, H, N, M, D = 1, 2, 30, 3, 4
    Q, K, V, _, _ = _np(workloads.make_random(B, H, N, M, D, seed=19))
    out = oracle.forward(Q, K, V, scale=0.5)
    S = 0.5 * np.einsum("hmd,bnhd->bhmn", Q, K)
    from scipy.special import logsumexp
    np.testing.assert_allclose(out["lse_enc"], logsumexp(S, axis=3), rtol=1e-13)
    np.testing.assert_allclose(out["lse_dec"], logsumexp(S, axis=2).transpose(0, 2, 1), rtol=1e-13)


def test_decode_rows_matches_full(oracle):
    B, H, N, M, D = 2, 2, 37, 5, 4
    Q, K, V, _, _ = _np(workloads.make_random(B, H, N, M, D, seed=21))
    out = oracle.forward(Q, K, V)
    rows = np.array([0, 5, 36, 37, 73])
    Yr = oracle.decode_rows(Q, K, out["Z"], rows)
    np.testing.assert_array_equal(Yr, out["Y"].reshape(B * N, H, D)[rows])


def test_eigenvalues_match_linear_time_algorithm(oracle):
    """Nonzero eigenvalues of the dense W equal the eigenvalues of the M x M matrix J J^T (Algorithm 1); they
    are real, lie in [0, 1], the largest is 1, and the returned vectors are eigenvectors of W."""
    from oracle import flare_spectral
    B, H, N, M, D = 1, 2, 80, 6, 4
    Q, K, V, _, _ = _np(workloads.make_random(B, H, N, M, D, seed=23, k_std=0.7))
    for h in range(H):
        _, _, W = oracle.mixing_matrices(Q, K, 0, h)
        ev = np.linalg.eigvals(W)
        assert np.abs(ev.imag).max() < 1e-9
        top = np.sort(ev.real)[::-1]
        lam, vecs = flare_spectral.eig_from_qk(Q[h], K[0, :, h, :])
        np.testing.assert_allclose(top[:M], lam, rtol=1e-9, atol=1e-12)
        assert np.abs(top[M:]).max() < 1e-10
        assert lam[0] == pytest.approx(1.0, abs=1e-12) and lam.min() >= -1e-14 and lam.max() <= 1 + 1e-12
        np.testing.assert_allclose(W @ vecs, vecs * lam[None, :], rtol=1e-8, atol=1e-10)


# ---------------------------------------------------------------- backward

def _loss(oracle, Q, K, V, dY, mask, scale):
    return float((oracle.forward(Q, K, V, key_mask=mask, scale=scale)["Y"] * dY).sum())


@pytest.mark.parametrize("masked", [False, True])
def test_backward_finite_differences(oracle, masked):
    B, H, N, M, D = 2, 2, 24, 3, 4
    inp = workloads.make_random(B, H, N, M, D, seed=29, masked_fraction=0.25 if masked else 0.0, with_dy=True,
                                k_std=0.6)
    Q, K, V, mask, dY = _np(inp)
    scale = 0.8
    g = oracle.backward(Q, K, V, dY, key_mask=mask, scale=scale)
    rng = np.random.default_rng(1)
    eps = 1e-6
    for name, arr in (("dQ", Q), ("dK", K), ("dV", V)):
        flat = arr.reshape(-1)
        for idx in rng.choice(flat.size, size=min(25, flat.size), replace=False):
            old = flat[idx]
            flat[idx] = old + eps; lp = _loss(oracle, Q, K, V, dY, mask, scale)
            flat[idx] = old - eps; lm = _loss(oracle, Q, K, V, dY, mask, scale)
            flat[idx] = old
            fd = (lp - lm) / (2 * eps)
            assert g[name].reshape(-1)[idx] == pytest.approx(fd, rel=2e-6, abs=2e-8), (name, idx)


def test_backward_matches_library_autograd(oracle):
    B, H, N, M, D = 2, 3, 40, 6, 8
    Q, K, V, _, dY = _np(workloads.make_random(B, H, N, M, D, seed=31, with_dy=True, k_std=0.5))
    scale = 1.0
    Qt = torch.from_numpy(Q).requires_grad_()
    Kt = torch.from_numpy(K).requires_grad_()
    Vt = torch.from_numpy(V).requires_grad_()
    sdpa = torch.nn.functional.scaled_dot_product_attention
    Kp, Vp = Kt.permute(0, 2, 1, 3), Vt.permute(0, 2, 1, 3)
    Qb = Qt.unsqueeze(0).expand(B, -1, -1, -1)
    Y = sdpa(Kp, Qb, sdpa(Qb, Kp, Vp, scale=scale), scale=scale).permute(0, 2, 1, 3)
    (Y * torch.from_numpy(dY)).sum().backward()
    g = oracle.backward(Q, K, V, dY, scale=scale)
    np.testing.assert_allclose(g["dQ"], Qt.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["dK"], Kt.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g["dV"], Vt.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_backward_value_gradient_sums(oracle):
    """dV = W^T dY and W 1 = 1, so sum_n dV_n = sum_n dY_n per (b, h, channel); masked tokens get dV = 0."""
    B, H, N, M, D = 2, 2, 50, 4, 4
    inp = workloads.make_random(B, H, N, M, D, seed=37, masked_fraction=0.2, with_dy=True)
    Q, K, V, mask, dY = _np(inp)
    g = oracle.backward(Q, K, V, dY, key_mask=mask)
    np.testing.assert_allclose(g["dV"].sum(axis=1), dY.sum(axis=1), rtol=1e-11, atol=1e-12)
    assert (g["dV"][mask == 0] == 0).all()


def test_gram_of_algorithm_one_against_the_two_softmax_matrices(oracle):
    """J = L_M^{1/2} A L_N^{1/2} has J[m,n]^2 = W_enc[m,n] W_dec[n,m] (A / row sum and A / column sum are the two softmax
    matrices), so J J^T can be rebuilt from the oracle's dense W_enc and W_dec, which come from other code."""
    from oracle import flare_spectral
    B, H, N, M, D = 1, 2, 70, 6, 4
    Q, K, V, _, _ = _np(workloads.make_random(B, H, N, M, D, seed=47))
    for h in range(H):
        We, Wd, _ = oracle.mixing_matrices(Q, K, 0, h, scale=0.6)
        J = np.sqrt(We * Wd.T)
        G, J_alg, _ = flare_spectral.gram_from_qk(Q[h], K[0, :, h], 0.6)
        np.testing.assert_allclose(J_alg, J, rtol=1e-12, atol=1e-300)
        np.testing.assert_allclose(G, J @ J.T, rtol=1e-12)
        np.testing.assert_allclose(np.trace(G), np.sum(We * Wd.T), rtol=1e-12)


def test_backward_with_separate_decode_queries(oracle):
    """The asymmetric variant's gradients: against library autograd through two attention calls with different
    queries (float64), against central differences in one entry of each query set, and, with Qd = Qe, against the
    symmetric backward (dQe + dQd = dQ)."""
    B, H, N, M, D = 2, 2, 19, 5, 4
    inp = workloads.make_random(B, H, N, M, D, seed=53, with_dy=True, k_std=0.6)
    Q, K, V, _, dY = _np(inp)
    Qd = _np(workloads.make_random(B, H, N, M, D, seed=54))[0]
    scale = 0.8
    g = oracle.backward_asym(Q, Qd, K, V, dY, scale=scale)
    Qe_t, Qd_t = torch.from_numpy(Q).requires_grad_(), torch.from_numpy(Qd).requires_grad_()
    Kt, Vt = torch.from_numpy(K).requires_grad_(), torch.from_numpy(V).requires_grad_()
    sdpa = torch.nn.functional.scaled_dot_product_attention
    Kp, Vp = Kt.permute(0, 2, 1, 3), Vt.permute(0, 2, 1, 3)
    Z = sdpa(Qe_t.unsqueeze(0).expand(B, -1, -1, -1), Kp, Vp, scale=scale)
    Y = sdpa(Kp, Qd_t.unsqueeze(0).expand(B, -1, -1, -1), Z, scale=scale).permute(0, 2, 1, 3)
    (Y * torch.from_numpy(dY)).sum().backward()
    for name, t in (("dQe", Qe_t), ("dQd", Qd_t), ("dK", Kt), ("dV", Vt)):
        np.testing.assert_allclose(g[name], t.grad.numpy(), rtol=1e-9, atol=1e-12, err_msg=name)

    def loss(Qe_, Qd_):
        Zl, _ = oracle.encode(Qe_, K, V, scale=scale)
        Yl, _ = oracle.decode(Qd_, K, Zl, scale=scale)
        return float((Yl * dY).sum())

    eps = 1e-6
    for which, idx in (("dQe", (1, 2, 3)), ("dQd", (0, 4, 1))):
        Qp, Qm = (Q.copy(), Qd.copy()), (Q.copy(), Qd.copy())
        k = 0 if which == "dQe" else 1
        Qp[k][idx] += eps
        Qm[k][idx] -= eps
        fd = (loss(*Qp) - loss(*Qm)) / (2 * eps)
        assert abs(fd - g[which][idx]) <= 1e-6 * max(1.0, abs(fd)), which
    sym = oracle.backward(Q, K, V, dY, scale=scale)
    same = oracle.backward_asym(Q, Q, K, V, dY, scale=scale)
    np.testing.assert_allclose(same["dQe"] + same["dQd"], sym["dQ"], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(same["dK"], sym["dK"], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(same["dV"], sym["dV"], rtol=1e-11, atol=1e-13)


def test_backward_rows_matches_full(oracle):
    """The sampled-rows backward is the full backward restricted to the listed tokens, bit for bit (dQ and dZ are
    full reductions in both)."""
    B, H, N, M, D = 2, 2, 41, 6, 4
    inp = workloads.make_random(B, H, N, M, D, seed=43, masked_fraction=0.2, with_dy=True)
    Q, K, V, mask, dY = _np(inp)
    full = oracle.backward(Q, K, V, dY, key_mask=mask, scale=0.7)
    rows = np.array([0, 3, 40, 41, 57, 81])
    part = oracle.backward_rows(Q, K, V, dY, rows, key_mask=mask, scale=0.7)
    np.testing.assert_array_equal(part["dQ"], full["dQ"])
    np.testing.assert_array_equal(part["dZ"], full["dZ"])
    np.testing.assert_array_equal(part["dK_rows"], full["dK"].reshape(B * N, H, D)[rows])
    np.testing.assert_array_equal(part["dV_rows"], full["dV"].reshape(B * N, H, D)[rows])


def test_bf16_storage_alone_breaks_the_stated_bound(oracle):
    """On the 2-D mesh workload (one batch item at its full length) the exact Y has entries of many RMS, and rounding
    the oracle's own Y to bfloat16 is by itself an error above 2e-2 RMS(Y): no kernel that stores bfloat16 can
    meet the stated bound there.  This is why the GPU tests allow exactly one rounding of the stored value on top
    of the stated bound where the stated bound fails (and report that they did)."""
    w = workloads.CONFIGS["mesh2d"].with_(B=1)
    Q, K, V, _, _ = _np(workloads.make_inputs(w))
    Z, _ = oracle.encode(Q, K, V)
    # the rows with the largest keys carry the largest outputs: decode those and a seeded sample for the RMS
    knorm = np.abs(K).reshape(w.N, -1).max(axis=1)
    rows = np.unique(np.concatenate([np.argsort(knorm)[-2048:], np.random.default_rng(0).choice(w.N, 8192, replace=False)]))
    sample = np.random.default_rng(1).choice(w.N, 8192, replace=False)
    Y = oracle.decode_rows(Q, K, Z, rows)
    rms = np.sqrt(np.mean(oracle.decode_rows(Q, K, Z, sample) ** 2))
    Yb = torch.from_numpy(Y).float().bfloat16().double().numpy()
    assert np.abs(Y).max() > 5.12 * rms
    assert np.abs(Yb - Y).max() > 2e-2 * rms             # storage rounding alone exceeds the stated bound
    assert (np.abs(Yb - Y) <= 2.0 ** -8 * np.abs(Y)).all()


def test_workload_recipes_are_seeded():
    w = workloads.CONFIGS["tiny"]
    a, b = workloads.make_inputs(w), workloads.make_inputs(w)
    assert torch.equal(a.Q, b.Q) and torch.equal(a.K, b.K) and torch.equal(a.V, b.V)
    assert a.K.shape == (1, 1024, 2, 16) and a.Q.shape == (2, 16, 16) and a.K.dtype == torch.float32
    p = workloads.make_inputs(workloads.CONFIGS["padded"].with_(B=2, N=200))
    assert p.key_mask.sum().item() == 2 * 180 and p.K.dtype == torch.bfloat16
    assert (p.K[p.key_mask == 0] == 0).all() and (p.V[p.key_mask == 0] == 0).all()
    c = workloads.make_inputs(workloads.CONFIGS["mesh3d_1m"].with_(N=512))
    assert c.K.shape == (1, 512, 8, 16)
