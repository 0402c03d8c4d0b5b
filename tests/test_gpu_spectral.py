"""Spectral analysis on the GPU (Algorithm 1 of the paper's spectral appendix) against the oracle (needs a B200).

flare_spectral_gram forms the M x M matrix J J^T from Q_lat, K and the two log-sum-exp outputs of flare_forward;
flare_spectral_eig solves the M x M symmetric eigenproblems.  The oracle (oracle/flare_spectral.py, pinned on the CPU
against a dense eigendecomposition of the N x N mixing matrix) follows the algorithm's steps in float64.
"""
import numpy as np
import pytest
import torch

from oracle import flare_spectral
from paper_2508_12594_b200 import flare, workloads
from tests._util import dev, to_np64

pytestmark = pytest.mark.gpu

CASES = [
    # B, H, N, M, D, dtype, q_std
    (1, 2, 1024, 16, 16, "f32", 1.0),        # the tiny configuration's shape: CUDA cores
    (2, 2, 972, 64, 16, "bf16", 1.0),        # the paper's spectra are of N = 972, M = 64: one latent block on the tensor cores
    (1, 2, 3001, 128, 16, "bf16", 0.7),      # all 128 lanes, several tiles, a ragged tail
    (1, 2, 1300, 256, 16, "bf16", 0.7),      # more than 128 latents, a multiple of 64: pairs of 64-latent blocks on the tensor cores
    (2, 2, 900, 192, 32, "bf16", 0.6),       # three blocks
    (1, 4, 1500, 128, 32, "bf16", 0.5),
    (1, 2, 700, 48, 32, "bf16", 1.0),        # a latent block that is mostly empty lanes
    (1, 2, 600, 400, 16, "bf16", 0.5),       # not a multiple of 64: CUDA cores
    (1, 2, 500, 32, 8, "bf16", 1.0),         # narrow heads: CUDA cores
]


def _forward_stats(Q, K, scale):
    V = torch.zeros_like(K)
    flare.flare_set_path(flare.PATH_EXACT)
    try:
        _, _, le, ld = flare.forward(Q, K, V, scale=scale, want_stats=True)
    finally:
        flare.flare_set_path(flare.PATH_AUTO)
    return le, ld


@pytest.mark.parametrize("case", CASES, ids=lambda c: "B{}H{}N{}M{}D{}{}q{}".format(*c))
def test_gram_and_eigenvalues(case):
    B, H, N, M, D, dtype, q_std = case
    inp = workloads.make_random(B, H, N, M, D, dtype=dtype, seed=N + M, k_std=0.8, q_std=q_std)
    Q, K = dev(inp.Q), dev(inp.K)
    desc = flare.make_desc(Q, K, 1.0)
    le, ld = _forward_stats(Q, K, 1.0)
    ws = flare.alloc_workspace(desc, flare.OP_SPECTRAL)
    G = torch.full((B, H, M, M), float("nan"), dtype=torch.float32, device="cuda")
    flare.flare_spectral_gram(desc, Q, K, le, ld, G, ws)
    torch.cuda.synchronize()
    flare.flare_check(ws)
    Gh = to_np64(G)
    ev = torch.empty(B, H, M, dtype=torch.float32, device="cuda")
    U = torch.empty(B, H, M, M, dtype=torch.float32, device="cuda")
    flare.flare_spectral_eig(G.clone(), ev, U)
    torch.cuda.synchronize()
    evh, Uh = to_np64(ev), to_np64(U)
    tol = 1e-4 if dtype == "f32" else 2e-2
    Qn, Kn = to_np64(inp.Q), to_np64(inp.K)
    for b in range(B):
        for h in range(H):
            G_ref, _, _ = flare_spectral.gram_from_qk(Qn[h], Kn[b, :, h], 1.0)
            rms = np.sqrt(np.mean(G_ref ** 2))
            assert np.abs(Gh[b, h] - G_ref).max() <= tol * rms, (b, h)
            assert np.abs(Gh[b, h] - Gh[b, h].T).max() <= 1e-6 * max(rms, 1e-30) + 1e-7     # symmetric as stored
            ev_ref, _ = flare_spectral.eig_from_qk(Qn[h], Kn[b, :, h], 1.0)
            # eigenvalues of the mixing matrix: in [0, 1], the largest is 1 (W is row-stochastic)
            assert np.abs(evh[b, h] - ev_ref).max() <= (1e-4 if dtype == "f32" else 5e-3), (b, h)
            assert abs(evh[b, h, 0] - 1.0) <= (1e-4 if dtype == "f32" else 5e-3)
            assert (np.diff(evh[b, h]) <= 1e-6).all()
            # the Jacobi kernel on its own: U diag(ev) U^T rebuilds the G it was given, U is orthogonal
            rebuilt = (Uh[b, h] * evh[b, h][None, :]) @ Uh[b, h].T
            assert np.abs(rebuilt - Gh[b, h]).max() <= 2e-4        # float32 rotations, up to 400 x 400
            assert np.abs(Uh[b, h].T @ Uh[b, h] - np.eye(M)).max() <= max(2e-4, 4e-6 * M)   # (rounding grows with the number of rotations)


def test_spectral_error_paths():
    inp = workloads.make_random(1, 2, 64, 16, 16, dtype="bf16", seed=1)
    Q, K = dev(inp.Q), dev(inp.K)
    desc = flare.make_desc(Q, K)
    le, ld = _forward_stats(Q, K, 1.0)
    G = torch.empty(1, 2, 16, 16, dtype=torch.float32, device="cuda")
    with pytest.raises(flare.FlareError) as e:
        flare.flare_spectral_gram(desc, Q, K, le, ld, G, torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == flare.ERR_WORKSPACE_TOO_SMALL
    import ctypes
    rc = flare.load().flare_spectral_eig(1, 4096, G.data_ptr(), G.data_ptr(), None, 0, None)
    assert rc == flare.ERR_INVALID_ARG
    torch.cuda.synchronize()
