"""Parity at the benchmark workloads' full sizes, in the launch configuration bench.py times (needs a B200).

The oracle computes every reduction in full (the latent sequence Z and its log-sum-exp rows: one pass over all
N tokens per latent) and the rows of Y for a seeded sample of tokens one by one (rows are independent given Z);
the CUDA path runs the whole problem through flare_forward exactly as the benchmark does.  Where the workload
has a backward pass and the oracle finishes it in seconds, the gradients are compared in full.
"""
import numpy as np
import pytest
import torch

from paper_2508_12594_b200 import flare, workloads
from tests._util import TOL, assert_stored_close, dev, rel_err, to_np64
from tests.test_gpu_backward import assert_grads_close

pytestmark = pytest.mark.gpu

SAMPLE_ROWS = 4096

FULL = [
    workloads.CONFIGS["mesh2d"],
    workloads.CONFIGS["padded"],
    workloads.CONFIGS["mesh3d_1m"],
    workloads.sweep_point(131072, 32),
    workloads.sweep_point(131072, 128),
    workloads.sweep_point(131072, 512),
    # the paper's million-point shape (head width 8, 1024 latents: narrow kernels, decode in latent ranges), cut to
    # a length the oracle encodes in seconds
    workloads.CONFIGS["field_1m"].with_(N=65536, name="field_1m@N=65536"),
]


@pytest.mark.parametrize("w", FULL, ids=lambda w: w.name)
def test_forward_full_size_sampled(oracle, w):
    inp = workloads.make_inputs(w)
    Q, K, V, mask = dev(inp.Q), dev(inp.K), dev(inp.V), dev(inp.key_mask)
    Y, Z, le, ld = flare.forward(Q, K, V, mask, scale=w.scale, want_stats=True)
    torch.cuda.synchronize()
    Qn, Kn, Vn = to_np64(inp.Q), to_np64(inp.K), to_np64(inp.V)
    mk = None if inp.key_mask is None else inp.key_mask.numpy()
    Z_ref, le_ref = oracle.encode(Qn, Kn, Vn, key_mask=mk, scale=w.scale)
    tol = TOL[w.dtype]
    assert rel_err(to_np64(Z), Z_ref) <= tol, f"{w.name} Z"
    fin = np.isfinite(le_ref)
    assert np.abs(to_np64(le)[fin] - le_ref[fin]).max() <= 2e-2
    rng = np.random.default_rng(w.seed)
    rows = np.sort(rng.choice(w.B * w.N, size=min(SAMPLE_ROWS, w.B * w.N), replace=False))
    # the last tile of every batch item and the first rows are always in the sample
    rows = np.unique(np.concatenate([rows, np.arange(0, 128), np.arange(w.B * w.N - 130, w.B * w.N)]))
    Y_ref = oracle.decode_rows(Qn, Kn, Z_ref, rows, scale=w.scale)              # [rows, H, D]
    Y_got = to_np64(Y).reshape(w.B * w.N, w.H, w.D)[rows]
    # error scale: RMS of the sampled reference rows (a seeded sample of the whole tensor)
    assert_stored_close(Y_got, Y_ref, w.dtype, f"{w.name} Y (sampled rows)")


BACKWARD_FULL = [workloads.CONFIGS["padded"], workloads.CONFIGS["mesh2d"].with_(backward=True),
                 workloads.sweep_point(131072, 128),
                 workloads.CONFIGS["field_1m"].with_(N=8192, name="field_1m@N=8192")]


@pytest.mark.parametrize("w", BACKWARD_FULL, ids=lambda w: w.name)
def test_backward_full_size(oracle, w):
    """Whole workloads at full size (the long-sequence classification batch, the 2-D mesh batch with its paired
    heads, one long sequence): all three gradients, element by element."""
    inp = workloads.make_inputs(w)
    Q, K, V, mask, dY = dev(inp.Q), dev(inp.K), dev(inp.V), dev(inp.key_mask), dev(inp.dY)
    _, dQ, dK, dV = flare.forward_backward(Q, K, V, dY, mask, w.scale, check=True)
    torch.cuda.synchronize()
    ref = oracle.backward(to_np64(inp.Q), to_np64(inp.K), to_np64(inp.V), to_np64(inp.dY),
                          key_mask=None if inp.key_mask is None else inp.key_mask.numpy(), scale=w.scale)
    assert_grads_close(dict(dQ=to_np64(dQ), dK=to_np64(dK), dV=to_np64(dV)), ref, w.dtype, w.name)
