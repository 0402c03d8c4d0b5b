"""Parity at the benchmark workloads' full sizes (needs a B200).

The oracle computes every reduction in full (the latent sequence Z and its log-sum-exp rows: one pass over all
N tokens per latent) and the rows of Y for a seeded sample of tokens one by one (rows are independent given Z);
the CUDA path runs the whole problem through flare_forward, both as the training call (all statistics asked
for) and as the inference call bench.py times (Z only, log-sum-exp outputs NULL: other forms of the kernels).
Backward: where the oracle finishes the whole backward in seconds the gradients are compared in full; at a
million tokens the oracle runs its reductions over all tokens in full (dQ, dZ) and the per-token gradients dK, dV
for a seeded sample of tokens.
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
    workloads.sweep_point(1048576, 32),
    workloads.sweep_point(1048576, 128),
    workloads.sweep_point(1048576, 512),
    # the paper's million-point shape (head width 8, 1024 latents: narrow kernels, decode in latent ranges), cut to
    # a length the oracle encodes in seconds
    workloads.CONFIGS["field_1m"].with_(N=65536, name="field_1m@N=65536"),
]


_REF_CACHE = {}


def _forward_reference(oracle, w, inp):
    """Z and lse_enc in full and a seeded sample of rows of Y from the oracle (shared by the two call forms)."""
    if w.name not in _REF_CACHE:
        _REF_CACHE.clear()                                  # one workload at a time: the inputs are large
        Qn, Kn, Vn = to_np64(inp.Q), to_np64(inp.K), to_np64(inp.V)
        mk = None if inp.key_mask is None else inp.key_mask.numpy()
        Z_ref, le_ref = oracle.encode(Qn, Kn, Vn, key_mask=mk, scale=w.scale)
        rng = np.random.default_rng(w.seed)
        rows = np.sort(rng.choice(w.B * w.N, size=min(SAMPLE_ROWS, w.B * w.N), replace=False))
        # the last tile of every batch item and the first rows are always in the sample
        rows = np.unique(np.concatenate([rows, np.arange(0, 128), np.arange(w.B * w.N - 130, w.B * w.N)]))
        Y_ref = oracle.decode_rows(Qn, Kn, Z_ref, rows, scale=w.scale)          # [rows, H, D]
        _REF_CACHE[w.name] = (Z_ref, le_ref, rows, Y_ref)
    return _REF_CACHE[w.name]


@pytest.mark.parametrize("stats", [True, False], ids=["train", "infer"])      # varies fastest: one oracle run per workload
@pytest.mark.parametrize("w", FULL, ids=lambda w: w.name)
def test_forward_full_size_sampled(oracle, w, stats):
    inp = workloads.make_inputs(w)
    Q, K, V, mask = dev(inp.Q), dev(inp.K), dev(inp.V), dev(inp.key_mask)
    desc = flare.make_desc(Q, K, w.scale)
    ws = flare.alloc_workspace(desc, flare.OP_FORWARD)
    Y = torch.empty_like(K)
    Z = torch.empty(w.B, w.H, w.M, w.D, dtype=torch.float32, device="cuda")
    le = torch.empty(w.B, w.H, w.M, dtype=torch.float32, device="cuda") if stats else None
    ld = torch.empty(w.B, w.N, w.H, dtype=torch.float32, device="cuda") if stats else None
    flare.flare_forward(desc, Q, K, V, mask, Y, Z, le, ld, ws)      # stats=False: exactly the benchmark's call
    torch.cuda.synchronize()
    flare.flare_check(ws)
    Z_ref, le_ref, rows, Y_ref = _forward_reference(oracle, w, inp)
    tol = TOL[w.dtype]
    assert rel_err(to_np64(Z), Z_ref) <= tol, f"{w.name} Z"
    if stats:
        fin = np.isfinite(le_ref)
        assert np.abs(to_np64(le)[fin] - le_ref[fin]).max() <= 2e-2
    Y_got = to_np64(Y.view(w.B * w.N, w.H, w.D)[torch.from_numpy(rows).cuda()])
    # error scale: RMS of the sampled reference rows (a seeded sample of the whole tensor)
    assert_stored_close(Y_got, Y_ref, w.dtype, f"{w.name} {'train' if stats else 'infer'} Y (sampled rows)")


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


# At a million tokens the oracle's per-token loop over every token would take many minutes: its reductions (dZ, dQ)
# run in full, dK and dV for a seeded sample of tokens.  (The 512-latent point of the sweep is left to the
# N = 131072 case above and the forward test: its oracle backward alone takes several minutes on the host cores.)
BACKWARD_SAMPLED = [workloads.CONFIGS["mesh3d_1m"].with_(backward=True), workloads.sweep_point(1048576, 32),
                    workloads.sweep_point(1048576, 128)]


@pytest.mark.parametrize("w", BACKWARD_SAMPLED, ids=lambda w: w.name)
def test_backward_full_size_sampled(oracle, w):
    inp = workloads.make_inputs(w)
    Q, K, V, mask, dY = dev(inp.Q), dev(inp.K), dev(inp.V), dev(inp.key_mask), dev(inp.dY)
    _, dQ, dK, dV = flare.forward_backward(Q, K, V, dY, mask, w.scale, check=True)
    torch.cuda.synchronize()
    rng = np.random.default_rng(w.seed + 1)
    rows = np.sort(rng.choice(w.B * w.N, size=SAMPLE_ROWS, replace=False))
    rows = np.unique(np.concatenate([rows, np.arange(0, 128), np.arange(w.B * w.N - 130, w.B * w.N)]))
    ref = oracle.backward_rows(to_np64(inp.Q), to_np64(inp.K), to_np64(inp.V), to_np64(inp.dY), rows,
                               key_mask=None if inp.key_mask is None else inp.key_mask.numpy(), scale=w.scale)
    idx = torch.from_numpy(rows).cuda()
    got = dict(dQ=to_np64(dQ), dK=to_np64(dK.view(w.B * w.N, w.H, w.D)[idx]), dV=to_np64(dV.view(w.B * w.N, w.H, w.D)[idx]))
    assert_grads_close(got, dict(dQ=ref["dQ"], dK=ref["dK_rows"], dV=ref["dV_rows"]), w.dtype, f"{w.name} (sampled rows)")
