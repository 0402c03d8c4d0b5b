"""The allocation-free encode entry point against the ordinary one (needs a B200).

Some callers hold only the tensors they were handed and may not allocate device memory where they call the
operator (a plugin with a fixed memory budget, a loop that must not enter the allocator).  For them the library
keeps a fixed scratch array inside its own device image; this file checks that encoding through it gives what
flare_encode gives with a caller-allocated workspace -- twice in a row with different inputs, because the
array is shared and keeps the previous call's contents -- and that a problem too large for it is refused.
Collected last on purpose: a failure here must not hide the other tests from a run that stops at the first.
"""
import numpy as np
import pytest
import torch

from paper_2508_12594_b200 import flare, workloads
from tests._util import TOL, dev, rel_err, to_np64

pytestmark = pytest.mark.gpu


def _encode_both(inp):
    Q, K, V, mask = dev(inp.Q), dev(inp.K), dev(inp.V), dev(inp.key_mask)
    desc = flare.make_desc(Q, K)
    B, H, M, D = desc.B, desc.H, desc.M, desc.D
    assert flare.flare_workspace_bytes(desc, flare.OP_ENCODE) <= flare.STATIC_SCRATCH_BYTES
    ws = flare.alloc_workspace(desc, flare.OP_ENCODE)
    Z_ref = torch.empty(B, H, M, D, dtype=torch.float32, device="cuda")
    le_ref = torch.empty(B, H, M, dtype=torch.float32, device="cuda")
    flare.flare_encode(desc, Q, K, V, mask, Z_ref, le_ref, ws)
    Z = torch.full_like(Z_ref, float("nan"))
    le = torch.full_like(le_ref, float("nan"))
    flare.flare_encode_static_scratch(desc, Q, K, V, mask, Z, le)
    torch.cuda.synchronize()
    return (Z, le), (Z_ref, le_ref)


def test_static_scratch_encode_matches_encode_twice_in_a_row(oracle):
    cases = [
        (workloads.CONFIGS["mesh3d_1m"].with_(N=20011), "bf16"),           # many splits: most of the partial slots
        (workloads.CONFIGS["padded"].with_(B=2, N=900), "bf16"),           # fewer, differently shaped partials + mask
        (workloads.CONFIGS["tiny"], "f32"),                                # the CUDA-core path
    ]
    for w, dtype in cases:
        inp = workloads.make_inputs(w)
        (Z, le), (Z_ref, le_ref) = _encode_both(inp)
        # the same kernels with the same split plan, only the scratch lives elsewhere: bit for bit the same
        assert torch.equal(Z, Z_ref) and torch.equal(le, le_ref), w.name
        flare.flare_check(None)                                            # no bounded wait gave up on the built-in array
        # and both against the oracle, within the forward's bound
        mk = None if inp.key_mask is None else inp.key_mask.numpy()
        Zo, leo = oracle.encode(to_np64(inp.Q), to_np64(inp.K), to_np64(inp.V), key_mask=mk, scale=w.scale)
        assert rel_err(to_np64(Z), Zo) <= TOL[dtype], w.name
        fin = np.isfinite(leo)
        assert np.array_equal(np.isfinite(to_np64(le)), fin)
        assert np.abs(to_np64(le)[fin] - leo[fin]).max() <= (1e-4 if dtype == "f32" else 2e-2), w.name


def test_static_scratch_refuses_what_does_not_fit():
    big = flare.FlareDesc(64, 8, 4096, 512, 64, flare.DTYPE_BF16, 1.0)
    assert flare.flare_workspace_bytes(big, flare.OP_ENCODE) > flare.STATIC_SCRATCH_BYTES
    Q = torch.zeros(8, 512, 64, dtype=torch.bfloat16, device="cuda")
    K = torch.zeros(1, dtype=torch.bfloat16, device="cuda")        # never read: the call must fail before any launch
    Z = torch.zeros(1, dtype=torch.float32, device="cuda")
    import ctypes
    rc = flare.load().flare_encode_static_scratch(ctypes.byref(big), Q.data_ptr(), K.data_ptr(), K.data_ptr(), None,
                                                  Z.data_ptr(), None, None)
    assert rc == flare.ERR_WORKSPACE_TOO_SMALL
    assert b"scratch" in flare.load().flare_last_cuda_error()
    torch.cuda.synchronize()
