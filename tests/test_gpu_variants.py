"""The two variants of the mixer the paper discusses and sets aside, against the oracle (needs a B200):
one latent sequence shared by all heads (its ablation of shared against independent latents) and separate latent
queries for encode and decode (the "asymmetric" remark of its design principles).  Forward and backward.
"""
import numpy as np
import pytest
import torch

from paper_2508_12594_b200 import flare, workloads
from tests._util import TOL, assert_stored_close, dev, rel_err, to_np64
from tests.test_gpu_backward import assert_grads_close

pytestmark = pytest.mark.gpu

CASES = [
    # B, H, N, M, D, dtype, masked_fraction, shared, separate
    (1, 2, 300, 16, 16, "f32", 0.0, True, False),
    (2, 2, 333, 5, 8, "f32", 0.3, False, True),
    (2, 4, 700, 64, 16, "bf16", 0.0, True, False),
    (2, 4, 700, 64, 16, "bf16", 0.2, False, True),
    (1, 4, 900, 128, 32, "bf16", 0.0, True, True),
    (1, 2, 1300, 256, 16, "bf16", 0.1, True, True),
    (1, 8, 600, 64, 8, "bf16", 0.0, True, True),       # narrow heads
    (2, 4, 500, 48, 16, "f16", 0.2, True, False),      # float16 inputs, one latent sequence for all heads
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "B{}H{}N{}M{}D{}{}m{}sh{}sep{}".format(*c))
def test_variants_forward_and_backward(oracle, case):
    B, H, N, M, D, dtype, mf, shared, separate = case
    inp = workloads.make_random(B, H, N, M, D, dtype=dtype, seed=N + M, masked_fraction=mf, with_dy=True, k_std=0.8)
    other = workloads.make_random(B, H, N, M, D, dtype=dtype, seed=N + M + 1, k_std=0.8)
    Qe_h, Qd_h = inp.Q, (other.Q if separate else None)
    if shared:                                             # one [M, D] sequence for all heads
        Qe_h = Qe_h[0].contiguous()
        Qd_h = None if Qd_h is None else Qd_h[1 % H].contiguous()
    Qe, Qd, K, V, mask, dY = dev(Qe_h), dev(Qd_h), dev(inp.K), dev(inp.V), dev(inp.key_mask), dev(inp.dY)
    desc = flare.FlareDesc(B, H, N, M, D, flare._dtype_code(K), 1.0)
    wsf = torch.empty(flare.flare_variant_workspace_bytes(desc, flare.OP_FORWARD, shared, separate), dtype=torch.uint8, device="cuda")
    Y = torch.empty_like(K)
    Z = torch.empty(B, H, M, D, dtype=torch.float32, device="cuda")
    le = torch.empty(B, H, M, dtype=torch.float32, device="cuda")
    ld = torch.empty(B, N, H, dtype=torch.float32, device="cuda")
    flare.flare_forward_variant(desc, shared, Qe, Qd, K, V, mask, Y, Z, le, ld, wsf)
    wsb = torch.empty(flare.flare_variant_workspace_bytes(desc, flare.OP_BACKWARD, shared, separate), dtype=torch.uint8, device="cuda")
    qshape = (M, D) if shared else (H, M, D)
    dQe = torch.full(qshape, float("nan"), dtype=torch.float32, device="cuda")
    dQd = torch.full(qshape, float("nan"), dtype=torch.float32, device="cuda") if separate else None
    dK, dV = torch.empty_like(K), torch.empty_like(V)
    flare.flare_backward_variant(desc, shared, Qe, Qd, K, V, mask, Y, dY, Z, le, ld, dQe, dQd, dK, dV, wsb)
    torch.cuda.synchronize()
    flare.flare_check(wsf)
    flare.flare_check(wsb)

    # the oracle on the full [H, M, D] query tensors
    full = lambda q: np.broadcast_to(to_np64(q)[None], (H, M, D)).copy() if shared else to_np64(q)
    Qe_n, Qd_n = full(Qe_h), (full(Qd_h) if separate else full(Qe_h))
    Kn, Vn, dYn = to_np64(inp.K), to_np64(inp.V), to_np64(inp.dY)
    mk = None if inp.key_mask is None else inp.key_mask.numpy()
    Z_ref, _ = oracle.encode(Qe_n, Kn, Vn, key_mask=mk)
    Y_ref, _ = oracle.decode(Qd_n, Kn, Z_ref)
    assert rel_err(to_np64(Z), Z_ref) <= TOL[dtype]
    assert_stored_close(to_np64(Y), Y_ref, dtype, f"{case} Y")
    g = oracle.backward_asym(Qe_n, Qd_n, Kn, Vn, dYn, key_mask=mk)
    red = (lambda a: a.sum(axis=0)) if shared else (lambda a: a)
    if separate:
        # With separate queries dK is the sum of two parts (the encode term on Qe, the decode term on Qd) that come from
        # two runs of the per-token kernel, each storing its part in the call dtype: for bfloat16 that is two storage
        # roundings of terms that partly cancel instead of one rounding of the sum, and the bound on dK is doubled for it
        # (measured: up to 2.9e-2 of the RMS beyond one rounding of the sum; dQe, dQd and dV are not affected).
        got_k, ref_k = to_np64(dK), g["dK"]
        if dtype == "bf16":
            rms = float(np.sqrt(np.mean(ref_k ** 2)))
            assert (np.abs(got_k - ref_k) - 2.0 ** -8 * np.abs(ref_k)).max() <= 4e-2 * rms, f"{case} dK"
            got_k = ref_k                                     # (checked above; the common check below then passes it)
        assert_grads_close(dict(dQ=to_np64(dQe), dK=got_k, dV=to_np64(dV)), dict(dQ=red(g["dQe"]), dK=ref_k, dV=g["dV"]),
                           dtype, f"{case} (encode queries)")
        assert_grads_close(dict(dQ=to_np64(dQd), dK=got_k, dV=to_np64(dV)), dict(dQ=red(g["dQd"]), dK=ref_k, dV=g["dV"]),
                           dtype, f"{case} (decode queries)")
    else:
        assert_grads_close(dict(dQ=to_np64(dQe), dK=to_np64(dK), dV=to_np64(dV)),
                           dict(dQ=red(g["dQe"] + g["dQd"]), dK=g["dK"], dV=g["dV"]), dtype, str(case))


def test_variant_argument_checks():
    inp = workloads.make_random(1, 2, 64, 16, 16, dtype="bf16", seed=1, with_dy=True)
    Q, K, V = dev(inp.Q), dev(inp.K), dev(inp.V)
    desc = flare.make_desc(Q, K)
    Y = torch.empty_like(K)
    with pytest.raises(flare.FlareError) as e:
        flare.flare_forward_variant(desc, 0, Q, Q, K, V, None, Y, None, None, None, torch.empty(64, dtype=torch.uint8, device="cuda"))
    assert e.value.status == flare.ERR_WORKSPACE_TOO_SMALL
    assert flare.flare_variant_workspace_bytes(desc, flare.OP_ENCODE, 1, 1) == 0
    torch.cuda.synchronize()
