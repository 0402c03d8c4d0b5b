"""Helpers shared by the GPU parity tests: run the CUDA path through the C-ABI binding, run the oracle on the
same stored input values, compare with the relative-to-RMS bound."""
import numpy as np
import torch

from paper_2508_12594_b200 import flare

# max |err| <= tol * RMS(reference), per tensor: 1e-5 for float32 inputs, 2e-2 for bfloat16 inputs with float32
# accumulation (three bf16 roundings of relative size 2^-9 each: the softmax weights, Z and the stored Y).
TOL = {"f32": 1e-5, "bf16": 2e-2, "f16": 2e-5}
# float16 inputs run in float32 arithmetic (scores summed in double), so the float32 bound applies with a little room
# for the float16 values' larger scores, plus one rounding of a stored float16 output (2^-11 |ref|, below).
STORE_ULP = {"f32": 0.0, "bf16": 2.0 ** -8, "f16": 2.0 ** -11}


def rel_err(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    return float(np.abs(got - ref).max()) / max(rms, 1e-300)


def bf16_round(x):
    """The float64 array rounded to bfloat16 (round to nearest even) and widened again."""
    return torch.from_numpy(np.asarray(x, dtype=np.float64)).float().bfloat16().double().numpy()


# Which bound every stored-tensor comparison met: (what, bound, max|err|/RMS, (max|err| - one rounding)/RMS).
# conftest.py writes the list to the file named by FLARE_PARITY_REPORT at the end of the session.
BOUND_LOG = []


def assert_stored_close(got, ref, dtype, what):
    """The bound on a tensor that is stored in the call dtype.  Returns "stated" or "stated+rounding".

    The stated bound is max|err| <= tol * RMS(ref).  For a bfloat16 tensor it cannot hold for entries larger than
    about 5 RMS whatever the kernel does: rounding the exact value to bfloat16 is an error of up to 2^-8 |ref|,
    which passes 2e-2 RMS at |ref| = 5.12 RMS (the mesh workloads have entries of 8 RMS and more; the oracle's own
    Y rounded to bfloat16 breaks the stated bound there, see test_oracle_pins.py).  So the stated bound is tried
    first, and where it fails the bound is the stated one plus exactly one rounding of the stored value:
    |err| <= tol * RMS(ref) + 2^-8 |ref|, element by element.  Which of the two a case needed is recorded."""
    tol = TOL[dtype]
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = max(float(np.sqrt(np.mean(ref ** 2))), 1e-300)
    err = np.abs(got - ref)
    plain = float(err.max()) / rms
    if plain <= tol:
        BOUND_LOG.append((what, "stated", plain, None))
        return "stated"
    assert dtype in ("bf16", "f16"), f"{what}: max|err|/RMS = {plain:.3e} > {tol}"
    excess = float((err - STORE_ULP[dtype] * np.abs(ref)).max()) / rms
    BOUND_LOG.append((what, "stated+rounding", plain, excess))
    assert excess <= tol, f"{what}: (max|err| - one rounding of the stored value)/RMS = {excess:.3e} > {tol}"
    return "stated+rounding"


def to_np64(t):
    return None if t is None else t.double().cpu().numpy()


def dev(t):
    return None if t is None else t.cuda()


def gpu_forward(inp, scale=1.0, canary=False, stats=True, path=None):
    """flare_forward on cuda:0.  path: None (the library's choice) or flare.PATH_EXACT / PATH_FAST for this call.  With canary=True the outputs sit inside larger buffers whose margins must stay
    untouched (checked here).  stats=False is the inference call the benchmark times: Z is asked for, the two
    log-sum-exp outputs are NULL (which selects other forms of the kernels).  Returns numpy float64
    dict(Y, Z, lse_enc, lse_dec), the last two None without stats."""
    Q, K, V, mask = dev(inp.Q), dev(inp.K), dev(inp.V), dev(inp.key_mask)
    desc = flare.make_desc(Q, K, scale)
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    ws = flare.alloc_workspace(desc, flare.OP_FORWARD)
    pad = 64 if canary else 0

    def padded(shape, dtype, fill):
        n = int(np.prod(shape))
        buf = torch.full((n + 2 * pad,), fill, dtype=dtype, device="cuda")
        return buf, buf[pad:pad + n].view(*shape)

    Yb, Y = padded((B, N, H, D), K.dtype, 777.0)
    Zb, Z = padded((B, H, M, D), torch.float32, 777.0)
    leb, le = padded((B, H, M), torch.float32, 777.0)
    ldb, ld = padded((B, N, H), torch.float32, 777.0)
    if pad % 8 != 0:
        raise AssertionError("canary margin must keep 16-byte alignment")
    if path is not None:
        flare.flare_set_path(path)
    try:
        flare.flare_forward(desc, Q, K, V, mask, Y, Z, le if stats else None, ld if stats else None, ws)
    finally:
        flare.flare_set_path(flare.PATH_AUTO)
    torch.cuda.synchronize()
    flare.flare_check(ws)
    if canary:
        for buf in (Yb, Zb, leb, ldb):
            assert (buf[:pad] == 777.0).all() and (buf[-pad:] == 777.0).all(), "write outside an output buffer"
    if not stats:
        assert (le == 777.0).all() and (ld == 777.0).all(), "an output that was not asked for was written"
    return dict(Y=to_np64(Y), Z=to_np64(Z), lse_enc=to_np64(le) if stats else None, lse_dec=to_np64(ld) if stats else None)


def oracle_forward(oracle, inp, scale=1.0):
    mask = None if inp.key_mask is None else inp.key_mask.numpy()
    return oracle.forward(to_np64(inp.Q), to_np64(inp.K), to_np64(inp.V), key_mask=mask, scale=scale)


def assert_forward_close(got, ref, dtype, what=""):
    tol = TOL[dtype]
    e = rel_err(got["Z"], ref["Z"])                      # Z is float32 in memory: the stated bound as it stands
    assert e <= tol, f"{what} Z: max|err|/RMS = {e:.3e} > {tol}"
    assert_stored_close(got["Y"], ref["Y"], dtype, f"{what} Y")
    for name in ("lse_enc", "lse_dec"):
        if got[name] is None:
            continue
        fin = np.isfinite(ref[name])
        assert np.array_equal(np.isneginf(got[name]), np.isneginf(ref[name])), f"{what} {name}: -inf pattern"
        if fin.any():
            err = np.abs(got[name][fin] - ref[name][fin]).max()
            assert err <= (2e-2 if dtype == "bf16" else 1e-4), f"{what} {name}: abs err {err:.3e}"
