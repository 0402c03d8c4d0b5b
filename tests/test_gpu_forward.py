"""Parity of the CUDA path against the CPU oracle, element by element, through the C-ABI (needs a B200)."""
import numpy as np
import pytest
import torch

from paper_2508_12594_b200 import flare, workloads
from tests._util import TOL, assert_forward_close, dev, gpu_forward, oracle_forward, rel_err, to_np64

pytestmark = pytest.mark.gpu


def test_tiny_config_fp32(oracle):
    w = workloads.CONFIGS["tiny"]
    inp = workloads.make_inputs(w)
    assert_forward_close(gpu_forward(inp, canary=True), oracle_forward(oracle, inp), "f32", "tiny")


# Shapes of the benchmark workloads at sizes the oracle finishes in seconds; N spans several tiles and ends in
# a ragged tail.
SCALED = [
    workloads.CONFIGS["mesh2d"].with_(B=2, N=3001),
    workloads.CONFIGS["padded"].with_(B=3, N=1000),
    workloads.CONFIGS["mesh3d_1m"].with_(N=5003),
    workloads.sweep_point(2500, 32),
    workloads.sweep_point(2500, 128),
    workloads.sweep_point(1300, 512),
]


# stats: the training call (Z and both log-sum-exp outputs) or the inference call the benchmark times (Z only; the
# library then runs other forms of its kernels: single bfloat16 encode weights, no statistics written).
# path: the exact forms of the tensor-core kernels (running maximum) or the fast ones (none; polynomial exponentials),
# forced, because left to itself the library takes the fast forms only for problems larger than these.
STATS = pytest.mark.parametrize("stats,path", [(True, flare.PATH_EXACT), (False, flare.PATH_EXACT), (True, flare.PATH_FAST),
                                               (False, flare.PATH_FAST)], ids=["train", "infer", "train-fast", "infer-fast"])


def _mode(stats, path):
    return ("train" if stats else "infer") + ("-fast" if path == flare.PATH_FAST else "")


@pytest.mark.parametrize("w", SCALED, ids=lambda w: w.name)
@pytest.mark.parametrize("paper_scale", [True, False], ids=["s=1", "s=1/sqrtD"])
@STATS
def test_scaled_down_workloads(oracle, w, paper_scale, stats, path):
    scale = 1.0 if paper_scale else w.D ** -0.5
    inp = workloads.make_inputs(w)
    assert_forward_close(gpu_forward(inp, scale, canary=True, stats=stats, path=path), oracle_forward(oracle, inp, scale),
                         w.dtype, f"{w.name} {_mode(stats, path)}")


EDGE = [
    # B, H, N, M, D, dtype, masked_fraction
    (1, 1, 1, 16, 16, "bf16", 0.0),
    (1, 1, 1, 1, 8, "f32", 0.0),
    (2, 3, 7, 16, 8, "bf16", 0.0),
    (1, 2, 127, 48, 16, "bf16", 0.0),
    (1, 2, 129, 64, 32, "bf16", 0.3),
    (2, 1, 300, 256, 64, "bf16", 0.0),
    (1, 1, 515, 512, 16, "bf16", 0.5),
    (1, 2, 1000, 80, 32, "bf16", 0.0),
    (2, 3, 1100, 32, 16, "bf16", 0.2),     # odd head count: one head per CTA although M <= 64
    (1, 4, 900, 16, 16, "bf16", 0.0),      # two heads per CTA, most latent lanes empty
    (1, 6, 450, 64, 32, "bf16", 0.3),      # two heads per CTA, all lanes in use, padding
    # head width 8 on the tensor cores: token tiles of 16 columns span two heads (the last head's upper half lies
    # beyond the tensor); a single head stays on the CUDA cores
    (2, 4, 1100, 64, 8, "bf16", 0.2),
    (1, 3, 900, 256, 8, "bf16", 0.0),
    (1, 2, 700, 400, 8, "bf16", 0.0),
    (1, 1, 300, 32, 8, "bf16", 0.0),
    # head width 4 (the paper's other setting for its PDE models)
    (2, 4, 300, 32, 4, "bf16", 0.1),
    (1, 16, 700, 64, 4, "bf16", 0.0),
    (12, 16, 500, 144, 4, "bf16", 0.2),
    (1, 2, 300, 32, 4, "bf16", 0.0),       # two heads of width 4: narrower than a tile, CUDA cores
    (1, 2, 200, 7, 4, "f32", 0.0),
    # more than 512 latents (the paper's million-point study goes to 2048)
    (1, 2, 700, 1024, 16, "bf16", 0.0),
    (1, 2, 300, 2048, 8, "bf16", 0.1),
    (2, 1, 400, 640, 32, "bf16", 0.0),
    (1, 2, 300, 1040, 16, "bf16", 0.2),     # decode ranges 4 x 256 + 16
    (3, 2, 333, 5, 32, "f32", 0.4),
    (1, 1, 2049, 300, 64, "f32", 0.0),
    (1, 4, 64, 1, 16, "f32", 0.0),
    # float16 inputs (the type the paper trains in): every entry point takes them, on the CUDA-core kernels
    (2, 3, 333, 48, 16, "f16", 0.3),
    (1, 2, 700, 300, 32, "f16", 0.0),
    (1, 4, 257, 7, 8, "f16", 0.0),
    (1, 2, 130, 64, 64, "f16", 0.2),
]


@pytest.mark.parametrize("case", EDGE, ids=lambda c: "B{}H{}N{}M{}D{}{}m{}".format(*c))
@STATS
def test_edge_shapes(oracle, case, stats, path):
    B, H, N, M, D, dtype, mf = case
    if dtype != "bf16" and path == flare.PATH_FAST:
        pytest.skip("float32 and float16 inputs run on the CUDA cores: one form only")
    inp = workloads.make_random(B, H, N, M, D, dtype=dtype, seed=N + M, masked_fraction=mf, k_std=0.8)
    assert_forward_close(gpu_forward(inp, canary=True, stats=stats, path=path), oracle_forward(oracle, inp), dtype,
                         f"{case} {_mode(stats, path)}")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_mask_degenerate_cases(oracle, dtype):
    """All but one token masked; one batch item entirely masked (Z = 0, lse_enc = -inf, Y = 0)."""
    inp = workloads.make_random(2, 2, 200, 16, 16, dtype=dtype, seed=5)
    mask = torch.zeros(2, 200, dtype=torch.uint8)
    mask[0, 137] = 1
    inp.key_mask = mask
    got, ref = gpu_forward(inp, canary=True), oracle_forward(oracle, inp)
    assert_forward_close(got, ref, dtype, "degenerate mask")
    assert (got["Z"][1] == 0).all() and (got["Y"][1] == 0).all() and np.isneginf(got["lse_enc"][1]).all()
    np.testing.assert_allclose(got["Z"][0], np.broadcast_to(to_np64(inp.V)[0, 137][:, None, :], got["Z"][0].shape),
                               rtol=1e-6)


def test_single_latent_broadcasts_one_row(oracle):
    inp = workloads.make_random(1, 2, 500, 1, 16, dtype="f32", seed=3)
    got = gpu_forward(inp)
    assert np.abs(got["Y"] - got["Y"][:, :1]).max() == 0.0
    assert_forward_close(got, oracle_forward(oracle, inp), "f32", "M=1")


def test_large_scores_do_not_overflow(oracle):
    """Scores of several tens (natural units): the running maximum keeps every exponential finite."""
    inp = workloads.make_random(1, 2, 700, 32, 32, dtype="bf16", seed=9, k_std=2.5, q_std=2.0)
    got, ref = gpu_forward(inp), oracle_forward(oracle, inp)
    assert np.isfinite(got["Y"]).all()
    assert_forward_close(got, ref, "bf16", "large scores")


@pytest.mark.parametrize("w", [workloads.CONFIGS["tiny"], workloads.CONFIGS["mesh3d_1m"].with_(N=40000)],
                         ids=lambda w: w.name)
def test_bitwise_reproducible(w):
    inp = workloads.make_inputs(w)
    Q, K, V = dev(inp.Q), dev(inp.K), dev(inp.V)
    outs = [flare.forward(Q, K, V, want_stats=True) for _ in range(3)]
    torch.cuda.synchronize()
    for o in outs[1:]:
        for a, b in zip(outs[0], o):
            assert torch.equal(a, b)


def test_encode_then_decode_equals_forward(oracle):
    inp = workloads.make_inputs(workloads.CONFIGS["padded"].with_(B=2, N=700))
    Q, K, V, mask = dev(inp.Q), dev(inp.K), dev(inp.V), dev(inp.key_mask)
    desc = flare.make_desc(Q, K)
    Y1, Z1, le1, ld1 = flare.forward(Q, K, V, mask, want_stats=True)
    ws = flare.alloc_workspace(desc, flare.OP_ENCODE)
    Z2, le2 = torch.empty_like(Z1), torch.empty_like(le1)
    flare.flare_encode(desc, Q, K, V, mask, Z2, le2, ws)
    Y2, ld2 = torch.empty_like(Y1), torch.empty_like(ld1)
    flare.flare_decode(desc, Q, K, Z2, Y2, ld2, flare.alloc_workspace(desc, flare.OP_DECODE))
    torch.cuda.synchronize()
    assert torch.equal(Z1, Z2) and torch.equal(le1, le2) and torch.equal(Y1, Y2) and torch.equal(ld1, ld2)
    # decode alone against the oracle's decode on the oracle's own Z
    ref = oracle_forward(oracle, inp)
    Zo = torch.from_numpy(ref["Z"]).float().cuda()
    flare.flare_decode(desc, Q, K, Zo, Y2, None)
    torch.cuda.synchronize()
    assert rel_err(to_np64(Y2), ref["Y"]) <= TOL["bf16"]
    # optional outputs may be NULL; Z may live in the workspace.  Without lse_enc the encode weights are single
    # bfloat16 values (with it, two halves, for a Z fit to be differentiated through), so Y agrees with the
    # oracle to the same bound but not bit for bit with Y1.
    wsf = flare.alloc_workspace(desc, flare.OP_FORWARD)
    Y3 = torch.empty_like(Y1)
    flare.flare_forward(desc, Q, K, V, mask, Y3, None, None, None, wsf)
    torch.cuda.synchronize()
    assert rel_err(to_np64(Y3), ref["Y"]) <= TOL["bf16"]
    assert rel_err(to_np64(Y3), to_np64(Y1)) <= TOL["bf16"]
    Y4 = torch.empty_like(Y1)
    flare.flare_forward(desc, Q, K, V, mask, Y4, None, None, None, wsf)
    torch.cuda.synchronize()
    assert torch.equal(Y3, Y4)


def test_error_paths_on_device():
    inp = workloads.make_random(1, 2, 64, 16, 16, dtype="bf16", seed=1)
    Q, K, V = dev(inp.Q), dev(inp.K), dev(inp.V)
    desc = flare.make_desc(Q, K)
    Y = torch.empty_like(K)
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(flare.FlareError) as e:
        flare.flare_forward(desc, Q, K, V, None, Y, None, None, None, small)
    assert e.value.status == flare.ERR_WORKSPACE_TOO_SMALL
    ws = flare.alloc_workspace(desc, flare.OP_FORWARD)
    import ctypes
    lib = flare.load()
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    rc = lib.flare_forward(ctypes.byref(desc), Q.data_ptr(), K.data_ptr() + 2, V.data_ptr(), None, Y.data_ptr(), None,
                           None, None, ws.data_ptr(), ws.numel(), st)
    assert rc == flare.ERR_INVALID_ARG
    rc = lib.flare_forward(ctypes.byref(desc), Q.data_ptr(), None, V.data_ptr(), None, Y.data_ptr(), None, None, None,
                           ws.data_ptr(), ws.numel(), st)
    assert rc == flare.ERR_INVALID_ARG
    torch.cuda.synchronize()


@pytest.mark.parametrize("k_std", [3.0, 8.0])
@STATS
def test_large_scores(oracle, k_std, stats, path):
    """Scores up to +-170 at scale 1: the running maximum is subtracted before every exponential; the fast forms find
    their inputs out of range and hand over to the exact ones."""
    inp = workloads.make_random(1, 2, 700, 128, 16, dtype="bf16", seed=7, k_std=k_std)
    got = gpu_forward(inp, canary=True, stats=stats, path=path)
    assert np.isfinite(got["Y"]).all() and np.isfinite(got["Z"]).all()
    assert_forward_close(got, oracle_forward(oracle, inp), "bf16", f"k_std={k_std}")


@pytest.mark.parametrize("w", [workloads.CONFIGS["mesh2d"].with_(B=2, N=3001), workloads.CONFIGS["padded"].with_(B=3, N=1000)],
                         ids=lambda w: w.name)
def test_forward_from_host_buffers(oracle, w):
    """flare_forward_host (the call behind the benchmark's end-to-end number): pinned host tensors in, a pinned host
    tensor out, the device tensors being staging buffers only; the host result against the oracle."""
    inp = workloads.make_inputs(w)
    hQ, hK, hV = inp.Q.pin_memory(), inp.K.pin_memory(), inp.V.pin_memory()
    hmask = None if inp.key_mask is None else inp.key_mask.pin_memory()
    hY = torch.full_like(inp.K, 777.0).pin_memory()
    desc = flare.make_desc(inp.Q, inp.K, w.scale)
    dQ, dK, dV, dY = (torch.full_like(t, 555.0, device="cuda") for t in (inp.Q, inp.K, inp.V, inp.K))
    dmask = None if hmask is None else torch.zeros_like(hmask, device="cuda")
    ws = flare.alloc_workspace(desc, flare.OP_FORWARD)
    flare.flare_forward_host(desc, hQ, hK, hV, hmask, hY, dQ, dK, dV, dmask, dY, ws)
    torch.cuda.synchronize()
    flare.flare_check(ws)
    ref = oracle_forward(oracle, inp, w.scale)
    from tests._util import assert_stored_close
    assert_stored_close(to_np64(hY), ref["Y"], w.dtype, f"{w.name} Y (host)")
    assert torch.equal(hY, dY.cpu()) and torch.equal(dK.cpu(), inp.K)


def test_bounded_wait_gives_up_and_reports(oracle):
    """A device-side wait that nothing completes runs out of its time budget, the kernel ends normally, flare_check
    reports FLARE_ERR_TIMEOUT, and the same workspace serves an ordinary forward afterwards."""
    inp = workloads.make_random(1, 2, 300, 32, 16, dtype="bf16", seed=2)
    Q, K, V = dev(inp.Q), dev(inp.K), dev(inp.V)
    desc = flare.make_desc(Q, K)
    ws = flare.alloc_workspace(desc, flare.OP_FORWARD)
    flare.flare_selftest_wait(ws, 1_000_000)                  # one millisecond
    torch.cuda.synchronize()
    with pytest.raises(flare.FlareError) as e:
        flare.flare_check(ws)
    assert e.value.status == flare.ERR_TIMEOUT
    Y = torch.empty_like(K)
    flare.flare_forward(desc, Q, K, V, None, Y, None, None, None, ws)
    torch.cuda.synchronize()
    flare.flare_check(ws)
    assert rel_err(to_np64(Y), oracle_forward(oracle, inp)["Y"]) <= TOL["bf16"]


@pytest.mark.parametrize("k_std,redo", [(0.5, False), (8.0, True)])
def test_fast_forms_hand_over_only_when_out_of_range(oracle, k_std, redo):
    """The flag words the fast forms raise (workspace header words 2 and 3: encode, decode) stay clear for ordinary
    inputs and go up for scores beyond the range the fast forms are valid for; the result is right in both cases."""
    inp = workloads.make_random(1, 2, 900, 128, 16, dtype="bf16", seed=11, k_std=k_std)
    Q, K, V = dev(inp.Q), dev(inp.K), dev(inp.V)
    desc = flare.make_desc(Q, K)
    ws = flare.alloc_workspace(desc, flare.OP_FORWARD)
    Y = torch.empty_like(K)
    flare.flare_set_path(flare.PATH_FAST)
    try:
        flare.flare_forward(desc, Q, K, V, None, Y, None, None, None, ws)
    finally:
        flare.flare_set_path(flare.PATH_AUTO)
    torch.cuda.synchronize()
    words = ws[:16].view(torch.int32).cpu()
    assert words[0] == 0 and bool(words[2]) == redo and bool(words[3]) == redo
    from tests._util import assert_stored_close
    assert_stored_close(to_np64(Y), oracle_forward(oracle, inp)["Y"], "bf16", f"fast forms, k_std={k_std}")


def test_tiny_scale_keeps_padding_out(oracle):
    """A scale so small that every score is practically zero, with a partial last tile: the tokens beyond N must still
    get weight exactly 0 (the form of the encode kernel that marks padding by a huge negative score is not taken then)."""
    inp = workloads.make_random(1, 2, 300, 256, 16, dtype="bf16", seed=13)
    got, ref = gpu_forward(inp, scale=1e-24, canary=True), oracle_forward(oracle, inp, scale=1e-24)
    assert_forward_close(got, ref, "bf16", "tiny scale")


def test_microbenchmarks_are_in_range():
    """The library's instruction-level measurements (the figures the kernel design quotes) on this GPU: the special-function
    unit alone delivers about 15 exponentials per clock per SM in the softmax loop, half of them on the FMA pipe about 24;
    a unit's tensor-core instructions hold the issuing thread for a few hundred cycles."""
    sfu_max = flare.flare_microbench(0, 5000)
    sfu = flare.flare_microbench(1, 5000)
    both = flare.flare_microbench(2, 5000)
    assert 11.0 <= sfu_max <= 16.5 and 11.0 <= sfu <= 16.5, (sfu_max, sfu)
    assert 18.0 <= both <= 32.0 and both > 1.2 * sfu, (both, sfu)
    issue, flip = flare.flare_microbench(3, 128), flare.flare_microbench(4, 128)
    assert 100 <= issue <= 1200 and 50 <= flip <= 1200, (issue, flip)
