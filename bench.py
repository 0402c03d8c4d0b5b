#!/usr/bin/env python
"""Benchmark of the FLARE token mixer on B200: one step = one flare_forward over one batch of synthetic input.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is whole-job tokens/s with inputs resident in HBM; `e2e` is the same
metric through flare_forward_host with pinned host buffers (host<->device copies inside the timed region);
`roofline` describes the slower of the two main kernels (encode, decode) against the measured peak;
`cpu_baseline` is the CPU oracle timed on a bounded sample of the same workload.  With N > 1 every rank runs
the same workload on its own batch (weak scaling, no collective on the data path).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2508_12594_b200 import workloads  # noqa: E402

METRIC = "FLARE fwd tokens/sec at N=1M on 1 B200"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes (read + write) of one launch of each main kernel on the full mesh3d_1m workload, from the ncu captures
# summarised under profiles/ (taken on a 262,144-token slice and scaled by 4: traffic is proportional to N).
# Valid for the kernels as profiled; set to None when a kernel changes until the capture is redone.
NCU_TRAFFIC = {("mesh3d_1m", "encode"): 4 * (134.328320e6 + 5.408256e6),     # profiles/encode_tc_fast_mesh3d_N262144.md
               ("mesh3d_1m", "decode"): 4 * (67.366912e6 + 26.701568e6)}     # profiles/decode_stream_mesh3d_N262144.md


def get_workload(name: str) -> workloads.Workload:
    if name in workloads.CONFIGS:
        return workloads.CONFIGS[name]
    if name.startswith("sweep_N"):
        n, m = name[len("sweep_N"):].split("_M")
        return workloads.sweep_point(int(n), int(m))
    raise SystemExit(f"unknown workload {name}")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(w: workloads.Workload, inp, sample_tokens: int):
    """Time the CPU oracle (as it stands) on the first `sample_tokens` tokens of every batch item."""
    from oracle import flare_oracle
    flare_oracle.build()
    n = min(w.N, sample_tokens)
    Q = inp.Q.double().numpy()
    K = inp.K[:, :n].double().numpy()
    V = inp.V[:, :n].double().numpy()
    mask = None if inp.key_mask is None else inp.key_mask[:, :n].numpy()
    t0 = time.perf_counter()
    flare_oracle.forward(Q, K, V, key_mask=mask, scale=w.scale)
    dt = time.perf_counter() - t0
    return w.B * n / dt, dt, n, flare_oracle.max_threads()


def max_over_ranks(ms: float, dist, device) -> float:
    """The slowest rank's time (every multi-GPU number is the maximum over ranks); `dist` is None on one rank."""
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_workload(w, rank: int):
    """Replicas: every rank draws its own batch from the same recipe (weak scaling), seed offset by the rank."""
    return w.with_(seed=w.seed + 1000 * rank)


def whole_job_value(w, world: int, ms_step: float) -> float:
    """Tokens per second over all replicas: every rank processes w.tokens per step."""
    return world * w.tokens / (ms_step / 1e3)


def self_launch(n: int):
    """`python bench.py --gpus N` outside a launcher: start the N replicas (one process per GPU) and relay rank 0's line."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.run(cmd).returncode)


def run_micro():
    """The instruction-level figures the kernels' design rests on, re-measured through flare_microbench."""
    from paper_2508_12594_b200 import flare
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    names = ["exp_per_clk_per_sm_running_max_sfu", "exp_per_clk_per_sm_no_max_sfu", "exp_per_clk_per_sm_no_max_sfu_plus_fma",
             "mma_unit_issue_cycles", "mma_commit_to_barrier_cycles"]
    out = {}
    for which, name in enumerate(names):
        flare.flare_microbench(which, 2000 if which < 3 else 64)                      # warm-up
        out[name] = flare.flare_microbench(which, 20000 if which < 3 else 256)
    print(json.dumps({"micro": out}))


def run_spectral(args, w):
    """Algorithm 1 (spectral appendix) on the GPU for the workload's shape: the forward that yields the two log-sum-exp
    arrays, the Gram matrix J J^T (one more pass over the tokens) and the M x M eigen-solver, each timed with CUDA events."""
    from paper_2508_12594_b200 import flare
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    inp = workloads.make_inputs(w)
    Q, K, V = inp.Q.cuda(), inp.K.cuda(), inp.V.cuda()
    desc = flare.make_desc(Q, K, 1.0)
    B, H, N, M, D = desc.B, desc.H, desc.N, desc.M, desc.D
    ws, wss = flare.alloc_workspace(desc, flare.OP_FORWARD), flare.alloc_workspace(desc, flare.OP_SPECTRAL)
    Y = torch.empty_like(K)
    Z = torch.empty(B, H, M, D, dtype=torch.float32, device="cuda")
    le = torch.empty(B, H, M, dtype=torch.float32, device="cuda")
    ld = torch.empty(B, N, H, dtype=torch.float32, device="cuda")
    G = torch.empty(B, H, M, M, dtype=torch.float32, device="cuda")
    Gc, ev = torch.empty_like(G), torch.empty(B, H, M, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()

    def timed(fn, steps):
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(steps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / steps

    steps = min(args.steps, 50)
    t_fwd = timed(lambda: flare.flare_forward(desc, Q, K, V, None, Y, Z, le, ld, ws, stream), steps)
    t_gram = timed(lambda: flare.flare_spectral_gram(desc, Q, K, le, ld, G, wss, stream), steps)

    def eig():
        Gc.copy_(G)
        flare.flare_spectral_eig(Gc, ev, None, 0, stream)
    t_eig = timed(eig, min(steps, 10))
    flare.flare_check(wss)
    top = float(ev[..., 0].mean())
    peaks, kind = load_peaks()
    flop = 2.0 * B * H * N * M * M                             # J J^T; the scores add 2 B H N M D
    print(json.dumps({"spectral": {
        "workload": w.name, "B": B, "H": H, "N": N, "M": M, "D": D, "dtype": w.dtype,
        "forward_with_statistics_ms": t_fwd, "gram_ms": t_gram, "eig_ms": t_eig,
        "gram_tflops": flop / (t_gram * 1e-3) / 1e12, "gram_frac_of_bf16_peak": flop / (t_gram * 1e-3) / 1e12 / peaks["bf16_tflops"],
        "gram_bytes_gbs": (B * N * H * D * (2 if w.dtype != "f32" else 4) + 4.0 * B * N * H) / (t_gram * 1e-3) / 1e9,
        "peak_kind": kind, "tokens_per_s": B * N / ((t_fwd + t_gram + t_eig) * 1e-3),
        "largest_eigenvalue_mean": top}}))


def run_reference(args, w):
    """The reference arm: the oracle on the host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = workloads.make_inputs(w.with_(N=min(w.N, args.ref_tokens)))
    times, cores, n = [], 1, 0
    for i in range(args.warmup + args.steps):
        v, dt, n, cores = oracle_sample(w.with_(N=inp.K.shape[1]), inp, args.ref_tokens)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = w.B * n / (ms / 1e3)
    sample = f"first {n} tokens of each of {w.B} batch item(s), all {w.H} heads, M={w.M}, D={w.D}"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "N": w.N, "M": w.M, "D": w.D, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="mesh3d_1m")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-tokens", type=int, default=524288, help="tokens per batch item in the oracle sample")
    ap.add_argument("--ref-tokens", type=int, default=65536)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--tokens", type=int, default=0, help="override N (a smaller case of the same workload)")
    ap.add_argument("--no-backward", action="store_true", help="skip the forward+backward leg")
    ap.add_argument("--micro", action="store_true", help="print the library's instruction-level measurements and exit")
    ap.add_argument("--spectral", action="store_true",
                    help="time the spectral analysis (Algorithm 1: forward statistics, Gram matrix, eigen-solver) on the workload and exit")
    args = ap.parse_args()
    w = get_workload(args.workload)
    if args.tokens > 0:
        w = w.with_(N=args.tokens, name=f"{w.name}@N={args.tokens}")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return self_launch(args.gpus)
    if args.impl == "reference":
        return run_reference(args, w)
    if args.micro:
        return run_micro()
    if args.spectral:
        return run_spectral(args, w)
    if args.warmup < 3:
        args.warmup = 3

    from paper_2508_12594_b200 import flare

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # every rank draws its own batch (weak scaling): same recipe, rank-dependent seed
    wr = rank_workload(w, rank)
    inp = workloads.make_inputs(wr)
    Q, K, V = inp.Q.cuda(), inp.K.cuda(), inp.V.cuda()
    mask = None if inp.key_mask is None else inp.key_mask.cuda()
    desc = flare.make_desc(Q, K, w.scale)
    ws = flare.alloc_workspace(desc, flare.OP_FORWARD)
    Y = torch.empty_like(K)
    Z = torch.empty(w.B, w.H, w.M, w.D, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()
    e = 4 if w.dtype == "f32" else 2
    tensor_bytes = w.B * w.N * w.H * w.D * e
    l2_note = "inputs larger than L2" if 3 * tensor_bytes > 2 * 126e6 else "L2 flushed between steps"
    flush = None if 3 * tensor_bytes > 2 * 126e6 else torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def step():
        if flush is not None:
            flush.zero_()
        flare.flare_forward(desc, Q, K, V, mask, Y, Z, None, None, ws, stream)

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    if flush is None:
        ev[0].record(stream)
        for _ in range(args.steps):
            step()
        ev[1].record(stream)
        barrier()
        ms_total = ev[0].elapsed_time(ev[1])
    else:  # time each step on its own so the flush stays outside
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in evs:
            flush.zero_()
            a.record(stream)
            flare.flare_forward(desc, Q, K, V, mask, Y, Z, None, None, ws, stream)
            b.record(stream)
        barrier()
        ms_total = sum(a.elapsed_time(b) for a, b in evs)
    # per-stage durations (encode incl. merge, decode), same inputs, events on the launching stream
    wse = flare.alloc_workspace(desc, flare.OP_ENCODE)
    wsd = flare.alloc_workspace(desc, flare.OP_DECODE)
    stage_ms = {}
    for name, fn in (("encode", lambda: flare.flare_encode(desc, Q, K, V, mask, Z, None, wse, stream)),
                     ("decode", lambda: flare.flare_decode(desc, Q, K, Z, Y, None, wsd, stream))):
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in pairs:
            if flush is not None:
                flush.zero_()
            a.record(stream); fn(); b.record(stream)
        torch.cuda.synchronize()
        stage_ms[name] = sum(a.elapsed_time(b) for a, b in pairs) / len(pairs)
    # forward + backward of the same batch (reported beside the forward-only metric): dY is seeded noise
    fwd_bwd = None
    if not args.no_backward:
        gen = torch.Generator(device="cuda").manual_seed(wr.seed + 7)
        dYt = torch.randn(K.shape, generator=gen, device="cuda", dtype=torch.float32).to(K.dtype)
        le = torch.empty(w.B, w.H, w.M, dtype=torch.float32, device="cuda")
        ld = torch.empty(w.B, w.N, w.H, dtype=torch.float32, device="cuda")
        wsb = flare.alloc_workspace(desc, flare.OP_BACKWARD)
        dQ = torch.empty(w.H, w.M, w.D, dtype=torch.float32, device="cuda")
        dK, dV = torch.empty_like(K), torch.empty_like(V)

        def both():
            if flush is not None:
                flush.zero_()
            flare.flare_forward(desc, Q, K, V, mask, Y, Z, le, ld, ws, stream)
            flare.flare_backward(desc, Q, K, V, mask, Y, dYt, Z, le, ld, dQ, dK, dV, wsb, stream)

        nb = max(1, min(args.steps, 50))
        for _ in range(3):
            both()
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(nb)]
        for a, b in pairs:
            if flush is not None:
                flush.zero_()
            a.record(stream)
            flare.flare_forward(desc, Q, K, V, mask, Y, Z, le, ld, ws, stream)
            flare.flare_backward(desc, Q, K, V, mask, Y, dYt, Z, le, ld, dQ, dK, dV, wsb, stream)
            b.record(stream)
        torch.cuda.synchronize()
        flare.flare_check(wsb)
        fb_ms = sum(a.elapsed_time(b) for a, b in pairs) / nb
        fwd_bwd = {"ms_per_step": fb_ms, "value": w.tokens / (fb_ms / 1e3), "unit": "tokens/s", "steps": nb,
                   "gpu_launches_per_step": flare.flare_launch_count(desc, flare.OP_FORWARD) +
                   flare.flare_launch_count(desc, flare.OP_BACKWARD),
                   "note": "per GPU; forward with saved statistics, then backward"}
        del dYt, dK, dV, wsb
    clocks = sampler.stop() if rank == 0 else None
    flare.flare_check(ws)

    ms_step = max_over_ranks(ms_total, dist, "cuda") / args.steps
    value = whole_job_value(w, world, ms_step)

    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, w, inp, flare, desc, ws, stream, barrier, dist, world, Q, K, V, mask, tensor_bytes, e)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    launches = args.steps * flare.flare_launch_count(desc, flare.OP_FORWARD)
    finish(args, w, inp, world, ms_step, value, stage_ms, clocks, e2e, tensor_bytes, e, l2_note, dist, fwd_bwd, launches)


def run_e2e(args, w, inp, flare, desc, ws, stream, barrier, dist, world, Q, K, V, mask, tensor_bytes, e):
    """End to end: pinned host buffers in, pinned host buffer out, through flare_forward_host."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    hQ, hK, hV = inp.Q.pin_memory(), inp.K.pin_memory(), inp.V.pin_memory()
    hmask = None if inp.key_mask is None else inp.key_mask.pin_memory()
    hY = torch.empty_like(inp.K).pin_memory()
    dQ, dK, dV, dY = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V), torch.empty_like(K)
    dmask = None if mask is None else torch.empty_like(mask)
    for _ in range(2):
        flare.flare_forward_host(desc, hQ, hK, hV, hmask, hY, dQ, dK, dV, dmask, dY, ws, stream)
    barrier()
    ev[0].record(stream)
    for _ in range(args.e2e_steps):
        flare.flare_forward_host(desc, hQ, hK, hV, hmask, hY, dQ, dK, dV, dmask, dY, ws, stream)
    ev[1].record(stream)
    barrier()
    e2e_ms = max_over_ranks(ev[0].elapsed_time(ev[1]), dist, "cuda") / args.e2e_steps
    h2d = 2 * tensor_bytes + w.H * w.M * w.D * e + (0 if mask is None else w.B * w.N)
    return {"value": world * w.tokens / (e2e_ms / 1e3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": tensor_bytes, "ms_per_step": e2e_ms}


def finish(args, w, inp, world, ms_step, value, stage_ms, clocks, e2e, tensor_bytes, e, l2_note, dist, fwd_bwd=None,
           launches=0):
    peaks, peak_kind = load_peaks()
    # Roofline of the slower main kernel.  Per stage and head the contraction work is 4*N*M*D FLOP (scores and
    # value contraction); the bytes are K and V read (encode) or K read and Y written (decode), plus Q_lat.
    flops_stage = 4.0 * w.B * w.H * w.N * w.M * w.D
    bytes_stage = 2.0 * tensor_bytes + w.H * w.M * w.D * e
    dom = max(stage_ms, key=stage_ms.get)
    t_dom = stage_ms[dom] / 1e3
    tensor_peak = peaks["bf16_tflops"] * (0.5 if w.dtype == "f32" else 1.0)
    t_tensor, t_hbm = flops_stage / (tensor_peak * 1e12), bytes_stage / (peaks["hbm_gbs"] * 1e9)
    if t_tensor >= t_hbm:
        roof = {"bound": "tensor", "achieved": flops_stage / t_dom / 1e12, "peak": tensor_peak, "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": bytes_stage / t_dom / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    base_name = w.name.split("@")[0]
    traffic = NCU_TRAFFIC.get((base_name, dom))
    if traffic is not None:
        traffic *= w.N / workloads.CONFIGS[base_name].N       # a --tokens slice of the profiled workload
    sm_clock = (clocks or {}).get("sm_mhz") or 1965.0
    roof.update({"traffic": traffic, "kernel": dom, "kernel_ms": stage_ms[dom], "peak_kind": peak_kind,
                 "stage_ms": stage_ms, "exp_per_s": w.B * w.H * w.N * w.M / t_dom,
                 "exp_per_clk_per_sm": w.B * w.H * w.N * w.M / t_dom / 148 / (sm_clock * 1e6)})
    # whole forward against the stated roofline: slower of 8*B*H*N*M*D FLOP at tensor peak and K, V, Q_lat, Y once
    fwd_t = max(2 * flops_stage / (tensor_peak * 1e12), (3 * tensor_bytes + w.H * w.M * w.D * e) / (peaks["hbm_gbs"] * 1e9))
    roof["forward_frac_of_stated_roofline"] = fwd_t / (ms_step / 1e3)

    out = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "N": w.N, "M": w.M, "D": w.D, "scale": w.scale,
                   "l2": l2_note, "parallelism": f"replicas x{world}"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roof,
    }
    if fwd_bwd is not None:
        out["fwd_bwd"] = fwd_bwd
    if not args.no_cpu_baseline:
        v, dt, n, cores = oracle_sample(w, inp, args.cpu_tokens)
        out["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                               "sample": f"first {n} tokens of each of {w.B} batch item(s), all heads, {dt:.1f} s"}
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
