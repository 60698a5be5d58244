#!/usr/bin/env python
"""Benchmark of the LoRAct hot path: one step = loract_compress + loract_weight_grad on one batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line.  `value` is GB/s of X (bytes of the activation matrix compressed and consumed
per second, whole job).  With N > 1 every rank runs its own batch -- data-parallel fine-tuning needs no
collective on this path -- and the time is the max over ranks.  Started without a launcher
(`python bench.py --gpus N`), the script starts its N ranks itself through torch.distributed.run.
`--impl reference` times the float64 CPU oracle on the same workload instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "compress+weight-grad GB/s of X"
DEFAULT_WORKLOAD = "llama7b_block"
MIN_TIMED_SECONDS = 1.0      # the K-step block is repeated until the timed region has run this long


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def dram_traffic(kernel: str, workload: str):
    """DRAM bytes per launch of `kernel` on `workload` from the kept profiler summaries
    (profiles/dram_traffic.md: one table row per captured kernel and workload), or None if none is kept."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.md")
    if not os.path.exists(path):
        return None
    for line in open(path):
        f = [x.strip() for x in line.strip().strip("|").split("|")]
        if len(f) >= 3 and f[0] == kernel and f[1] == workload:
            try:
                return float(f[2])
            except ValueError:
                return None
    return None


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); smax = float(f[1])
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax,
                "reasons": sorted(reasons), "samples": len(sm)}


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def oracle_step(Xd, Gd, w):
    """One pass of the hot path in the float64 oracle: Algorithm 1 + the factor-form weight gradient."""
    from oracle import loract_oracle as orc
    U, V, _ = orc.decompose(Xd, w.rank, seed=w.seed)
    return orc.weight_grad(U, V, Gd)


def time_oracle(Xd, Gd, w, max_seconds: float, max_reps: int):
    """The oracle as it stands on the whole configuration: at least one step, then more while the budget
    lasts.  Returns (seconds per step, repetitions)."""
    t0 = time.perf_counter()
    reps = 0
    while reps < 1 or (time.perf_counter() - t0 < max_seconds and reps < max_reps):
        oracle_step(Xd, Gd, w)
        reps += 1
    return (time.perf_counter() - t0) / reps, reps


def run_reference(args):
    """--impl reference: the float64 oracle on the host cores, every step the whole workload (all rows)."""
    from paper_2509_23472_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.get_workload(args.workload)
    inp = synth.make_inputs(w)
    Xd, Gd = inp["X"].double().numpy(), inp["G"].double().numpy()
    # a few minutes at most: the step count asked for is capped by a time budget, the rows never are
    budget = 120.0
    warm_done, tw = 0, time.perf_counter()
    while warm_done < args.warmup and (warm_done < 1 or time.perf_counter() - tw < 30.0):
        oracle_step(Xd, Gd, w)
        warm_done += 1
    t0 = time.perf_counter()
    done = 0
    while done < args.steps and (done < 1 or time.perf_counter() - t0 < budget):
        oracle_step(Xd, Gd, w)
        done += 1
    dt = (time.perf_counter() - t0) / done
    gbs = w.n_tokens * w.d * w.elem_bytes / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": done, "warmup": warm_done, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "n_tokens": w.n_tokens, "d": w.d, "rank": w.rank, "g": w.g},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cpu_threads(), "kind": "oracle",
                         "sample": f"all {w.n_tokens} token rows, {done} steps (of {args.steps} asked for, "
                                   f"{budget:.0f} s budget), float64 numpy"},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "tokens_per_s": w.n_tokens / dt,
    }
    print(json.dumps(line))


def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n: int, argv) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks through torch.distributed.run."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def run_plumbing_only(args):
    """The rank plumbing of the benchmark without its GPU work (for world-size-2 tests on CPU process groups):
    every rank takes its batch description, the ranks meet at the two barriers, a per-rank time becomes the
    whole-job figure through the same functions the GPU run uses, rank 0 prints the line."""
    import torch
    import torch.distributed as dist
    from paper_2509_23472_b200 import dp, synth
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    w = synth.get_workload(args.workload)
    w_rank = dp.rank_workload(w, rank)
    if world > 1:
        dist.barrier()
    fake_ms = 1.0 + rank            # stands in for a rank's measured time: the slowest rank must win
    if world > 1:
        dist.barrier()
    (ms,) = dp.max_over_ranks([fake_ms], dist if world > 1 else None)
    if rank == 0:
        print(json.dumps({"plumbing_only": True, "n_gpus": world, "ms_per_step": ms,
                          "value": dp.whole_job_gbs(world, w.n_tokens * w.d * w.elem_bytes, ms),
                          "seeds": [dp.rank_workload(w, r).seed for r in range(world)],
                          "call_ids": [dp.rank_call_id(r) for r in range(world)], "my_seed": w_rank.seed}))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="loract", choices=["loract", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="repeat the block of --steps steps until the timed region has run this long (0: one block; "
                         "for runs under a profiler)")
    ap.add_argument("--plumbing-only", action="store_true",
                    help="rank start-up, barriers and the max over ranks only, on a gloo group, no GPU work")
    ap.add_argument("--kernel-only", nargs="?", const="pass1", default=None,
                    choices=["pass1", "pass2", "reconstruct"],
                    help="run only one kernel a few times (pass 1 or pass 2 of Algorithm 1, or Reconstruct): the "
                         "small case for profiler captures")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.plumbing_only:
        run_plumbing_only(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "loract" else args.warmup
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import __graft_entry__ as entry
    from paper_2509_23472_b200 import binding as B
    from paper_2509_23472_b200 import dp, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        entry.build()
    if dist is not None:
        dist.barrier()
    B.lib()

    w = synth.get_workload(args.workload)
    # data-parallel replicas: every rank draws its own batch and samples its own rows
    w_rank = dp.rank_workload(w, rank)
    inp = synth.make_inputs(w_rank, device=dev)
    X, G = inp["X"], inp["G"]
    N, d, r, g = w.n_tokens, w.d, w.rank, w.g
    es = w.elem_bytes
    desc = B.make_desc(X, r, seed=w_rank.seed, call_id=dp.rank_call_id(rank))
    ws = B.alloc_workspace(desc, dev)
    U = torch.empty(N, r, dtype=X.dtype, device=dev)
    V = torch.empty(r, d, dtype=X.dtype, device=dev)
    idx = torch.empty(r, dtype=torch.int32, device=dev)
    dW = torch.empty(d, g, dtype=torch.float32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def step(Xin, Gin):
        B.compress(Xin, r, ws=ws, out=(U, V, idx), desc=desc)
        B.weight_grad(U, V, Gin, dW=dW, ws=ws)

    # Three copies of the inputs take turns, so a step's input was last touched two steps (and more than
    # twice the L2 capacity of other traffic) ago: the inputs are larger than L2 and never resident.
    n_copies = 3
    Xs = [X] + [X.clone() for _ in range(n_copies - 1)]
    Gs = [G] + [G.clone() for _ in range(n_copies - 1)]

    def timed(fn, steps, flush_l2=False):
        """Per-step device times (CUDA events on the launching stream).  fn takes the step number.  With
        flush_l2 a 256 MiB memset runs before every step, outside the events."""
        evs = []
        for i in range(steps):
            if flush_l2:
                flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn(i)
            e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    if args.kernel_only:
        Om = torch.randn(r, d, device=dev).to(X.dtype)
        Uk = torch.randn(N, r, device=dev).to(X.dtype)
        Xt = torch.empty_like(X)
        for _ in range(args.warmup + args.steps):
            flush.zero_()
            if args.kernel_only == "pass1":
                B.debug_gemm([X], [Om], N, r, d, False, False, out_mode=B.OUT_SPLIT, engine=1)
            elif args.kernel_only == "pass2":
                B.debug_project(desc, Uk, X, V, ws)
            else:
                B.reconstruct(Uk, Om, out=Xt)
        torch.cuda.synchronize()
        print(json.dumps({"kernel_only": args.kernel_only, "launches": args.warmup + args.steps}))
        return

    for _ in range(args.warmup):
        step(X, G)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = B.kernel_launch_count()
    torch.cuda.synchronize()
    # The timed region: blocks of exactly `steps` steps, each step between its own pair of events, repeated
    # until the region has run for --min-seconds (default 1 s), so that the clock record has samples under load.
    times = []
    repeats = 0
    t_wall = time.perf_counter()
    while True:
        times += timed(lambda i: step(Xs[i % n_copies], Gs[i % n_copies]), args.steps)
        repeats += 1
        enough = time.perf_counter() - t_wall >= args.min_seconds or repeats >= 4000
        if dist is not None:   # every rank runs the same number of blocks: rank 0 decides
            flag = torch.tensor([1 if enough else 0], device=dev)
            dist.broadcast(flag, 0)
            enough = bool(flag.item())
        if enough:
            break
    torch.cuda.synchronize()
    launches = B.kernel_launch_count() - launches0       # every kernel of the library inside the timed region
    if dist is not None:
        dist.barrier()
    total_ms = sum(times)
    n_timed = len(times)
    flushed = timed(lambda i: step(Xs[i % n_copies], Gs[i % n_copies]), max(3, args.steps // 2), flush_l2=True)

    # ---- the device status word of the compression itself (loract_weight_grad re-uses the workspace and
    # clears the word at its start, so it is read between the two calls here)
    B.compress(Xs[0], r, ws=ws, out=(U, V, idx), desc=desc)
    status_compress = B.read_device_status(ws)
    # what the device decided about the second orthonormalisation round, and the estimate it decided on
    second_round, orth_estimate, orth_rounds = B.round_gate_words(ws) if w.dtype == "bf16" else (1, float("nan"), 2)
    B.weight_grad(U, V, Gs[0], dW=dW, ws=ws)
    status_wgrad = B.read_device_status(ws)

    # ---- where the time goes: one more step with an event behind every kernel (outside the timed region)
    B.debug_trace_begin(dev)
    step(Xs[1], Gs[1])
    stages = B.debug_trace_end(dev)

    # ---- two independent batches in flight (context only, not `value`): in fine-tuning the compression of one
    # layer's activation does not wait for the next layer's, so a trainer can keep two calls running on two
    # streams; the latency-bound small-block kernels (8 SMs) then overlap the other call's streaming passes.
    streams = [torch.cuda.Stream(device=dev) for _ in range(2)]
    lanes = []
    for _ in range(2):
        lanes.append(dict(ws=B.alloc_workspace(desc, dev), U=torch.empty_like(U), V=torch.empty_like(V),
                          idx=torch.empty_like(idx), dW=torch.empty_like(dW)))

    def step_on(lane, Xin, Gin):
        B.compress(Xin, r, ws=lane["ws"], out=(lane["U"], lane["V"], lane["idx"]), desc=desc)
        B.weight_grad(lane["U"], lane["V"], Gin, dW=lane["dW"], ws=lane["ws"])

    def two_stream_run(steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        cur = torch.cuda.current_stream(dev)
        e0.record(cur)
        for st in streams:
            st.wait_event(e0)
        for i in range(steps):
            with torch.cuda.stream(streams[i % 2]):
                step_on(lanes[i % 2], Xs[i % n_copies], Gs[i % n_copies])
        for st in streams:
            ev = torch.cuda.Event()
            ev.record(st)
            cur.wait_event(ev)
        e1.record(cur)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    two_stream_run(4)
    two_ms = two_stream_run(args.steps) / args.steps

    # ---- end to end: inputs start in pinned host memory, the gradient is read back to the host
    Xh, Gh = X.cpu().pin_memory(), G.cpu().pin_memory()
    Xd2, Gd2 = torch.empty_like(X), torch.empty_like(G)
    dWh = torch.empty(d, g, dtype=torch.float32).pin_memory()

    def step_e2e(_i=0):
        Xd2.copy_(Xh, non_blocking=True)
        Gd2.copy_(Gh, non_blocking=True)
        step(Xd2, Gd2)
        dWh.copy_(dW, non_blocking=True)

    for _ in range(2):
        step_e2e()
    torch.cuda.synchronize()
    e2e_steps = max(3, args.steps // 3)
    e2e_serial_ms = sum(timed(step_e2e, e2e_steps))

    # The same steps as a user who feeds the GPU from the host would run them: two device buffers, the copy of
    # step i + 1's inputs on a second stream while step i computes.  Every step's host-to-device copy and its
    # device-to-host read are inside the timed region; the time is from the first copy to the last read.
    Xd3, Gd3 = torch.empty_like(X), torch.empty_like(G)
    bufs = [(Xd2, Gd2), (Xd3, Gd3)]
    copy_stream = torch.cuda.Stream(device=dev)
    cur = torch.cuda.current_stream(dev)

    def e2e_pipelined(n_steps):
        ready = [torch.cuda.Event() for _ in range(n_steps)]
        done = [torch.cuda.Event() for _ in range(n_steps)]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(cur)
        copy_stream.wait_event(e0)
        for i in range(n_steps):
            xb, gb = bufs[i % 2]
            with torch.cuda.stream(copy_stream):
                if i >= 2:
                    copy_stream.wait_event(done[i - 2])      # the buffer's previous step has finished with it
                xb.copy_(Xh, non_blocking=True)
                gb.copy_(Gh, non_blocking=True)
                ready[i].record(copy_stream)
            cur.wait_event(ready[i])
            step(xb, gb)
            dWh.copy_(dW, non_blocking=True)
            done[i].record(cur)
        e1.record(cur)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    e2e_pipelined(3)
    e2e_ms = e2e_pipelined(e2e_steps)
    clocks = sampler.stop()

    # ---- the three streaming kernels alone, each in the launch shape the step uses: pass 1 (Y = X Omega^T),
    # pass 2 (V = U^T X) and Reconstruct (X~ = U V).  Back-to-back launches between one pair of events (the
    # copies of X take turns), so that the launch latency of a single call is not counted as kernel time.
    iso = {}
    if X.dtype == torch.bfloat16:
        Om = torch.randn(r, d, device=dev).to(X.dtype)
        Yh = torch.empty(N, r, dtype=X.dtype, device=dev)
        Yl = torch.empty_like(Yh)
        Vt = torch.empty_like(V)
        Xt = torch.empty_like(X)
        group = 2 * n_copies

        def iso_time(one):
            for j in range(3):
                one(j)

            def grp(_i=0):
                for j in range(group):
                    one(j)
            return statistics.mean(timed(grp, 6)) / group

        iso["pass1"] = iso_time(lambda j: B.debug_gemm([Xs[j % n_copies]], [Om], N, r, d, False, False,
                                                       out_mode=B.OUT_SPLIT, engine=1, out=(Yh, Yl)))
        iso["pass2"] = iso_time(lambda j: B.debug_project(desc, U, Xs[j % n_copies], Vt, ws))
        iso["reconstruct"] = iso_time(lambda j: B.reconstruct(U, V, out=Xt))
        del Xt

    total_ms, e2e_ms = dp.max_over_ranks([total_ms, e2e_ms], dist, dev)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    ms_per_step = total_ms / n_timed
    x_bytes = N * d * es
    value = dp.whole_job_gbs(world, x_bytes, ms_per_step)
    e2e_value = dp.whole_job_gbs(world, x_bytes, e2e_ms / e2e_steps)
    # Algorithmic bytes per launch.  Pass 1: X read once, the test matrix read once, Y written once as a bf16
    # pair.  Pass 2: X and U read once, V written once.  Reconstruct: U and V read once, X~ written once.
    alg = {"pass1": N * d * es + r * d * es + N * r * 4,
           "pass2": N * d * es + N * r * es + r * d * es,
           "reconstruct": N * d * es + N * r * es + r * d * es}
    names = {"pass1": "pass 1, Y = X Omega^T (gemm_tc_pair_kernel<K-major,K-major>)",
             "pass2": "pass 2, V = U^T X (as loract_compress runs it)",
             "reconstruct": "Reconstruct, X~ = U V (gemm_tc_stream_kernel)"}
    rooflines = []
    for k in ("pass1", "pass2", "reconstruct"):
        if k not in iso:
            continue
        ms = iso[k]
        achieved = alg[k] / (ms * 1e-3) / 1e9
        rooflines.append({"kernel": names[k], "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"],
                          "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
                          "traffic": dram_traffic(k, w.name), "ms_per_launch": ms, "algorithmic_bytes": alg[k],
                          "tflops": 2.0 * N * d * r / (ms * 1e-3) / 1e12})
    # whole-step floor: X once + factors + gathered rows (strict), against measured HBM bandwidth; 4Ndr flops
    # against the measured bf16 peak (burst figure); whichever is slower
    strict_bytes = x_bytes + (N * r + 2 * r * d) * es + (N * r + N * g + r * d) * es + 4 * d * g
    step_floor_ms = max(strict_bytes / (peaks["hbm_gbs"] * 1e9), 4.0 * N * d * r / (peaks["bf16_tflops"] * 1e12)) * 1e3

    cpu = None
    if not args.no_cpu_baseline:
        # the oracle on the whole configuration (all rows): the repetitions are capped, never the rows
        Xc, Gc = X.double().cpu().numpy(), G.double().cpu().numpy()
        dt, reps = time_oracle(Xc, Gc, w_rank, max_seconds=15.0, max_reps=20)
        cpu = {"value": N * d * es / dt / 1e9, "unit": "GB/s", "cores": cpu_threads(), "kind": "oracle",
               "sample": f"all {N} token rows, {reps} repetitions, float64 numpy", "ms_per_step": dt * 1e3}

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "n_tokens": N, "d": d, "rank": r, "g": g,
                   "l2": "inputs larger than L2: three copies of X and G (402 MB of X against 126 MB of L2) take "
                         "turns, no explicit flush; ms_per_step_l2_flushed has a 256 MiB memset before every step",
                   "step": "loract_compress + one loract_weight_grad (all consumers' G concatenated)",
                   "timed_region": f"{repeats} blocks of {args.steps} steps back to back, {total_ms / 1e3:.2f} s in all",
                   "parallelism": f"dp{world} (independent batches, no collective)"},
        "tokens_per_s": world * N / (ms_per_step * 1e-3),
        "step_roofline_frac": step_floor_ms / ms_per_step,
        "step_floor_ms": step_floor_ms,
        "repeats": repeats, "timed_steps": n_timed,
        "ms_min": min(times), "ms_median": statistics.median(times), "ms_mean": ms_per_step,
        "ms_per_step_l2_flushed": sum(flushed) / len(flushed),
        "stages_us": [[name, round(us, 1)] for name, us in stages],
        "two_streams": {"ms_per_step": two_ms, "value": world * x_bytes / (two_ms * 1e-3) / 1e9, "unit": "GB/s",
                        "note": "two independent batches in flight on two streams; context, not the headline"},
        "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": X.numel() * es + G.numel() * es,
                "d2h_bytes_per_step": dW.numel() * 4, "ms_per_step": e2e_ms / e2e_steps,
                "ms_per_step_one_stream": e2e_serial_ms / e2e_steps,
                "how": "pinned host inputs copied on a second stream into two device buffers while the previous step computes; every step's copies are inside the timed region"},
        "gpu_launches": int(launches), "gpu_launches_per_step": int(launches) // n_timed, "device_status": status_compress, "device_status_weight_grad": status_wgrad,
        "orthonormalisation": {"rounds": orth_rounds, "estimate_trace_inv_scaled_gram": orth_estimate},
        "clocks": clocks,
        "roofline": rooflines[0] if rooflines else None, "rooflines": rooflines, "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
