"""Times every workload of `synth` through the public binding and prints one markdown table.

    python -m paper_2509_23472_b200.report [--reps 30] [--only NAME[,NAME...]] [--no-sweep]

Per workload: `loract_compress` (or `loract_compress_prenorm` where the workload has a norm), all of its
`loract_weight_grad` calls (one call with every consumer's G concatenated, and one call per consumer),
`loract_reconstruct`, and the randomized-SVD comparator at equal rank (one power iteration) beside it.
Timing: CUDA events on the launching stream, 5 warm-up calls, then `reps` calls with a 256 MiB memset
before each one (outside the events) so the input is not L2-resident; the median is reported.  The relative
Frobenius error of the reconstruction is measured with the library's own `loract_reconstruct` and plain
torch norms (row chunks, fp32).  Nothing here runs on a CPU.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import sys

import torch

from . import binding as B
from . import synth


def _peaks():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    path = os.path.join(root, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return p["hbm_gbs"], p["bf16_tflops"], "measured"
    return 6650.0, 1590.0, "fallback"


def _median_us(fn, reps, flush):
    for _ in range(5):
        fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1) * 1e3)
    return statistics.median(ts), min(ts)


def _rel_error(X, U, V):
    """||X - U V||_F / ||X||_F with U V from loract_reconstruct, accumulated over row chunks in fp32/fp64."""
    Xt = B.reconstruct(U, V)
    num = den = 0.0
    step = max(1, (1 << 25) // X.shape[1])
    for s in range(0, X.shape[0], step):
        a = X[s:s + step].float()
        num += float((a - Xt[s:s + step].float()).pow(2).sum(dtype=torch.float64))
        den += float(a.pow(2).sum(dtype=torch.float64))
    return (num / den) ** 0.5


def truncate_to_rank(Q: torch.Tensor, Bm: torch.Tensor, r: int):
    """The last step of the randomized SVD (Section 3.2): the rank-l pair (Q, B = Q^T X) cut to rank r through
    the singular value decomposition of the small matrix B = W S Z^T: (Q W_r, W_r^T B) = (Q W_r, S_r Z_r^T).  float64 torch on the
    device, outside the comparator's timed region (the l x d decomposition is not part of what the paper
    counts as the cost of either method); the result is rounded to the factors' type."""
    if Q.shape[1] == r:
        return Q, Bm
    B64 = Bm.double()
    # left singular vectors of B from the symmetric eigenproblem of the small l x l matrix B B^T (float64)
    _, W = torch.linalg.eigh(B64 @ B64.t())
    Wr = W[:, -r:]
    return (Q.double() @ Wr).to(Q.dtype), (Wr.t() @ B64).to(Bm.dtype)


def measure(w: synth.Workload, reps: int, dev, flush) -> dict:
    inp = synth.make_inputs(w, device=dev)
    X, G = inp["X"], inp["G"]
    N, d, r, g, es = w.n_tokens, w.d, w.rank, w.g, w.elem_bytes
    desc = B.make_desc(X, r, seed=w.seed, call_id=0)
    ws = B.alloc_workspace(desc, dev)
    row = {"workload": w.name, "N": N, "d": d, "r": r, "g": g, "dtype": w.dtype}

    if w.prenorm is None:
        U = torch.empty(N, r, dtype=X.dtype, device=dev)
        V = torch.empty(r, d, dtype=X.dtype, device=dev)
        idx = torch.empty(r, dtype=torch.int32, device=dev)
        row["compress_us"], row["compress_min_us"] = _median_us(
            lambda: B.compress(X, r, ws=ws, out=(U, V, idx), desc=desc), reps, flush)
        target = X
    else:
        kind = B.NORM_RMS if w.prenorm == "rms" else B.NORM_LAYER
        eps = 1e-6 if w.prenorm == "rms" else 1e-5
        holder = {}

        def run():
            holder["out"] = B.compress_prenorm(X, inp["gamma"], inp["beta"], eps, kind, r, seed=w.seed, ws=ws)
        row["compress_us"], row["compress_min_us"] = _median_us(run, reps, flush)
        target, _, _, U, V, _ = holder["out"]
    row["status"] = B.read_device_status(ws)
    # rounds of the Gram-based orthonormalisation the device chose (fp32 inputs always take two)
    row["rounds"] = B.round_gate_words(ws)[2] if w.dtype == "bf16" else 2
    row["rel_err"] = _rel_error(target, U, V)

    dW = torch.empty(d, g, dtype=torch.float32, device=dev)
    row["wgrad_us"], _ = _median_us(lambda: B.weight_grad(U, V, G, dW=dW, ws=ws), reps, flush)
    if w.consumers > 1:
        gc = g // w.consumers
        Gs = [G[:, i * gc:(i + 1) * gc] for i in range(w.consumers)]
        dWs = [torch.empty(d, gc, dtype=torch.float32, device=dev) for _ in Gs]

        def per_consumer():
            for Gi, dWi in zip(Gs, dWs):
                B.weight_grad(U, V, Gi, dW=dWi, ws=ws)
        row["wgrad_per_consumer_us"], _ = _median_us(per_consumer, reps, flush)
    Xt = torch.empty_like(target)
    row["reconstruct_us"], _ = _median_us(lambda: B.reconstruct(U, V, out=Xt), reps, flush)
    del Xt

    if w.dtype == "bf16" and w.prenorm is None:
        # l = r + 8 test vectors, one power iteration, then cut to rank r: the comparison is at equal rank
        over = 8
        holder = {}

        def run_rsvd_with(extra):
            d0 = B.make_desc(X, r, seed=w.seed, call_id=0)
            need = int(B.lib().loract_rsvd_workspace_bytes(ctypes.byref(d0), extra))
            rws = torch.empty(need, dtype=torch.uint8, device=dev)

            def run():
                holder["out"] = B.rsvd(X, r, oversample=extra, power_iters=1, seed=w.seed, ws=rws)
            t, _ = _median_us(run, max(5, reps // 3), flush)
            return t, B.read_device_status(rws)

        row["rsvd_us"], row["rsvd_status"] = run_rsvd_with(over)
        if (row["rsvd_status"] & B.DEV_NONFINITE) or not bool(torch.isfinite(holder["out"][1].float()).all()):
            # the un-preconditioned Gaussian sketch is beyond what an fp32 Gram matrix resolves here: fall back to
            # the comparator without extra test vectors and say so (column "RSVD l")
            over = 0
            row["rsvd_us"], row["rsvd_status"] = run_rsvd_with(over)
        Q, Bm = holder["out"]
        row["rsvd_l"] = r + over
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        Qr, Br = truncate_to_rank(Q, Bm, r)
        e1.record()
        torch.cuda.synchronize()
        row["rsvd_truncate_us"] = e0.elapsed_time(e1) * 1e3   # off the comparator's clock, reported beside it
        row["rsvd_rel_err"] = _rel_error(X, Qr, Br)

    hbm, tf, src = _peaks()
    t = (row["compress_us"] + row["wgrad_us"]) * 1e-6
    x_bytes = N * d * es
    strict = x_bytes + (N * r + 2 * r * d) * es + (N * r + N * g + r * d) * es + 4 * d * g
    floor = max(strict / (hbm * 1e9), 4.0 * N * d * r / (tf * 1e12))
    row["gbs_of_x"] = x_bytes / t / 1e9
    row["tokens_per_s"] = N / t
    row["floor_us"] = floor * 1e6
    row["frac_of_floor"] = floor / t
    row["peaks"] = src
    return row


COLUMNS = [("workload", "workload", "{}"), ("N", "N", "{}"), ("d", "d", "{}"), ("r", "r", "{}"),
           ("compress_us", "compress us", "{:.0f}"), ("wgrad_us", "wgrad us", "{:.0f}"),
           ("wgrad_per_consumer_us", "wgrad per consumer us", "{:.0f}"), ("reconstruct_us", "reconstruct us", "{:.0f}"),
           ("gbs_of_x", "GB/s of X", "{:.0f}"), ("tokens_per_s", "tokens/s", "{:.3g}"),
           ("floor_us", "floor us", "{:.0f}"), ("frac_of_floor", "floor / time", "{:.3f}"),
           ("rel_err", "rel. error", "{:.4f}"), ("rounds", "rounds", "{}"), ("rsvd_l", "RSVD l", "{}"), ("rsvd_us", "RSVD us", "{:.0f}"),
           ("rsvd_truncate_us", "RSVD cut to r us", "{:.0f}"), ("rsvd_rel_err", "RSVD rel. error at rank r", "{:.4f}"), ("rsvd_status", "RSVD status", "{}"), ("status", "status", "{}")]


def to_markdown(rows) -> str:
    out = ["| " + " | ".join(h for _, h, _ in COLUMNS) + " |", "|" + "---|" * len(COLUMNS)]
    for r in rows:
        out.append("| " + " | ".join(f.format(r[k]) if k in r and r[k] is not None else "-"
                                     for k, _, f in COLUMNS) + " |")
    return "\n".join(out)


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--reps", type=int, default=30)
    ap.add_argument("--only", default="")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--json", action="store_true", help="one JSON object per workload instead of the table")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("report needs a CUDA device: the hot path has no CPU fallback")
    dev = torch.device("cuda", 0)
    B.lib()
    names = list(synth.WORKLOADS)
    if not args.no_sweep:
        names += [f"llama13b_s{s}_r{r}" for s in (1024, 2048, 4096, 8192) for r in (64, 128, 256, 512)]
    if args.only:
        names = [n for n in args.only.split(",") if n]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    rows = []
    for n in names:
        rows.append(measure(synth.get_workload(n), args.reps, dev, flush))
        torch.cuda.empty_cache()
        if args.json:
            print(json.dumps(rows[-1]), flush=True)
    if not args.json:
        print(to_markdown(rows))
    return 0


if __name__ == "__main__":
    sys.exit(main())
