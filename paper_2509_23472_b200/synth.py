"""Seeded synthetic activations for the LoRAct hot path.

This module only *draws inputs*.  It holds none of the method's arithmetic (no
sampling of rows, no decomposition) so that the float64 oracle and the CUDA
path can both be fed from it without sharing any code of the method itself.

Recipe (one for every workload):  ``X = (A * sigma) @ B + nu * E`` with
``A (N x R)``, ``B (R x d)``, ``E (N x d)`` i.i.d. N(0,1), drawn in that order
in float32 from one ``torch.Generator`` seeded with the workload's seed, then
rounded once to the workload's dtype.  The nominal spectra ``sigma_i`` are long
tailed, like the measured activation spectra in the paper's Fig. 2; the realised
singular values are only nominally ``sigma_i`` because Gaussian factors are not
orthonormal.  ``G`` (upstream gradients of the LoRA consumers) is i.i.d. N(0,1)
in X's dtype from seed+1000.  The pre-norm workload also draws ``gamma`` and
``beta`` from seed+2000.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Callable, Optional

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    n_tokens: int
    d: int
    dtype: str               # "f32" | "bf16"
    rank: int                # r = k of Algorithm 1
    signal_rank: int         # R
    spectrum: str            # "geom:0.9" | "pow:1.5" | "exp:40"
    noise: float             # nu
    g: int                   # total columns of G (all consumers concatenated)
    consumers: int = 1       # number of LoRA consumers sharing the compression
    prenorm: Optional[str] = None   # None | "rms" | "layer"

    def sigma(self) -> torch.Tensor:
        kind, par = self.spectrum.split(":")
        i = torch.arange(1, self.signal_rank + 1, dtype=torch.float64)
        p = float(par)
        if kind == "geom":
            s = p ** i
        elif kind == "pow":
            s = i ** (-p)
        elif kind == "exp":
            s = torch.exp(-i / p)
        else:
            raise ValueError(self.spectrum)
        return s.to(torch.float32)

    @property
    def torch_dtype(self) -> torch.dtype:
        return {"f32": torch.float32, "bf16": torch.bfloat16}[self.dtype]

    @property
    def elem_bytes(self) -> int:
        return {"f32": 4, "bf16": 2}[self.dtype]


def _w(name, seed, n, d, dtype, r, R, spec, nu, g, consumers=1, prenorm=None):
    return Workload(name, seed, n, d, dtype, r, R, spec, nu, g, consumers, prenorm)


# The five configurations the headline metric is defined on.
WORKLOADS = {
    # small fp32 case the float64 oracle finishes in well under a second
    "small_f32": _w("small_f32", 0, 512, 768, "f32", 64, 48, "geom:0.9", 1e-3, 16),
    # ViT-B/16: 64 images x 197 tokens, LayerNorm input shared by q/k/v LoRA-A gradients
    "vit_b16_prenorm": _w("vit_b16_prenorm", 1, 64 * 197, 768, "bf16", 96, 128, "pow:1.5",
                          1e-2, 48, consumers=3, prenorm="layer"),
    # LLaMA-7B block input: 8 x 2048 tokens, six LoRA-A consumers (q/k/v/o/gate/up)
    "llama7b_block": _w("llama7b_block", 2, 8 * 2048, 4096, "bf16", 256, 512, "exp:40",
                        1e-2, 96, consumers=6),
    # LLaMA-7B MLP intermediate activation, down_proj LoRA-A
    "llama7b_mlp": _w("llama7b_mlp", 3, 16384, 11008, "bf16", 512, 1024, "pow:1.0", 1e-2, 16),
}


def llama13b_sweep_point(seq: int, rank: int) -> Workload:
    """One point of the LLaMA-13B long-context sweep: batch 4 x seq tokens, d = 5120."""
    seqs = (1024, 2048, 4096, 8192)
    ranks = (64, 128, 256, 512)
    idx = seqs.index(seq) * len(ranks) + ranks.index(rank)
    return _w(f"llama13b_s{seq}_r{rank}", 4 + idx, 4 * seq, 5120, "bf16", rank, 768,
              "exp:64", 1e-2, 16)


def get_workload(name: str) -> Workload:
    if name in WORKLOADS:
        return WORKLOADS[name]
    if name.startswith("llama13b_s"):
        s, r = name[len("llama13b_s"):].split("_r")
        return llama13b_sweep_point(int(s), int(r))
    raise KeyError(name)


def scaled(w: Workload, n_tokens: int = None, d: int = None, rank: int = None,
           signal_rank: int = None, name: str = None) -> Workload:
    """Same recipe at another size (parity tests use reduced shapes)."""
    return dataclasses.replace(
        w, n_tokens=n_tokens or w.n_tokens, d=d or w.d, rank=rank or w.rank,
        signal_rank=signal_rank or w.signal_rank, name=name or (w.name + "_scaled"))


def low_rank_plus_noise(n: int, d: int, signal_rank: int, sigma: torch.Tensor, noise: float,
                        seed: int, dtype: torch.dtype, device="cpu") -> torch.Tensor:
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    prev = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    try:
        A = torch.randn(n, signal_rank, generator=gen, device=device, dtype=torch.float32)
        B = torch.randn(signal_rank, d, generator=gen, device=device, dtype=torch.float32)
        X = (A * sigma.to(device)) @ B
        del A, B
        # the noise is added in row chunks so the largest case needs one extra N x d buffer at most
        step = max(1, (1 << 26) // max(d, 1))
        for s in range(0, n, step):
            e = min(n, s + step)
            X[s:e].add_(torch.randn(e - s, d, generator=gen, device=device, dtype=torch.float32),
                        alpha=noise)
    finally:
        torch.backends.cuda.matmul.allow_tf32 = prev
    return X.to(dtype)


def make_inputs(w: Workload, device="cpu") -> dict:
    """Returns {"X", "G"[, "gamma", "beta"]} on ``device`` in the workload's dtype."""
    X = low_rank_plus_noise(w.n_tokens, w.d, w.signal_rank, w.sigma(), w.noise, w.seed,
                            w.torch_dtype, device)
    gen = torch.Generator(device=device)
    gen.manual_seed(w.seed + 1000)
    G = torch.randn(w.n_tokens, w.g, generator=gen, device=device,
                    dtype=torch.float32).to(w.torch_dtype)
    out = {"X": X, "G": G}
    if w.prenorm is not None:
        gen.manual_seed(w.seed + 2000)
        gamma = 1.0 + 0.1 * torch.randn(w.d, generator=gen, device=device, dtype=torch.float32)
        beta = 0.1 * torch.randn(w.d, generator=gen, device=device, dtype=torch.float32)
        out["gamma"] = gamma.to(w.torch_dtype)
        out["beta"] = beta.to(w.torch_dtype) if w.prenorm == "layer" else None
    return out


def exact_low_rank(n: int, d: int, inner: int, seed: int, device="cpu") -> torch.Tensor:
    """float64 matrix of rank <= inner (product of two Gaussian factors), for exact-recovery checks."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    B = torch.randn(n, inner, generator=gen, device=device, dtype=torch.float64)
    C = torch.randn(inner, d, generator=gen, device=device, dtype=torch.float64)
    return B @ C / math.sqrt(inner)


def plant_private_outliers(X: torch.Tensor, n_out: int, scale: float, seed: int) -> torch.Tensor:
    """A coherent variant of an input: `n_out` feature columns are cleared everywhere and each is given one
    entry of size scale * (RMS of X) in a token row of its own.  These rank-one components live on single
    rows, so a uniform row sample that misses those rows cannot see them (the regime where the paper's
    coherence term bites); the rest of X is unchanged.  Rows and columns are drawn from `seed`."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    n, d = X.shape
    rows = torch.randperm(n, generator=gen)[:n_out].to(X.device)
    cols = torch.randperm(d, generator=gen)[:n_out].to(X.device)
    rms = float(X.float().pow(2).mean().sqrt())
    Y = X.clone()
    Y[:, cols] = 0
    Y[rows, cols] = torch.tensor(scale * rms, dtype=X.dtype, device=X.device)
    return Y
