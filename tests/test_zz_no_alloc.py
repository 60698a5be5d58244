"""The entry point for callers that cannot allocate (loract_weight_grad_static) against the ordinary one.

Some callers -- a backward hook that runs while the framework's allocator is locked or out of memory, a
runtime whose memory plan was fixed ahead of time -- cannot hand the library a workspace.  The static
variant keeps its intermediate in a fixed array inside the library instead.  This file is collected last
on purpose: it must pass both alone in a fresh process and after every other test has used the library.
"""
import pytest
import torch

import __graft_entry__ as entry
from paper_2509_23472_b200 import binding as B
from paper_2509_23472_b200 import synth

pytestmark = pytest.mark.gpu


def _rel(a, b):
    return float((a.double() - b.double()).norm() / b.double().norm())


def test_static_scratch_weight_grad_matches_the_workspace_version_twice_in_a_row():
    entry.build()
    dev = torch.device("cuda:0")
    w = synth.scaled(synth.WORKLOADS["llama7b_block"], n_tokens=3000, d=768, rank=64, signal_rank=128)
    inp = synth.make_inputs(w, device=dev)
    X, G = inp["X"], inp["G"]                      # g = 96
    U, V, _ = B.compress(X, 64, seed=w.seed)
    ref = B.weight_grad(U, V, G)
    # first call (this also performs the per-device address look-up), then a second call with other data:
    # the shared array still holds the first call's intermediates and must not leak into the second
    out1 = torch.full_like(ref, float("nan"))
    B.weight_grad_static(U, V, G, out1)
    G2 = (G.float() * -0.5 + 1.0).to(G.dtype)[:, :48].contiguous()
    ref2 = B.weight_grad(U, V, G2)
    out2 = torch.full_like(ref2, float("nan"))
    B.weight_grad_static(U, V, G2, out2)
    torch.cuda.synchronize()
    assert _rel(out1, ref) <= 1e-5
    assert _rel(out2, ref2) <= 1e-5
    # accumulate adds onto what the caller passed
    B.weight_grad_static(U, V, G2, out2, accumulate=True)
    torch.cuda.synchronize()
    assert _rel(out2, 2 * ref2) <= 1e-5
    # fp32 factors go through the CUDA-core kernels and the same array
    Uf, Vf, Gf = U.float(), V.float(), G.float()
    reff = B.weight_grad(Uf, Vf, Gf)
    outf = torch.empty_like(reff)
    B.weight_grad_static(Uf, Vf, Gf, outf)
    torch.cuda.synchronize()
    assert _rel(outf, reff) <= 1e-5


def test_static_scratch_rejects_sizes_beyond_its_array_and_launches_nothing():
    entry.build()
    dev = torch.device("cuda:0")
    U = torch.zeros(1024, 512, dtype=torch.bfloat16, device=dev)
    V = torch.zeros(512, 1024, dtype=torch.bfloat16, device=dev)
    G = torch.zeros(1024, 256, dtype=torch.bfloat16, device=dev)
    dW = torch.zeros(1024, 256, dtype=torch.float32, device=dev)
    before = B.kernel_launch_count()
    with pytest.raises(B.LoractError) as e:
        B.weight_grad_static(U, V, G, dW)          # rank 512 x g 256 does not fit in the 1 MiB array
    assert e.value.code == 2
    assert B.kernel_launch_count() == before
    B.weight_grad_static(U, V, G[:, :128], dW[:, :128].contiguous())   # rank 512 x g 128 fits
    torch.cuda.synchronize()
