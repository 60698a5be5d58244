"""The entry point for callers that cannot allocate (loract_weight_grad_static) against the ordinary one.

Some callers -- a backward hook that runs while the framework's allocator is locked or out of memory, a
runtime whose memory plan was fixed ahead of time -- cannot hand the library a workspace.  The static
variant keeps its intermediate in a fixed array inside the library instead.  This file is collected last
on purpose: it must pass both alone in a fresh process and after every other test has used the library.
"""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from oracle import loract_oracle as orc
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
    assert B.weight_grad_static_status(dev) == 0
    # and against the oracle's formula on the same factors (the bar of the weight-gradient tests)
    want = orc.weight_grad(U.double().cpu().numpy(), V.double().cpu().numpy(), G.double().cpu().numpy())
    assert np.linalg.norm(out1.double().cpu().numpy() - want) / np.linalg.norm(want) <= 1e-3
    # a warm call takes no device memory: the free-memory figure of the driver does not move
    free0 = torch.cuda.mem_get_info(dev)[0]
    B.weight_grad_static(U, V, G2, out2)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info(dev)[0] == free0
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
    # the descriptor rules are those of loract_weight_grad: rank <= n_tokens, rank <= d
    with pytest.raises(B.LoractError) as e:
        B.weight_grad_static(U[:256], V, G[:256, :16], dW[:, :16].contiguous())
    assert e.value.code == 1


@pytest.mark.parametrize("dtype,n,r,g", [(torch.bfloat16, 8192, 512, 128), (torch.float32, 4096, 256, 240)])
def test_static_scratch_with_fewer_partial_sums_than_the_workspace_version(dtype, n, r, g):
    """Large rank * g leaves room for fewer partial sums of T in the fixed array than the workspace version
    takes (bf16: 2 instead of 32; fp32 from 4096 rows: 3 instead of 16): the split over the tokens is coarser,
    the result the same up to the order of the additions."""
    entry.build()
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev)
    gen.manual_seed(r + g)
    d = 1024
    U = (torch.randn(n, r, generator=gen, device=dev) / n ** 0.5).to(dtype)
    V = torch.randn(r, d, generator=gen, device=dev).to(dtype)
    G = torch.randn(n, g, generator=gen, device=dev).to(dtype)
    ref = B.weight_grad(U, V, G)
    out = torch.full_like(ref, float("nan"))
    B.weight_grad_static(U, V, G, out)
    torch.cuda.synchronize()
    assert _rel(out, ref) <= 1e-5
    assert B.weight_grad_static_status(dev) == 0
