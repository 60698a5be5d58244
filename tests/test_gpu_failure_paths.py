"""Failure paths that can be taken without faulting, trapping or hanging a GPU.

(a) A bounded device-side wait that runs out: a tiny kernel waits, with the library's own wait helpers, on a
    barrier that nothing completes; after a millisecond it gives up, records LORACT_DEV_WAIT_EXPIRED and returns.
(b) A non-finite input: the factorisation notices it (the trace of a Gram matrix is not finite), records
    LORACT_DEV_NONFINITE and runs to its end; the next call on clean data is clean.
"""
import time

import pytest
import torch

import __graft_entry__ as entry
from paper_2509_23472_b200 import binding as B
from paper_2509_23472_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    entry.build()
    B.lib()
    return torch.device("cuda:0")


@pytest.mark.parametrize("which", [0, 1])   # 0: tensor-core engine's wait, 1: cluster factorisation's wait
def test_a_bounded_wait_runs_out_and_reports_it(dev, which):
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    t0 = time.perf_counter()
    B.debug_wait_expiry(which, 1_000_000, status)          # one millisecond
    torch.cuda.synchronize()
    elapsed = time.perf_counter() - t0
    word = int(status.item()) & 0xFFFFFFFF
    assert word == B.DEV_WAIT_EXPIRED
    assert elapsed < 1.0                                     # it gave up at its limit, not at the built-in one
    assert B.status_from_device_word(word) == 7              # LORACT_ERR_TIMEOUT
    # the context is intact: an ordinary call right behind it works and is clean
    w = synth.scaled(synth.WORKLOADS["llama7b_block"], n_tokens=1024, d=512, rank=64, signal_rank=128)
    X = synth.make_inputs(w, device=dev)["X"]
    desc = B.make_desc(X, 64, w.seed)
    ws = B.alloc_workspace(desc, dev)
    U, V, _ = B.compress(X, 64, seed=w.seed, ws=ws)
    assert B.read_device_status(ws) == 0
    assert bool(torch.isfinite(U.float()).all())


def test_status_word_mapping_is_a_pure_host_function(dev):
    assert B.status_from_device_word(0) == 0
    assert B.status_from_device_word(B.DEV_PIVOT_CLAMPED) == 0          # a warning only
    assert B.status_from_device_word(B.DEV_NONFINITE) == 6              # LORACT_ERR_NUMERIC
    assert B.status_from_device_word(B.DEV_SAMPLER_SHORT | B.DEV_PIVOT_CLAMPED) == 6
    assert B.status_from_device_word(B.DEV_WAIT_EXPIRED | B.DEV_NONFINITE) == 7


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_non_finite_input_is_flagged_and_the_next_call_is_clean(dev, dtype):
    w = synth.scaled(synth.WORKLOADS["llama7b_block"], n_tokens=1024, d=512, rank=64, signal_rank=128)
    X = synth.make_inputs(w, device=dev)["X"].to(dtype)
    desc = B.make_desc(X, 64, w.seed)
    ws = B.alloc_workspace(desc, dev)
    idx = B.sample_indices(desc, dev)
    bad = X.clone()
    bad[int(idx[3].item()), 17] = float("nan")             # inside a sampled row: it reaches every Gram matrix
    U, V, idx2 = B.compress(bad, 64, seed=w.seed, ws=ws)
    word = B.read_device_status(ws)
    assert torch.equal(idx, idx2)                            # the sample does not depend on the data
    assert word & B.DEV_NONFINITE, hex(word)
    assert not (word & B.DEV_WAIT_EXPIRED)
    assert B.status_from_device_word(word) == 6
    # same workspace, clean data: clean word, finite orthonormal factors
    U, V, _ = B.compress(X, 64, seed=w.seed, ws=ws)
    assert B.read_device_status(ws) == 0
    assert bool(torch.isfinite(U.float()).all()) and bool(torch.isfinite(V.float()).all())
    G = U.double().t() @ U.double()
    assert float((G - torch.eye(64, dtype=torch.float64, device=dev)).abs().max()) <= 4e-3


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_weight_grad_starts_from_a_clean_status_word(dev, dtype):
    # The first kernel of loract_weight_grad clears the status word itself (tensor-core path) or a memset does
    # (CUDA-core path): whatever an earlier call left there must not be reported for this one.
    w = synth.scaled(synth.WORKLOADS["llama7b_block"], n_tokens=2048, d=512, rank=64, signal_rank=128)
    inp = synth.make_inputs(w, device=dev)
    X, G = inp["X"].to(dtype), inp["G"].to(dtype)
    ws = B.alloc_workspace(B.make_desc(X, 64, w.seed), dev)
    U, V, _ = B.compress(X, 64, seed=w.seed, ws=ws)
    ws[0:4] = torch.tensor([0xEF, 0xBE, 0x00, 0x00], dtype=torch.uint8, device=dev)   # stale bits of some earlier call
    torch.cuda.synchronize()
    dW = B.weight_grad(U, V, G, ws=ws)
    assert B.read_device_status(ws) == 0
    ref = (U.double() @ V.double()).t() @ G.double()
    assert float(torch.linalg.norm(dW.double() - ref) / torch.linalg.norm(ref)) <= 1e-3
