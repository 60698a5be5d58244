"""GPU tests of the device-side decision between one and two orthonormalisation rounds (the QR step of
Algorithm 1 done through Gram matrices).

Algorithm 1 only asks for an orthonormal basis of range(Y); the device gets it as Y L^-T with W = Y^T Y = L L^T and
repeats that round when the first Gram matrix was too ill conditioned for one round to reach the orthonormality bar.
The decision is taken on the device from est = trace((D W D)^-1), D = diag(W)^(-1/2).  Checked here: the deciding
kernel against the same quantity in float64; that one round and two rounds give the same projection and both meet
the orthonormality bar where the device chooses one round; that hard inputs are sent to two rounds."""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from paper_2509_23472_b200 import binding as B, synth
from tests.parity_util import TOL_ORTH, gpu_err, orth_bound, orth_defect

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    entry.build()
    B.lib()
    yield torch.device("cuda:0")
    B.debug_set_round_gate(0.0)


def spd_scaled(r: int, cond: float, spread: float, seed: int) -> np.ndarray:
    """S C S with C of unit diagonal scale and condition number about `cond`, S a diagonal spanning `spread`."""
    rng = np.random.default_rng(seed)
    Q, _ = np.linalg.qr(rng.standard_normal((r, r)))
    C = (Q * np.logspace(0.0, -np.log10(cond), r)) @ Q.T
    s = np.logspace(0.0, -np.log10(spread), r)[rng.permutation(r)]
    return C * s[:, None] * s[None, :]


@pytest.mark.parametrize("r,cond,spread", [(8, 1e1, 1.0), (64, 1e2, 1e3), (136, 1e3, 1e2), (256, 1e4, 1e4),
                                           (264, 1e2, 1.0), (512, 1e3, 1e3), (640, 1e2, 1e1)])
def test_deciding_kernel_matches_float64_trace(dev, r, cond, spread):
    W = spd_scaled(r, cond, spread, seed=r)
    W32 = torch.tensor(W, dtype=torch.float32, device=dev)
    Linv = np.linalg.inv(np.linalg.cholesky(W32.double().cpu().numpy()))
    Lh = torch.tensor(Linv, dtype=torch.float32, device=dev).bfloat16().contiguous()
    Lh64 = Lh.double().cpu().numpy()
    # the definition, from the operands the kernel is given: sum_ij Lh_ij^2 W_jj
    est_ref = float(((Lh64 ** 2) * np.diag(W32.double().cpu().numpy())[None, :]).sum())
    # and what it estimates: trace((D W D)^-1) (Lh is L^-1 rounded to 8 bits, so to about 1 %)
    d = 1.0 / np.sqrt(np.diag(W))
    tr = float(np.trace(np.linalg.inv(W * d[:, None] * d[None, :])))
    for thr, want in ((est_ref * 1.01, 0), (est_ref * 0.99, 1)):
        again, est, rounds = B.debug_round_gate(W32, Lh, thr)
        assert abs(est - est_ref) <= 1e-5 * est_ref
        assert abs(est - tr) <= 0.03 * tr
        assert again == want and rounds == 1 + want
    # a status bit forces the second round whatever the estimate; so does an estimate that is not a number
    status = torch.full((1,), B.DEV_PIVOT_CLAMPED, dtype=torch.int32, device=dev)
    assert B.debug_round_gate(W32, Lh, float("inf"), status)[0] == 1
    bad = W32.clone(); bad[0, 0] = float("nan")
    assert B.debug_round_gate(bad, Lh, float("inf"))[0] == 1
    assert B.debug_round_gate(W32, Lh, -1.0)[0] == 1


@pytest.mark.parametrize("n,d,r,R", [(4096, 1024, 64, 256), (8192, 2048, 256, 512), (3072, 1536, 384, 768)])
def test_one_round_and_two_rounds_agree(dev, n, d, r, R):
    w = synth.scaled(synth.get_workload("llama7b_block"), n_tokens=n, d=d, rank=r, signal_rank=R)
    X = synth.make_inputs(w, device=dev)["X"]
    X64 = X.double()
    ws = B.alloc_workspace(B.make_desc(X, r, seed=w.seed), dev)
    out = {}
    for label, thr in (("two", -1.0), ("auto", 0.0)):
        B.debug_set_round_gate(thr)
        U, V, _ = B.compress(X, r, seed=w.seed, ws=ws)
        torch.cuda.synchronize()
        assert B.read_device_status(ws) == 0
        out[label] = (U.clone(), V.clone(), B.round_gate_words(ws))
    B.debug_set_round_gate(0.0)
    assert out["two"][2][2] == 2 and out["two"][2][0] == 1
    # these inputs are well within one round's reach: the device must see that
    assert out["auto"][2][2] == 1 and out["auto"][2][0] == 0
    assert abs(out["auto"][2][1] - out["two"][2][1]) <= 1e-3 * out["two"][2][1]   # same estimate either way
    for label in out:
        U, V, _ = out[label]
        assert orth_defect(U) <= orth_bound(U)
    P1 = out["auto"][0].double() @ out["auto"][1].double()
    P2 = out["two"][0].double() @ out["two"][1].double()
    # same subspace: the two projections differ by the storage rounding of the factors only
    assert float(torch.linalg.norm(P1 - P2) / torch.linalg.norm(X64)) <= 2.0 ** -8
    assert abs(gpu_err(X64, *out["auto"][:2]) - gpu_err(X64, *out["two"][:2])) <= 1e-3


def test_ill_conditioned_sketch_takes_the_second_round(dev):
    # A sketch whose trailing columns are almost dependent: rank-deficient input (rank 40 < r = 64 plus tiny noise).
    n, d, r = 4096, 1024, 64
    g = torch.Generator(device="cpu").manual_seed(11)
    A = torch.randn(n, 40, generator=g); Bm = torch.randn(40, d, generator=g)
    X = ((A @ Bm) + 1e-4 * torch.randn(n, d, generator=g)).to(torch.bfloat16).to(dev)
    ws = B.alloc_workspace(B.make_desc(X, r, seed=5), dev)
    B.debug_set_round_gate(0.0)
    U, V, _ = B.compress(X, r, seed=5, ws=ws)
    torch.cuda.synchronize()
    again, est, rounds = B.round_gate_words(ws)
    assert rounds == 2 and again == 1
    assert bool(torch.isfinite(U.float()).all())
    # the leading 40 directions carry X: the projection reproduces it to bf16 accuracy
    assert gpu_err(X.double(), U, V) <= 1e-2
