"""GPU tests of the small-block step of the orthonormalisation (the QR step of Algorithm 1 through Gram matrices):
from W = sum of partials, the inverse of the Cholesky factor of W + shift * mean(diag W) * I.

Checked against the definition in float64 (numpy's Cholesky and inverse): the device's L^{-1} must be lower
triangular, must whiten W (L^{-1} W L^{-T} = I up to fp32 rounding times the condition number) and must
agree with the float64 inverse factor.  Sizes cover every block count of the shared-memory cluster kernel
(r <= 256, including ragged last blocks) and the general kernel (r > 256)."""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from paper_2509_23472_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    entry.build()
    B.lib()
    return torch.device("cuda:0")


def spd(r: int, cond: float, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    Q, _ = np.linalg.qr(rng.standard_normal((r, r)))
    s = np.logspace(0.0, -np.log10(cond), r)
    return (Q * s) @ Q.T


@pytest.mark.parametrize("r,n_partials,cond", [(16, 1, 1e2), (32, 3, 1e3), (48, 2, 1e3), (64, 4, 1e4),
                                              (96, 1, 1e4), (128, 5, 1e5), (160, 2, 1e3), (192, 1, 1e3),
                                              (208, 3, 1e4), (224, 1, 1e2), (240, 2, 1e5), (256, 16, 1e5),
                                              (256, 1, 1.5), (272, 2, 1e3), (320, 1, 1e4), (384, 3, 1e5),
                                              (496, 2, 1e3), (512, 4, 1e4), (520, 1, 1e3), (640, 2, 1e4)])
def test_inverse_cholesky_factor(dev, r, n_partials, cond):
    W = spd(r, cond, seed=r + n_partials)
    rng = np.random.default_rng(7)
    # partials that sum to W: W / n plus zero-sum symmetric perturbations
    P = np.repeat(W[None] / n_partials, n_partials, axis=0)
    if n_partials > 1:
        Z = rng.standard_normal((n_partials, r, r)) * 0.1 * np.abs(W).mean()
        Z = Z + Z.transpose(0, 2, 1)
        Z -= Z.mean(axis=0, keepdims=True)
        P = P + Z
    P32 = torch.tensor(P, dtype=torch.float32, device=dev)
    W32 = P32.double().sum(0).cpu().numpy()           # what the device actually sums (up to fp32 order)
    shift = 1e-6
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    for _ in range(2):                                 # twice: the second call must not depend on the first
        L32, Lh, Ll = B.debug_small_block(P32, use_f64=False, shift_rel=shift, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    X = L32.double().cpu().numpy()
    assert np.all(np.isfinite(X))
    assert np.abs(np.triu(X, 1)).max() == 0.0
    Ws = W32 + shift * np.trace(W32) / r * np.eye(r)
    Lref = np.linalg.cholesky(Ws)
    Xref = np.linalg.inv(Lref)
    white = X @ Ws @ X.T
    eps32 = 2.0 ** -24
    kappa = np.linalg.cond(Ws)
    assert np.abs(white - np.eye(r)).max() <= 50 * r * eps32 * kappa + 1e-5
    assert np.linalg.norm(X - Xref) <= (50 * r * eps32 * kappa + 1e-5) * np.linalg.norm(Xref)
    # the bf16 pair carries the same matrix to 16 bits
    pair = Lh.double().cpu().numpy() + Ll.double().cpu().numpy()
    assert np.abs(pair - X).max() <= 2.0 ** -15 * np.abs(X).max()


def test_non_positive_pivot_is_clamped_and_reported(dev):
    r = 64
    W = spd(r, 1e2, seed=3)
    W[40, 40] = -1.0                                   # indefinite: the pivot of column 40 cannot be positive
    P32 = torch.tensor(W[None], dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    L32, _, _ = B.debug_small_block(P32, use_f64=False, shift_rel=0.0, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) & B.DEV_PIVOT_CLAMPED
    assert bool(torch.isfinite(L32).all())


def test_two_level_scheme_judges_the_schur_complement_on_the_scale_of_the_whole_matrix(dev):
    # r = 512 goes through two 256-wide factorisations joined by a Schur complement.  Here the last 256 columns
    # of the factored Gram matrix are exact linear combinations of the first 256, so that complement is
    # nothing but the rounding noise of W22 - L21 L21^T (about 1e-7 of W's diagonal, of either sign).  The
    # shift and the pivot floor of the second factorisation must come from W's diagonal: taken from the
    # complement's own, they would let that noise through as pivots and the inverse would blow up.
    # Expected: a finite factor whose leading block is still the inverse Cholesky factor of W11 and whose
    # trailing block is bounded by the inverse square root of the shift.
    r = 512
    rng = np.random.default_rng(11)
    Y1 = 30.0 * rng.standard_normal((2048, 256))
    C = rng.standard_normal((256, 256)) / 16.0
    Y = np.concatenate([Y1, Y1 @ C], axis=1)
    W = Y.T @ Y / 2048.0
    shift = 3e-6
    P32 = torch.tensor(W[None], dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    L32, Lh, Ll = B.debug_small_block(P32, use_f64=False, shift_rel=shift, status=status)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(L32).all()) and bool(torch.isfinite(Lh.float()).all())
    assert not int(status.item()) & B.DEV_NONFINITE
    W11 = W[:256, :256] + shift * np.trace(W) / 512 * np.eye(256)
    X11 = L32[:256, :256].double().cpu().numpy()
    assert np.abs(X11 @ W11 @ X11.T - np.eye(256)).max() <= 1e-3
    scale = np.trace(W[:256, :256]) / 256
    assert float(L32[256:, 256:].abs().max()) <= 4.0 / np.sqrt(shift * scale)
