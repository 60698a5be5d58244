"""float64 CPU oracle for the LoRAct activation-compression hot path.

TEST INFRASTRUCTURE ONLY.  Nothing in the product (the CUDA library and its
Python binding) imports, links or calls this file; only the tests, the smoke
check and the benchmark's CPU-baseline leg do.  It shares no code with the CUDA
path.  Everything is plain numpy in float64, one statement per step of the
paper, with no blocking, fusion or reordering, so that it can be checked
against the paper by eye.  Library primitives used as single steps: matrix
product, thin QR, SVD.

What follows the paper, and where:
  * ``decompose``      Algorithm 1 (sampling-based orthogonal decomposition)
  * ``reconstruct``    Section 3.1, the Reconstruct equation  A~ = U V
  * ``weight_grad``    Section 3.1: the gradient is taken at A~; for a linear
                       consumer Z = A W that is A~^T G
  * ``norm_forward`` / ``compress_prenorm`` / ``prenorm_backward``
                       Section 3.3, the pre-norm unit and its three gradient
                       equations
  * ``activation_forward`` / ``activation_backward``
                       Section 3.1, the gradient equation for an element-wise
                       Z = f(X) whose saved activation A = X is compressed:
                       grad_X = grad_Z * f'(A~)
  * ``truncated_svd``  Section 3.2 (the Eckart-Young optimum, yardstick)
  * ``rsvd``           Section 3.2: the same steps as Algorithm 1 with the
                       sampled rows replaced by a Gaussian test matrix
  * ``halko_bound_sq`` the deterministic bound of Theorem 3.3

Readings taken where the paper is silent (all listed in the design notes):
rows are tokens; rows are sampled uniformly without replacement, exactly k of
them (no oversampling); the generator is Philox4x32-10 (Salmon et al., SC'11)
and the sample is the first k distinct values of a fixed candidate stream;
t defaults to 0; any thin QR is acceptable (Q is unique only up to column
signs, and up to the completion when Y is rank deficient).

Parity pins (tests/test_oracle_*.py): Philox against the published
known-answer vectors; the sampler by brute-force properties; Algorithm 1 by
exact recovery of rank-<=k inputs (the rank(A)<=k case of the proof of
Theorem 3.3), by Q^T Q = I, Q^T (A - U V) = 0, by the bound of Theorem 3.3 on
tiny inputs with the bound evaluated from a full SVD, and by Eckart-Young;
RSVD by the Halko-Martinsson-Tropp expectation bound quoted in Section 3.2;
the norms by a hand-computed case.  One statement is *parity unpinned*: the
paper's qualitative claim that the sampled test matrix is as accurate as the
Gaussian one -- the comparison is reported, not asserted.
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------
# Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
# as 1, 2, 3", SC'11).  Ten rounds; round function and constants as published.
# --------------------------------------------------------------------------
_PHILOX_M0 = 0xD2511F53
_PHILOX_M1 = 0xCD9E8D57
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_MASK32 = 0xFFFFFFFF


def philox4x32_10(counter, key):
    """One Philox4x32-10 block.  counter: 4 uint32, key: 2 uint32 -> 4 uint32 (python ints)."""
    c0, c1, c2, c3 = (int(x) & _MASK32 for x in counter)
    k0, k1 = (int(x) & _MASK32 for x in key)
    for _ in range(10):
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> 32, p0 & _MASK32
        hi1, lo1 = p1 >> 32, p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + _PHILOX_W0) & _MASK32
        k1 = (k1 + _PHILOX_W1) & _MASK32
    return c0, c1, c2, c3


def _split64(x):
    x = int(x) & 0xFFFFFFFFFFFFFFFF
    return x & _MASK32, x >> 32


def candidate(i: int, n_rows: int, seed: int, call_id: int) -> int:
    """Candidate number i of the row-sampling stream: a value in [0, n_rows).

    Word (i mod 4) of the Philox block with key = seed and counter
    (i div 4, 0, call_id low, call_id high), mapped to the range by the
    multiply-shift  (w * n_rows) >> 32.
    """
    s_lo, s_hi = _split64(seed)
    c_lo, c_hi = _split64(call_id)
    w = philox4x32_10((i // 4, 0, c_lo, c_hi), (s_lo, s_hi))[i % 4]
    return (w * int(n_rows)) >> 32


def sample_indices(n_rows: int, k: int, seed: int, call_id: int = 0) -> np.ndarray:
    """Algorithm 1, sampling step: k distinct row indices, uniform without replacement.

    Defined as the first k distinct values of the candidate stream, kept in
    stream order.
    """
    if not (0 < k <= n_rows):
        raise ValueError("need 0 < k <= n_rows")
    seen = set()
    out = []
    i = 0
    while len(out) < k:
        c = candidate(i, n_rows, seed, call_id)
        if c not in seen:
            seen.add(c)
            out.append(c)
        i += 1
    return np.asarray(out, dtype=np.int64)


def standard_normals(count: int, seed: int, call_id: int = 0) -> np.ndarray:
    """count N(0,1) numbers from Philox + Box-Muller (used by the RSVD yardstick).

    Block q (counter (q, 1, call_id low, call_id high), key = seed) gives words
    w0..w3; u = (w0 + 1) / 2^32 in (0, 1], v = w1 / 2^32;
    z0 = sqrt(-2 ln u) cos(2 pi v), z1 = sqrt(-2 ln u) sin(2 pi v); w2, w3 give
    z2, z3 the same way.  Number e of the sequence is z_(e mod 4) of block e div 4.
    """
    s_lo, s_hi = _split64(seed)
    c_lo, c_hi = _split64(call_id)
    out = np.empty(((count + 3) // 4) * 4, dtype=np.float64)
    for q in range(out.size // 4):
        w = philox4x32_10((q & _MASK32, 1, c_lo, c_hi), (s_lo, s_hi))
        for h in range(2):
            u = (w[2 * h] + 1) / 4294967296.0
            v = w[2 * h + 1] / 4294967296.0
            rad = np.sqrt(-2.0 * np.log(u))
            out[4 * q + 2 * h] = rad * np.cos(2.0 * np.pi * v)
            out[4 * q + 2 * h + 1] = rad * np.sin(2.0 * np.pi * v)
    return out[:count]


# --------------------------------------------------------------------------
# Algorithm 1 and its consumers
# --------------------------------------------------------------------------
def _f64(a):
    return np.asarray(a, dtype=np.float64)


def range_finder(A, Omega_T, t: int = 0):
    """Algorithm 1 from the sketch to the orthonormal basis, for a given test matrix (rows of Omega_T are the
    test vectors).

    Y = A Omega;  t times { Y = QR;  Y = A (A^T Q) };  Y = QR;  returns Q (m x k).
    """
    A = _f64(A)
    Y = A @ _f64(Omega_T).T                      # the sketch
    for _ in range(int(t)):                      # the power-iteration loop
        Q, _ = np.linalg.qr(Y, mode="reduced")
        Y = A @ (A.T @ Q)
    Q, _ = np.linalg.qr(Y, mode="reduced")       # QR of the sketch
    return Q


def decompose(A, k: int, t: int = 0, seed: int = 0, call_id: int = 0, idx=None):
    """Algorithm 1.  Returns (U (m x k), V (k x n), idx (k,))."""
    A = _f64(A)
    m, _ = A.shape
    if idx is None:
        idx = sample_indices(m, k, seed, call_id)    # the sampling step
    idx = np.asarray(idx, dtype=np.int64)
    A_k = A[idx, :]                                  # the sampled rows
    Q = range_finder(A, A_k, t)                      # sketch, loop, QR
    U = Q                                            # the factor pair
    V = Q.T @ A
    return U, V, idx


def reconstruct(U, V):
    """A~ = U V  (the Reconstruct step of Section 3.1)."""
    return _f64(U) @ _f64(V)


def weight_grad(U, V, G):
    """A~^T G evaluated from the factors as V^T (U^T G); A~ is never formed."""
    return _f64(V).T @ (_f64(U).T @ _f64(G))


def weight_grad_via_reconstruct(U, V, G):
    """A~^T G as the paper states it: reconstruct first, then differentiate the linear map."""
    return reconstruct(U, V).T @ _f64(G)


def rel_fro_error(A, U, V) -> float:
    A = _f64(A)
    return float(np.linalg.norm(A - reconstruct(U, V)) / np.linalg.norm(A))


def orthogonality_defect(U) -> float:
    U = _f64(U)
    return float(np.max(np.abs(U.T @ U - np.eye(U.shape[1]))))


# --------------------------------------------------------------------------
# Pre-norm unit (Section 3.3)
# --------------------------------------------------------------------------
def norm_forward(X, gamma, beta=None, eps: float = 1e-6, kind: str = "rms"):
    """A = Norm(X).  Returns (A, rstd (m,), mean (m,) or None).

    kind "rms":   A = X / RMS(X) * gamma, RMS_i = sqrt(mean_j X_ij^2 + eps)
    kind "layer": A = (X - mean_i) / sqrt(var_i + eps) * gamma + beta (the textbook LayerNorm,
                  needed because the ViT workload's blocks use it; the paper writes the RMS form)
    """
    X = _f64(X)
    gamma = _f64(gamma)
    if kind == "rms":
        rstd = 1.0 / np.sqrt(np.mean(X * X, axis=1) + eps)
        return X * rstd[:, None] * gamma[None, :], rstd, None
    if kind == "layer":
        mean = np.mean(X, axis=1)
        xc = X - mean[:, None]
        rstd = 1.0 / np.sqrt(np.mean(xc * xc, axis=1) + eps)
        A = xc * rstd[:, None] * gamma[None, :]
        if beta is not None:
            A = A + _f64(beta)[None, :]
        return A, rstd, mean
    raise ValueError(kind)


def compress_prenorm(X, gamma, beta, eps, kind, k, t=0, seed=0, call_id=0, in_dtype=None):
    """Store the normalised block input once, compressed, together with the per-row statistic.

    ``in_dtype`` (a numpy-compatible caster, e.g. a bf16 round-trip) is applied to A before
    compression when the stored activation is kept in a narrower type than float64.
    """
    A, rstd, mean = norm_forward(X, gamma, beta, eps, kind)
    if in_dtype is not None:
        A = _f64(in_dtype(A))
    U, V, idx = decompose(A, k, t, seed, call_id)
    return A, rstd, mean, U, V, idx


def prenorm_backward_rms(A_tilde, gamma, rstd, grad_A):
    """The three gradient equations of Section 3.3 for the RMS form.

    Xbar = A~ / gamma;  grad_Xbar = grad_A * gamma;
    grad_X = rstd * (grad_Xbar - Xbar * mean_j(grad_Xbar * Xbar)).
    """
    gamma = _f64(gamma)
    Xbar = _f64(A_tilde) / gamma[None, :]
    gXbar = _f64(grad_A) * gamma[None, :]
    inner = np.mean(gXbar * Xbar, axis=1)
    return _f64(rstd)[:, None] * (gXbar - Xbar * inner[:, None])


# --------------------------------------------------------------------------
# Element-wise consumers (Section 3.1: the derivative of Z = f(X) is taken at A~)
# --------------------------------------------------------------------------
def _std_normal_cdf(a):
    from math import erf, sqrt
    return 0.5 * (1.0 + np.vectorize(erf)(a / sqrt(2.0)))


def activation_forward(A, kind: str = "silu"):
    """Z = f(A) element-wise.  "silu": a / (1 + exp(-a));  "gelu": a * Phi(a), Phi the standard normal
    distribution function (the exact form, not the tanh approximation)."""
    A = _f64(A)
    if kind == "silu":
        return A / (1.0 + np.exp(-A))
    if kind == "gelu":
        return A * _std_normal_cdf(A)
    raise ValueError(kind)


def activation_backward(A_tilde, grad_Z, kind: str = "silu"):
    """grad_X = grad_Z * f'(A~), the gradient equation of Section 3.1 for an element-wise f.

    silu: f'(a) = s (1 + a (1 - s)), s = 1 / (1 + exp(-a));
    gelu: f'(a) = Phi(a) + a phi(a), phi the standard normal density.
    """
    a = _f64(A_tilde)
    if kind == "silu":
        s = 1.0 / (1.0 + np.exp(-a))
        d = s * (1.0 + a * (1.0 - s))
    elif kind == "gelu":
        d = _std_normal_cdf(a) + a * np.exp(-0.5 * a * a) / np.sqrt(2.0 * np.pi)
    else:
        raise ValueError(kind)
    return _f64(grad_Z) * d


# --------------------------------------------------------------------------
# Yardsticks
# --------------------------------------------------------------------------
def truncated_svd(A, k: int):
    """Best rank-k approximation (Eckart-Young): returns (U_k, diag(s_k) V_k^T)."""
    Uf, s, Vt = np.linalg.svd(_f64(A), full_matrices=False)
    return Uf[:, :k], s[:k, None] * Vt[:k, :]


def rsvd(A, k: int, oversample: int = 0, power_iters: int = 0, seed: int = 0, call_id: int = 0,
         truncate: bool = True):
    """Randomized SVD of Halko, Martinsson and Tropp: Algorithm 1 with a Gaussian test matrix.

    l = k + oversample Gaussian test vectors (n x l, filled row-major from
    ``standard_normals``).  With truncate=True the l-column basis is cut to rank
    k through the SVD of B = Q^T A; with truncate=False the rank-l pair (Q, Q^T A) is returned.
    """
    A = _f64(A)
    _, n = A.shape
    l = k + oversample
    Omega = standard_normals(n * l, seed, call_id).reshape(n, l)
    Q = range_finder(A, Omega.T, power_iters)
    B = Q.T @ A
    if not truncate or l == k:
        return Q, B
    Ub, s, Vt = np.linalg.svd(B, full_matrices=False)
    return Q @ Ub[:, :k], s[:k, None] * Vt[:k, :]


def halko_bound_sq(A, Omega, k: int) -> float:
    """Right-hand side of Theorem 3.3 in the spectral norm:
    ||Sigma_2||^2 + ||Sigma_2 Omega_2 Omega_1^+||^2, with Omega (n x l) an arbitrary test matrix,
    Omega_1 = V_1^T Omega, Omega_2 = V_2^T Omega, V_1 the first k right singular vectors of A.
    Returns +inf when Omega_1 does not have full row rank.
    """
    A = _f64(A)
    _, s, Vt = np.linalg.svd(A, full_matrices=True)
    n = A.shape[1]
    sig = np.zeros(n)
    sig[: s.size] = s
    V1t, V2t = Vt[:k, :], Vt[k:, :]
    O1, O2 = V1t @ _f64(Omega), V2t @ _f64(Omega)
    if np.linalg.matrix_rank(O1) < k:
        return float("inf")
    S2 = sig[k:]
    tail = (S2[:, None] * O2) @ np.linalg.pinv(O1)
    s2max = S2.max() if S2.size else 0.0
    return float(s2max ** 2 + np.linalg.norm(tail, 2) ** 2)
