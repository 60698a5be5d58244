"""Shared helpers of the GPU parity tests: run the CUDA path and the float64 oracle on the same seeded
input and compare what is unique (the sampled rows, the projection error, orthonormality, the weight
gradient) -- never the entries of U, which are fixed only up to the choice of basis."""
import numpy as np
import torch

from oracle import loract_oracle as orc
from paper_2509_23472_b200 import binding as B

# tolerances of the parity statement
TOL_ERR = {"bf16": 2e-2, "f32": 1e-4}   # |err_gpu - err_oracle|, relative Frobenius errors
TOL_ORTH = 1e-3                          # max |U^T U - I|
TOL_WGRAD = 2e-2                         # ||dW_gpu - dW_oracle||_F / ||dW_oracle||_F


def tol_projection(err_oracle: float, dtype_key: str) -> float:
    """Bar for ||U_g V_g - U_o V_o||_F / ||X||_F, the distance between the two projections of X.

    P_Y X is unique when Y = X A_k^T has full column rank, so the two sides must agree up to (a) the storage
    rounding of the factors and (b) the tilt of the computed subspace.  (a): U and V are each rounded once to
    the storage type, relative rounding error u per entry (2^-9 for bf16, 2^-24 for fp32), independent, so
    U V moves by about sqrt(2) * u / sqrt(3) of its norm: 1.6e-3 for bf16.  (b): the device rounds the
    preconditioned test matrix to the storage type and keeps the sketch to 16 bits, which tilts only the
    trailing directions of range(Y), those whose singular values are at the level of the projection error
    itself; tilting a direction of weight s by an angle t moves the projection by s * t, so this part scales
    with the error level.  Measured on all five configurations, the sixteen sweep points and the reduced shapes:
    1.6e-3 to 3.2e-3 for bf16 whatever the error level (0.002 to 0.84), i.e. the storage rounding alone (the
    largest values at 64 to 400 rows), and 5e-7 for fp32.  The bar is 2^-8 + err / 100 for bf16 and
    5e-6 + err / 100 for fp32."""
    if dtype_key == "bf16":
        return 2.0 ** -8 + 0.01 * err_oracle
    return 5e-6 + 0.01 * err_oracle


def to64(t: torch.Tensor) -> np.ndarray:
    return t.detach().double().cpu().numpy()


def gpu_err(X64: torch.Tensor, U: torch.Tensor, V: torch.Tensor) -> float:
    """||X - U V||_F / ||X||_F in float64 (torch on the device: test arithmetic, not the product)."""
    R = X64 - U.double() @ V.double()
    return float(torch.linalg.norm(R) / torch.linalg.norm(X64))


def orth_defect(U: torch.Tensor) -> float:
    U64 = U.double()
    return float((U64.t() @ U64 - torch.eye(U.shape[1], dtype=torch.float64, device=U.device)).abs().max())


def orth_bound(U: torch.Tensor, spiky: bool = False) -> float:
    """The orthonormality bar.  1e-3, except where the storage type itself cannot reach it: rounding an
    exactly orthonormal basis to bf16 leaves a defect of about 2^-9 * sqrt(12 / n_tokens), which exceeds 1e-3
    below roughly a thousand rows.  There the bar is 1.25 x the defect of the exactly orthonormalised basis of
    the same subspace after rounding to bf16, i.e. "as orthonormal as the storage type allows".  The same
    applies (`spiky`) when basis vectors concentrate on single rows: an entry near 1 rounds by up to 2^-9, which
    moves a column's squared norm by up to 4e-3 whatever the number of rows."""
    if U.dtype != torch.bfloat16 or (U.shape[0] >= 2048 and not spiky):
        return TOL_ORTH
    Q = torch.linalg.qr(U.double())[0].bfloat16()
    return max(TOL_ORTH, 1.25 * orth_defect(Q) + 1e-4)


def oracle_run(X: torch.Tensor, rank: int, seed: int, call_id: int = 0, G: torch.Tensor = None):
    Xd = to64(X)
    Uo, Vo, idx = orc.decompose(Xd, rank, seed=seed, call_id=call_id)
    out = {"idx": idx, "err": orc.rel_fro_error(Xd, Uo, Vo), "U": Uo, "V": Vo}
    if G is not None:
        out["dW"] = orc.weight_grad(Uo, Vo, to64(G))
    return out


def projection_distance(X64: torch.Tensor, U: torch.Tensor, V: torch.Tensor, Uo: np.ndarray, Vo: np.ndarray) -> float:
    """||U V - U_o V_o||_F / ||X||_F in float64 (torch on the device: test arithmetic, not the product)."""
    dev = X64.device
    ref = torch.from_numpy(Uo).to(dev) @ torch.from_numpy(Vo).to(dev)
    return float(torch.linalg.norm(U.double() @ V.double() - ref) / torch.linalg.norm(X64))


def check_compress(X, rank, seed, call_id=0, G=None, dtype_key="bf16", ws=None, require_status=0,
                   full_rank=True):
    """Runs loract_compress (+ weight_grad) and the oracle; asserts the parity statement; returns both.
    `full_rank`: Y = X A_k^T has full column rank, so the projection U V itself is unique and is compared with
    the oracle's (not the exactly-low-rank, zero and r = min(N, d) cases, where the completion of the basis is
    free or the projection is the identity on a rounding-level residual)."""
    desc = B.make_desc(X, rank, seed, call_id)
    ws = ws if ws is not None else B.alloc_workspace(desc, X.device)
    U, V, idx = B.compress(X, rank, seed=seed, call_id=call_id, ws=ws)
    status = B.read_device_status(ws)
    ref = oracle_run(X, rank, seed, call_id, G)
    assert np.array_equal(idx.cpu().numpy().astype(np.int64), ref["idx"]), "sampled rows differ"
    if require_status is not None:
        assert status == require_status, f"device status {status:#x}"
    X64 = X.double()
    e_gpu = gpu_err(X64, U, V)
    assert abs(e_gpu - ref["err"]) <= TOL_ERR[dtype_key], (e_gpu, ref["err"])
    d = orth_defect(U)
    assert d <= orth_bound(U), (d, orth_bound(U))
    res = {"U": U, "V": V, "idx": idx, "err": e_gpu, "ref": ref, "orth": d, "ws": ws}
    if full_rank:
        res["proj"] = projection_distance(X64, U, V, ref["U"], ref["V"])
        print(f"[parity] {tuple(X.shape)} r={rank} {dtype_key}: err gpu {e_gpu:.5f} oracle {ref['err']:.5f} "
              f"projection distance {res['proj']:.2e} (bar {tol_projection(ref['err'], dtype_key):.2e})")
        assert res["proj"] <= tol_projection(ref["err"], dtype_key), (res["proj"], ref["err"])
    if G is not None:
        dW = B.weight_grad(U, V, G)
        rel = np.linalg.norm(to64(dW) - ref["dW"]) / np.linalg.norm(ref["dW"])
        assert rel <= TOL_WGRAD, rel
        res["dW"], res["wgrad_rel"] = dW, rel
    return res
