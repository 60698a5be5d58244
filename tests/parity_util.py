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


def check_compress(X, rank, seed, call_id=0, G=None, dtype_key="bf16", ws=None, require_status=0):
    """Runs loract_compress (+ weight_grad) and the oracle; asserts the parity statement; returns both."""
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
    if G is not None:
        dW = B.weight_grad(U, V, G)
        rel = np.linalg.norm(to64(dW) - ref["dW"]) / np.linalg.norm(ref["dW"])
        assert rel <= TOL_WGRAD, rel
        res["dW"], res["wgrad_rel"] = dW, rel
    return res
