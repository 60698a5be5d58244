"""Thin ctypes binding of libloract.so.

Argument marshalling only: every step of the path runs in the CUDA kernels of the library.
PyTorch is used for device memory and streams.  There is no CPU fallback: if the library cannot be
loaded, or a tensor is not on a CUDA device, the call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libloract.so")

F32, BF16 = 0, 1
NORM_RMS, NORM_LAYER = 0, 1
DEV_PIVOT_CLAMPED, DEV_WAIT_EXPIRED, DEV_SAMPLER_SHORT, DEV_NONFINITE = 1, 2, 4, 8

EXPORTS = (
    "loract_workspace_bytes", "loract_sample_indices", "loract_compress", "loract_reconstruct",
    "loract_weight_grad", "loract_weight_grad_static", "loract_weight_grad_static_status", "loract_compress_prenorm",
    "loract_prenorm_backward_workspace_bytes", "loract_prenorm_backward", "loract_activation_backward",
    "loract_joint_workspace_bytes", "loract_joint_sample_rows", "loract_joint_sketch", "loract_joint_orthonormalise",
    "loract_joint_project", "loract_joint_finish", "loract_rsvd_workspace_bytes", "loract_rsvd",
    "loract_read_device_status", "loract_status_from_device_word", "loract_status_string",
    "loract_kernel_launch_count",
)


class Desc(ctypes.Structure):
    _fields_ = [("n_tokens", ctypes.c_int64), ("d", ctypes.c_int64), ("ldx", ctypes.c_int64),
                ("rank", ctypes.c_int32), ("power_iters", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("seed", ctypes.c_uint64), ("call_id", ctypes.c_uint64)]


class LoractError(RuntimeError):
    def __init__(self, code: int, what: str):
        extra = ""
        if code == 5:
            try:
                extra = f", cudaError {int(lib().loract_debug_last_cuda_error())}"
            except Exception:
                pass
        super().__init__(f"{what}: status {code} ({status_string(code)}{extra})")
        self.code = code


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the library (building nothing: run ``__graft_entry__.build()`` or ``build.py`` first)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2509_23472_b200.build`")
        l = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        dp = ctypes.POINTER(Desc)
        l.loract_workspace_bytes.restype = sz
        l.loract_workspace_bytes.argtypes = [dp]
        l.loract_sample_indices.restype = ctypes.c_int
        l.loract_sample_indices.argtypes = [dp, vp, vp, sz, vp]
        l.loract_compress.restype = ctypes.c_int
        l.loract_compress.argtypes = [dp, vp, vp, vp, vp, vp, sz, vp]
        l.loract_reconstruct.restype = ctypes.c_int
        l.loract_reconstruct.argtypes = [dp, vp, vp, vp, vp]
        l.loract_weight_grad.restype = ctypes.c_int
        l.loract_weight_grad.argtypes = [dp, vp, vp, vp, i32, i64, vp, ctypes.c_int, vp, sz, vp]
        l.loract_weight_grad_static.restype = ctypes.c_int
        l.loract_weight_grad_static.argtypes = [dp, vp, vp, vp, i32, i64, vp, ctypes.c_int, vp]
        l.loract_weight_grad_static_status.restype = ctypes.c_int
        l.loract_weight_grad_static_status.argtypes = [ctypes.POINTER(ctypes.c_uint32), vp]
        l.loract_compress_prenorm.restype = ctypes.c_int
        l.loract_compress_prenorm.argtypes = [dp, vp, vp, vp, ctypes.c_float, i32, vp, vp, vp, vp, vp, vp,
                                              vp, sz, vp]
        l.loract_prenorm_backward_workspace_bytes.restype = sz
        l.loract_prenorm_backward_workspace_bytes.argtypes = [dp]
        l.loract_prenorm_backward.restype = ctypes.c_int
        l.loract_prenorm_backward.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        l.loract_activation_backward.restype = ctypes.c_int
        l.loract_activation_backward.argtypes = [dp, vp, vp, vp, i32, vp, vp]
        l.loract_joint_workspace_bytes.restype = sz
        l.loract_joint_workspace_bytes.argtypes = [dp]
        l.loract_joint_sample_rows.restype = ctypes.c_int
        l.loract_joint_sample_rows.argtypes = [dp, i64, i64, vp, vp, vp, vp, sz, vp]
        l.loract_joint_sketch.restype = ctypes.c_int
        l.loract_joint_sketch.argtypes = [dp, vp, vp, vp, vp, sz, vp]
        l.loract_joint_orthonormalise.restype = ctypes.c_int
        l.loract_joint_orthonormalise.argtypes = [dp, i32, vp, vp, vp, vp, sz, vp]
        l.loract_joint_project.restype = ctypes.c_int
        l.loract_joint_project.argtypes = [dp, vp, vp, vp, vp, sz, vp]
        l.loract_joint_finish.restype = ctypes.c_int
        l.loract_joint_finish.argtypes = [dp, vp, vp, vp]
        l.loract_rsvd_workspace_bytes.restype = sz
        l.loract_rsvd_workspace_bytes.argtypes = [dp, i32]
        l.loract_rsvd.restype = ctypes.c_int
        l.loract_rsvd.argtypes = [dp, i32, vp, vp, vp, vp, sz, vp]
        l.loract_read_device_status.restype = ctypes.c_int
        l.loract_read_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), vp]
        l.loract_status_from_device_word.restype = ctypes.c_int
        l.loract_status_from_device_word.argtypes = [ctypes.c_uint32]
        l.loract_status_string.restype = ctypes.c_char_p
        l.loract_status_string.argtypes = [ctypes.c_int]
        l.loract_kernel_launch_count.restype = ctypes.c_uint64
        l.loract_kernel_launch_count.argtypes = []
        _lib = l
    return _lib


def status_string(code: int) -> str:
    return lib().loract_status_string(code).decode()


def status_from_device_word(word: int) -> int:
    return int(lib().loract_status_from_device_word(word))


def kernel_launch_count() -> int:
    return int(lib().loract_kernel_launch_count())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _cuda(t: torch.Tensor, what: str) -> torch.Tensor:
    if not t.is_cuda:
        raise RuntimeError(f"{what} must live on a CUDA device (there is no CPU path)")
    return t


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(dev) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(dev).cuda_stream)


def make_desc(X: torch.Tensor, rank: int, seed: int = 0, call_id: int = 0, power_iters: int = 0) -> Desc:
    if X.dim() != 2 or X.stride(1) != 1:
        raise ValueError("X must be a 2-D row-major tensor")
    return Desc(X.shape[0], X.shape[1], X.stride(0), rank, power_iters, _dtype_code(X), 0,
                seed & 0xFFFFFFFFFFFFFFFF, call_id & 0xFFFFFFFFFFFFFFFF)


def desc_for(n_tokens: int, d: int, rank: int, dtype: torch.dtype, seed: int = 0, call_id: int = 0) -> Desc:
    return Desc(n_tokens, d, d, rank, 0, BF16 if dtype == torch.bfloat16 else F32, 0, seed, call_id)


def workspace_bytes(desc: Desc) -> int:
    return int(lib().loract_workspace_bytes(ctypes.byref(desc)))


def alloc_workspace(desc: Desc, device) -> torch.Tensor:
    n = workspace_bytes(desc)
    if n == 0:
        raise LoractError(1, "loract_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def _check(code: int, what: str):
    if code != 0:
        raise LoractError(code, what)


def sample_indices(desc: Desc, device, ws: Optional[torch.Tensor] = None) -> torch.Tensor:
    idx = torch.empty(desc.rank, dtype=torch.int32, device=device)
    ws = ws if ws is not None else torch.empty(256, dtype=torch.uint8, device=device)
    _check(lib().loract_sample_indices(ctypes.byref(desc), _ptr(idx), _ptr(ws), ws.numel(), _stream(device)),
           "loract_sample_indices")
    return idx


def compress(X: torch.Tensor, rank: int, seed: int = 0, call_id: int = 0, ws: Optional[torch.Tensor] = None,
             out: Optional[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]] = None, desc: Optional[Desc] = None,
             power_iters: int = 0):
    """Algorithm 1 with t = power_iters.  Returns (U, V, idx)."""
    _cuda(X, "X")
    desc = desc or make_desc(X, rank, seed, call_id, power_iters)
    ws = ws if ws is not None else alloc_workspace(desc, X.device)
    if out is None:
        U = torch.empty(X.shape[0], rank, dtype=X.dtype, device=X.device)
        V = torch.empty(rank, X.shape[1], dtype=X.dtype, device=X.device)
        idx = torch.empty(rank, dtype=torch.int32, device=X.device)
    else:
        U, V, idx = out
    _check(lib().loract_compress(ctypes.byref(desc), _ptr(X), _ptr(U), _ptr(V), _ptr(idx), _ptr(ws), ws.numel(),
                                 _stream(X.device)), "loract_compress")
    return U, V, idx


def reconstruct(U: torch.Tensor, V: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """X~ = U V."""
    _cuda(U, "U"); _cuda(V, "V")
    n, r = U.shape
    d = V.shape[1]
    out = out if out is not None else torch.empty(n, d, dtype=U.dtype, device=U.device)
    desc = Desc(n, d, out.stride(0), r, 0, _dtype_code(U), 0, 0, 0)
    _check(lib().loract_reconstruct(ctypes.byref(desc), _ptr(U), _ptr(V), _ptr(out), _stream(U.device)),
           "loract_reconstruct")
    return out


def weight_grad(U: torch.Tensor, V: torch.Tensor, G: torch.Tensor, dW: Optional[torch.Tensor] = None,
                accumulate: bool = False, ws: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dW = (U V)^T G from the factors, fp32 (d x g)."""
    _cuda(U, "U"); _cuda(V, "V"); _cuda(G, "G")
    n, r = U.shape
    d = V.shape[1]
    g = G.shape[1]
    if G.stride(1) != 1:
        raise ValueError("G must be row-major")
    desc = Desc(n, d, d, r, 0, _dtype_code(U), 0, 0, 0)
    ws = ws if ws is not None else alloc_workspace(desc, U.device)
    if dW is None:
        dW = torch.zeros(d, g, dtype=torch.float32, device=U.device) if accumulate else \
            torch.empty(d, g, dtype=torch.float32, device=U.device)
    _check(lib().loract_weight_grad(ctypes.byref(desc), _ptr(U), _ptr(V), _ptr(G), g, G.stride(0), _ptr(dW),
                                    1 if accumulate else 0, _ptr(ws), ws.numel(), _stream(U.device)),
           "loract_weight_grad")
    return dW


def weight_grad_static(U: torch.Tensor, V: torch.Tensor, G: torch.Tensor, dW: torch.Tensor,
                       accumulate: bool = False) -> torch.Tensor:
    """dW = (U V)^T G without a workspace: for callers that cannot allocate device memory (a backward hook
    under a locked or exhausted allocator, a fixed memory plan).  The caller passes the output too; the
    intermediate lives in a fixed 1 MiB array inside the library, shared by all calls -- do not overlap
    two of them on the GPU.  Raises LoractError(2) when rank * g exceeds what that array holds."""
    _cuda(U, "U"); _cuda(V, "V"); _cuda(G, "G"); _cuda(dW, "dW")
    n, r = U.shape
    d = V.shape[1]
    g = G.shape[1]
    if G.stride(1) != 1 or dW.shape != (d, g) or dW.dtype != torch.float32 or not dW.is_contiguous():
        raise ValueError("G must be row-major and dW a contiguous fp32 (d x g) tensor")
    desc = Desc(n, d, d, r, 0, _dtype_code(U), 0, 0, 0)
    _check(lib().loract_weight_grad_static(ctypes.byref(desc), _ptr(U), _ptr(V), _ptr(G), g, G.stride(0), _ptr(dW),
                                           1 if accumulate else 0, _stream(U.device)), "loract_weight_grad_static")
    return dW


def weight_grad_static_status(device) -> int:
    """Device status word of the last loract_weight_grad_static call on the current device (0 = clean)."""
    out = ctypes.c_uint32(0)
    _check(lib().loract_weight_grad_static_status(ctypes.byref(out), _stream(device)),
           "loract_weight_grad_static_status")
    return int(out.value)


def compress_prenorm(X: torch.Tensor, gamma: torch.Tensor, beta: Optional[torch.Tensor], eps: float, kind: int,
                     rank: int, seed: int = 0, call_id: int = 0, want_A: bool = True,
                     ws: Optional[torch.Tensor] = None):
    """Pre-norm unit: A = Norm(X), compressed once.  Returns (A or None, rstd, mean or None, U, V, idx)."""
    _cuda(X, "X"); _cuda(gamma, "gamma")
    desc = make_desc(X, rank, seed, call_id)
    ws = ws if ws is not None else alloc_workspace(desc, X.device)
    n, d = X.shape
    A = torch.empty(n, d, dtype=X.dtype, device=X.device) if want_A else None
    rstd = torch.empty(n, dtype=torch.float32, device=X.device)
    mean = torch.empty(n, dtype=torch.float32, device=X.device) if kind == NORM_LAYER else None
    U = torch.empty(n, rank, dtype=X.dtype, device=X.device)
    V = torch.empty(rank, d, dtype=X.dtype, device=X.device)
    idx = torch.empty(rank, dtype=torch.int32, device=X.device)
    _check(lib().loract_compress_prenorm(ctypes.byref(desc), _ptr(X), _ptr(gamma), _ptr(beta), eps, kind, _ptr(A),
                                         _ptr(rstd), _ptr(mean), _ptr(U), _ptr(V), _ptr(idx), _ptr(ws),
                                         ws.numel(), _stream(X.device)), "loract_compress_prenorm")
    return A, rstd, mean, U, V, idx


def prenorm_backward(U: torch.Tensor, V: torch.Tensor, gamma: torch.Tensor, rstd: torch.Tensor,
                     grad_A: torch.Tensor, ws: Optional[torch.Tensor] = None) -> torch.Tensor:
    """grad_X of the RMS pre-norm unit from the compressed normalised activation (Section 3.3)."""
    for t, what in ((U, "U"), (V, "V"), (gamma, "gamma"), (rstd, "rstd"), (grad_A, "grad_A")):
        _cuda(t, what)
    n, r = U.shape
    d = V.shape[1]
    if grad_A.shape != (n, d) or grad_A.stride(1) != 1:
        raise ValueError("grad_A must be a row-major (n_tokens x d) tensor")
    desc = Desc(n, d, grad_A.stride(0), r, 0, _dtype_code(U), 0, 0, 0)
    need = int(lib().loract_prenorm_backward_workspace_bytes(ctypes.byref(desc)))
    if need == 0:
        raise LoractError(1, "loract_prenorm_backward_workspace_bytes")
    ws = ws if ws is not None else torch.empty(need, dtype=torch.uint8, device=U.device)
    grad_X = torch.empty_strided((n, d), (grad_A.stride(0), 1), dtype=grad_A.dtype, device=grad_A.device)
    _check(lib().loract_prenorm_backward(ctypes.byref(desc), _ptr(U), _ptr(V), _ptr(gamma), _ptr(rstd), _ptr(grad_A),
                                         _ptr(grad_X), _ptr(ws), ws.numel(), _stream(U.device)),
           "loract_prenorm_backward")
    return grad_X


ACT_SILU, ACT_GELU = 0, 1


def activation_backward(U: torch.Tensor, V: torch.Tensor, grad_Z: torch.Tensor, kind: int = ACT_SILU) -> torch.Tensor:
    """grad_X = grad_Z * f'(U V) for an element-wise activation whose input was compressed (Section 3.1)."""
    for t, what in ((U, "U"), (V, "V"), (grad_Z, "grad_Z")):
        _cuda(t, what)
    n, r = U.shape
    d = V.shape[1]
    if grad_Z.shape != (n, d) or grad_Z.stride(1) != 1:
        raise ValueError("grad_Z must be a row-major (n_tokens x d) tensor")
    desc = Desc(n, d, grad_Z.stride(0), r, 0, _dtype_code(U), 0, 0, 0)
    grad_X = torch.empty_strided((n, d), (grad_Z.stride(0), 1), dtype=grad_Z.dtype, device=grad_Z.device)
    _check(lib().loract_activation_backward(ctypes.byref(desc), _ptr(U), _ptr(V), _ptr(grad_Z), kind, _ptr(grad_X),
                                            _stream(U.device)), "loract_activation_backward")
    return grad_X


def rsvd(X: torch.Tensor, rank: int, oversample: int = 8, power_iters: int = 1, seed: int = 0, call_id: int = 0,
         ws: Optional[torch.Tensor] = None):
    """Randomized SVD comparator: returns the un-truncated pair (Q (n x l), B (l x d)), l = rank + oversample."""
    _cuda(X, "X")
    desc = make_desc(X, rank, seed, call_id, power_iters)
    d0 = make_desc(X, rank, seed, call_id, 0)
    need = int(lib().loract_rsvd_workspace_bytes(ctypes.byref(d0), oversample))
    if need == 0:
        raise LoractError(1, "loract_rsvd_workspace_bytes")
    ws = ws if ws is not None else torch.empty(need, dtype=torch.uint8, device=X.device)
    l = rank + oversample
    Q = torch.empty(X.shape[0], l, dtype=X.dtype, device=X.device)
    B = torch.empty(l, X.shape[1], dtype=X.dtype, device=X.device)
    _check(lib().loract_rsvd(ctypes.byref(desc), oversample, _ptr(X), _ptr(Q), _ptr(B), _ptr(ws), ws.numel(),
                             _stream(X.device)), "loract_rsvd")
    return Q, B


def read_device_status(ws: torch.Tensor) -> int:
    out = ctypes.c_uint32(0)
    _check(lib().loract_read_device_status(_ptr(ws), ctypes.byref(out), _stream(ws.device)),
           "loract_read_device_status")
    return int(out.value)


# ---------------------------------------------------------------------------------------------
# Test hooks (include/loract_debug.h)
# ---------------------------------------------------------------------------------------------
OUT_F32, OUT_BF16, OUT_SPLIT, OUT_F64 = 0, 1, 2, 3
DEBUG_EXPORTS = ("loract_debug_gemm", "loract_debug_small_block", "loract_debug_set_pair_mode",
                 "loract_debug_last_cuda_error", "loract_debug_trace_begin", "loract_debug_trace_end",
                 "loract_debug_wait_expiry", "loract_debug_project", "loract_debug_gemm_halved",
                 "loract_debug_reduce_sym", "loract_debug_set_round_gate", "loract_debug_round_gate")


def _debug_lib():
    l = lib()
    if not getattr(l, "_debug_ready", False):
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        l.loract_debug_gemm.restype = ctypes.c_int
        l.loract_debug_gemm.argtypes = [i32, i32, i32, i32, i32, ctypes.POINTER(vp), i64, ctypes.POINTER(vp), i64,
                                        i32, i32, i32, i32, vp, vp, i64, i32, i64, i32, i32, vp, vp]
        l.loract_debug_gemm_halved.restype = ctypes.c_int
        l.loract_debug_gemm_halved.argtypes = [i32, i32, i32, i32, i32, ctypes.POINTER(vp), i64, ctypes.POINTER(vp),
                                               i64, i32, i32, i32, i32, i32, vp, vp, i64, i32, i64, i32, i32, vp, vp]
        l.loract_debug_reduce_sym.restype = ctypes.c_int
        l.loract_debug_reduce_sym.argtypes = [vp, i32, i64, i32, vp, vp]
        l.loract_debug_small_block.restype = ctypes.c_int
        l.loract_debug_small_block.argtypes = [i32, vp, i32, i32, i64, i32, ctypes.c_float, vp, vp, vp, vp, vp, vp]
        l.loract_debug_round_gate.restype = ctypes.c_int
        l.loract_debug_round_gate.argtypes = [vp, vp, i32, ctypes.c_float, vp, vp, vp]
        l._debug_ready = True
    return l


def debug_gemm(A_terms, B_terms, M: int, N: int, K: int, a_mn: bool, b_mn: bool, out_mode: int = OUT_F32,
               engine: int = 1, splits: int = 1, acc64: bool = False, status: Optional[torch.Tensor] = None,
               out: Optional[Tuple[torch.Tensor, Optional[torch.Tensor]]] = None, halve_at_term: int = 0):
    """C = sum_t A_t B_t through one of the two contraction kernels.  Operands are 2-D row-major tensors
    stored [M][K] / [K][M] (a_mn) and [N][K] / [K][N] (b_mn).  Returns C (or (hi, lo), or the partials).
    halve_at_term = h > 0: the sum of the terms before h is halved before term h is added."""
    l = _debug_lib()
    dev = A_terms[0].device
    nt = len(A_terms)
    PA = (ctypes.c_void_p * nt)(*[a.data_ptr() for a in A_terms])
    PB = (ctypes.c_void_p * nt)(*[b.data_ptr() for b in B_terms])
    tcode = lambda t: {torch.float32: 0, torch.bfloat16: 1}[t.dtype]
    if out is not None:
        C0, C1 = out          # caller-provided outputs (timing loops: nothing is allocated or cleared here)
    elif out_mode == OUT_F32:
        C0 = torch.zeros(splits, M, N, dtype=torch.float32, device=dev); C1 = None
    elif out_mode == OUT_F64:
        C0 = torch.zeros(splits, M, N, dtype=torch.float64, device=dev); C1 = None
    elif out_mode == OUT_BF16:
        C0 = torch.zeros(M, N, dtype=torch.bfloat16, device=dev); C1 = None
    else:
        C0 = torch.zeros(M, N, dtype=torch.bfloat16, device=dev); C1 = torch.zeros_like(C0)
    _check(l.loract_debug_gemm_halved(M, N, K, int(a_mn), int(b_mn), PA, A_terms[0].stride(0), PB,
                                      B_terms[0].stride(0), tcode(A_terms[0]), tcode(B_terms[0]), nt, halve_at_term,
                                      out_mode, _ptr(C0), _ptr(C1), N, splits, M * N, int(acc64), engine,
                                      _ptr(status), _stream(dev)), "loract_debug_gemm")
    if out_mode in (OUT_F32, OUT_F64):
        return C0 if splits > 1 else C0[0]
    return C0 if C1 is None else (C0, C1)


def debug_reduce_sym(partials: torch.Tensor) -> torch.Tensor:
    """Test hook: S + S^T for S the sum of the (n_partials, r, r) fp32 tensor over its first index."""
    l = _debug_lib()
    n, r, _ = partials.shape
    out = torch.empty(r, r, dtype=torch.float32, device=partials.device)
    _check(l.loract_debug_reduce_sym(_ptr(partials), n, r * r, r, _ptr(out), _stream(partials.device)),
           "loract_debug_reduce_sym")
    return out


def debug_wait_expiry(which: int, limit_ns: int, status: torch.Tensor) -> None:
    """Test hook: a kernel whose bounded wait (0: tensor-core engine, 1: cluster factorisation) runs out after
    limit_ns and ORs DEV_WAIT_EXPIRED into the uint32 `status` tensor."""
    l = _debug_lib()
    l.loract_debug_wait_expiry.restype = ctypes.c_int
    l.loract_debug_wait_expiry.argtypes = [ctypes.c_int32, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_void_p]
    _check(l.loract_debug_wait_expiry(which, limit_ns, _ptr(status), _stream(status.device)),
           "loract_debug_wait_expiry")


def debug_project(desc: Desc, U: torch.Tensor, X: torch.Tensor, V: torch.Tensor, ws: torch.Tensor) -> None:
    """Test / timing hook: V = U^T X exactly as loract_compress runs its last step."""
    l = _debug_lib()
    l.loract_debug_project.restype = ctypes.c_int
    l.loract_debug_project.argtypes = [ctypes.POINTER(Desc)] + [ctypes.c_void_p] * 4 + [ctypes.c_size_t, ctypes.c_void_p]
    _check(l.loract_debug_project(ctypes.byref(desc), _ptr(U), _ptr(X), _ptr(V), _ptr(ws), ws.numel(),
                                  _stream(X.device)), "loract_debug_project")


def debug_set_pair_mode(on: bool) -> None:
    """Test hook: False keeps every contraction on the one-CTA tensor-core kernel."""
    l = _debug_lib()
    l.loract_debug_set_pair_mode.restype = None
    l.loract_debug_set_pair_mode.argtypes = [ctypes.c_int32]
    l.loract_debug_set_pair_mode(1 if on else 0)


def debug_set_round_gate(threshold: float) -> None:
    """Test hook: threshold of the device-side decision to run the second orthonormalisation round (negative: always
    two rounds; inf: one round unless a status bit is set; 0: the default)."""
    l = _debug_lib()
    l.loract_debug_set_round_gate.restype = None
    l.loract_debug_set_round_gate.argtypes = [ctypes.c_float]
    l.loract_debug_set_round_gate(float(threshold))


def debug_round_gate(W: torch.Tensor, linv_hi: torch.Tensor, threshold: float,
                     status: Optional[torch.Tensor] = None):
    """Test hook: the deciding kernel alone.  Returns (second round needed, est, rounds)."""
    l = _debug_lib()
    r = W.shape[0]
    words = torch.zeros(3, dtype=torch.int32, device=W.device)
    _check(l.loract_debug_round_gate(_ptr(W), _ptr(linv_hi), r, ctypes.c_float(threshold), _ptr(status), _ptr(words),
                                     _stream(W.device)), "loract_debug_round_gate")
    w = words.cpu()
    return int(w[0]), float(w[1:2].view(torch.float32).item()), int(w[2])


def round_gate_words(ws: torch.Tensor):
    """(second round ran, estimate trace((D W D)^-1), rounds) of the last orthonormalisation run on workspace `ws`."""
    w = ws[16:28].cpu()
    return int(w[0:4].view(torch.int32).item()), float(w[4:8].view(torch.float32).item()), int(w[8:12].view(torch.int32).item())


def debug_trace_begin(device) -> None:
    l = _debug_lib()
    l.loract_debug_trace_begin.restype = None
    l.loract_debug_trace_begin.argtypes = [ctypes.c_void_p]
    l.loract_debug_trace_begin(_stream(device))


def debug_trace_end(device, max_entries: int = 256):
    """Returns [(label, microseconds), ...] for the kernels launched since debug_trace_begin."""
    l = _debug_lib()
    l.loract_debug_trace_end.restype = ctypes.c_int32
    l.loract_debug_trace_end.argtypes = [ctypes.c_void_p, ctypes.c_char_p, ctypes.POINTER(ctypes.c_float), ctypes.c_int32]
    names = ctypes.create_string_buffer(64 * max_entries)
    us = (ctypes.c_float * max_entries)()
    n = l.loract_debug_trace_end(_stream(device), names, us, max_entries)
    if n < 0:
        raise LoractError(5, "loract_debug_trace_end")
    return [(names.raw[64 * i:64 * (i + 1)].split(b"\0", 1)[0].decode(), float(us[i])) for i in range(n)]


def debug_small_block(partials: torch.Tensor, use_f64: bool, shift_rel: float,
                      status: Optional[torch.Tensor] = None):
    """partials: (n_partials, r, r) fp32 or fp64.  Returns (Linv fp32, hi bf16, lo bf16)."""
    l = _debug_lib()
    dev = partials.device
    n_p, r, _ = partials.shape
    scratch = torch.empty(2 * r * r + 2 * 256 * (256 + max(r - 256, 0) + max(r - 512, 0)) + 64 * r, dtype=torch.float64 if use_f64 else torch.float32,
                          device=dev)
    L32 = torch.zeros(r, r, dtype=torch.float32, device=dev)
    Lh = torch.zeros(r, r, dtype=torch.bfloat16, device=dev)
    Ll = torch.zeros(r, r, dtype=torch.bfloat16, device=dev)
    _check(l.loract_debug_small_block(r, _ptr(partials), int(partials.dtype == torch.float64), n_p, r * r,
                                      int(use_f64), shift_rel, _ptr(scratch), _ptr(L32), _ptr(Lh), _ptr(Ll),
                                      _ptr(status), _stream(dev)), "loract_debug_small_block")
    return L32, Lh, Ll
