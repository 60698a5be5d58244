"""Joint compression of ONE activation matrix whose token rows are sharded over several GPUs.

Algorithm 1 at t = 0 as one factorisation of the whole matrix (sequence / context parallelism): every shard runs
the stages of ``loract_joint_*`` (include/loract.h) on its own rows, and between the stages the small matrices
are added over the shards -- the sampled rows (rank x d), two rank x rank Gram matrices, V (rank x d).  All
arithmetic is in the library's kernels; this module marshals arguments and calls the reduction in between.

``JointShard`` is one shard's side.  ``joint_compress`` runs a rank's shard inside a torch.distributed process
group (NCCL all-reduce; received data lands in local memory before the next kernel reads it).
``joint_compress_shards`` runs several shards of one matrix on ONE device, stage by stage, adding the partial
matrices itself in shard order: the same arithmetic without a process group, which is how the path is tested
where only one GPU is at hand.
"""
from __future__ import annotations

import ctypes
from typing import Callable, List, Sequence

import torch

from . import binding as B


class JointShard:
    """The rows [row0, row0 + n_local) of an (n_global x d) bf16 matrix, and the stages it runs."""

    def __init__(self, X_local: torch.Tensor, n_global: int, row0: int, rank: int, seed: int = 0, call_id: int = 0):
        if not X_local.is_cuda or X_local.dim() != 2 or X_local.stride(1) != 1:
            raise ValueError("X_local must be a row-major matrix on a CUDA device (there is no CPU path)")
        self.X, self.n_global, self.row0, self.r = X_local, int(n_global), int(row0), int(rank)
        self.dev = X_local.device
        n, d = X_local.shape
        self.desc = B.make_desc(X_local, rank, seed, call_id)
        need = int(B.lib().loract_joint_workspace_bytes(ctypes.byref(self.desc)))
        if need == 0:
            raise B.LoractError(1, "loract_joint_workspace_bytes")
        self.ws = torch.empty(need, dtype=torch.uint8, device=self.dev)
        self.S = torch.empty(rank, d, dtype=X_local.dtype, device=self.dev)
        self.idx = torch.empty(rank, dtype=torch.int32, device=self.dev)
        self.W = torch.empty(rank, rank, dtype=torch.float32, device=self.dev)
        self.U = torch.empty(n, rank, dtype=torch.bfloat16, device=self.dev)
        self.Vp = torch.empty(rank, d, dtype=torch.float32, device=self.dev)
        self.V = torch.empty(rank, d, dtype=torch.bfloat16, device=self.dev)

    def _args(self):
        return B._ptr(self.ws), self.ws.numel(), B._stream(self.dev)

    def sample_rows(self) -> torch.Tensor:
        B._check(B.lib().loract_joint_sample_rows(ctypes.byref(self.desc), self.n_global, self.row0, B._ptr(self.X),
                                                  B._ptr(self.S), B._ptr(self.idx), *self._args()),
                 "loract_joint_sample_rows")
        return self.S

    def sketch(self, S_sum: torch.Tensor) -> torch.Tensor:
        B._check(B.lib().loract_joint_sketch(ctypes.byref(self.desc), B._ptr(self.X), B._ptr(S_sum), B._ptr(self.W),
                                             *self._args()), "loract_joint_sketch")
        return self.W

    def orthonormalise(self, round_: int, W_sum: torch.Tensor) -> torch.Tensor:
        """Round 0 returns the shard's second Gram matrix (in the buffer W_sum is NOT aliased with), round 1 U."""
        out = self.W if round_ == 0 else None
        B._check(B.lib().loract_joint_orthonormalise(ctypes.byref(self.desc), round_, B._ptr(W_sum), B._ptr(out),
                                                     B._ptr(self.U) if round_ == 1 else None, *self._args()),
                 "loract_joint_orthonormalise")
        return self.W if round_ == 0 else self.U

    def project(self) -> torch.Tensor:
        B._check(B.lib().loract_joint_project(ctypes.byref(self.desc), B._ptr(self.U), B._ptr(self.X),
                                              B._ptr(self.Vp), *self._args()), "loract_joint_project")
        return self.Vp

    def finish(self, V_sum: torch.Tensor) -> torch.Tensor:
        B._check(B.lib().loract_joint_finish(ctypes.byref(self.desc), B._ptr(V_sum), B._ptr(self.V),
                                             B._stream(self.dev)), "loract_joint_finish")
        return self.V

    def device_status(self) -> int:
        return B.read_device_status(self.ws)


def run_stages(shards: Sequence[JointShard], add: Callable[[List[torch.Tensor]], torch.Tensor]):
    """The stage sequence for the shards this process holds.  `add` takes the shards' partial matrices of one
    stage and returns their sum over ALL shards of the matrix (a new tensor every shard may read)."""
    S_sum = add([s.sample_rows() for s in shards])
    W1 = add([s.sketch(S_sum) for s in shards])
    W2 = add([s.orthonormalise(0, W1) for s in shards])
    for s in shards:
        s.orthonormalise(1, W2)
    V_sum = add([s.project() for s in shards])
    return [(s.U, s.finish(V_sum), s.idx) for s in shards]


def sum_in_order(parts: List[torch.Tensor]) -> torch.Tensor:
    """The partial matrices of the shards held by this process, added in shard order (float32 for the bf16 rows:
    every row has one non-zero contribution, so the sum is exact)."""
    acc = parts[0].float().clone()
    for p in parts[1:]:
        acc += p.float()
    return acc.to(parts[0].dtype)


def joint_compress_shards(X_shards: Sequence[torch.Tensor], rank: int, seed: int = 0, call_id: int = 0):
    """Several shards of one matrix on one device (no process group): returns [(U_shard, V, idx), ...]; V and idx
    are the same for every shard.  The concatenation of the U_shard is the U of the whole matrix."""
    n_global = sum(int(x.shape[0]) for x in X_shards)
    shards, row0 = [], 0
    for x in X_shards:
        shards.append(JointShard(x, n_global, row0, rank, seed, call_id))
        row0 += int(x.shape[0])
    return run_stages(shards, sum_in_order), shards


def joint_compress(X_local: torch.Tensor, n_global: int, row0: int, rank: int, seed: int = 0, call_id: int = 0,
                   group=None):
    """This process's shard inside an initialised torch.distributed group: returns (U_local, V, idx)."""
    import torch.distributed as dist
    shard = JointShard(X_local, n_global, row0, rank, seed, call_id)

    def add(parts):
        t = parts[0].clone()
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
        return t
    (out,) = run_stages([shard], add)
    return out
