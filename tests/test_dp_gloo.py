"""The N > 1 layout of the benchmark on a CPU process group (gloo, world size 2).

The hot path shards by batch with no collective, so what there is to check across ranks is the bookkeeping:
every rank draws a batch and a row sample of its own, rank 0 keeps the single-GPU workload, and the per-rank
times become one whole-job number through a maximum over ranks.  The row samples come from the oracle's
sampler (the device's is checked bit for bit against it in the GPU tests)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import loract_oracle as orc
from paper_2509_23472_b200 import dp, synth


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        base = synth.scaled(synth.get_workload("llama7b_block"), n_tokens=256, d=64, rank=16, signal_rank=32)
        w = dp.rank_workload(base, rank)
        X = synth.make_inputs(w)["X"]
        idx = torch.from_numpy(orc.sample_indices(w.n_tokens, w.rank, w.seed, dp.rank_call_id(rank)).astype(np.int64))
        head = X[:4, :8].float().contiguous()
        idxs = [torch.empty_like(idx) for _ in range(world)]
        heads = [torch.empty_like(head) for _ in range(world)]
        dist.all_gather(idxs, idx)
        dist.all_gather(heads, head)
        # per-rank step times: rank r is the slowest in entry r
        times = [1.0 + (rank == 0), 1.0 + (rank == 1)]
        agg = dp.max_over_ranks(times, dist)
        out[rank] = dict(seed=w.seed, idx_differ=not torch.equal(idxs[0], idxs[1]),
                         data_differ=not torch.equal(heads[0], heads[1]),
                         rank0_is_base=(w.seed == base.seed) if rank == 0 else None, agg=agg,
                         shape=(w.n_tokens, w.d, w.rank))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_get_their_own_batches_and_one_whole_job_number():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = {k: dict(v) for k, v in out.items()}
    assert set(res) == {0, 1}
    assert res[0]["rank0_is_base"] is True
    assert res[1]["seed"] - res[0]["seed"] == dp.SEED_STRIDE
    for r in (0, 1):
        assert res[r]["idx_differ"] and res[r]["data_differ"]
        assert res[r]["agg"] == [2.0, 2.0]            # the maximum over ranks, seen by every rank
        assert res[r]["shape"] == (256, 64, 16)       # weak scaling: the per-rank shape does not change
    # whole-job throughput: both ranks' bytes over the slowest rank's time
    assert dp.whole_job_gbs(2, 10 ** 9, 1000.0) == 2.0
    # without a process group the aggregate is the identity
    assert dp.max_over_ranks([3.0, 1.5]) == [3.0, 1.5]


def test_bench_starts_its_own_ranks_when_run_without_a_launcher():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment starts two ranks itself (through
    torch.distributed.run) and reports n_gpus 2.  --plumbing-only keeps it to what runs without a GPU: rank
    start-up on a gloo group, the barriers, the max over ranks and the whole-job figure."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items()
           if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--plumbing-only"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                              # rank 0 alone prints
    out = json.loads(lines[0])
    base = synth.get_workload("llama7b_block")
    assert out["n_gpus"] == 2 and out["plumbing_only"] is True
    assert out["ms_per_step"] == 2.0                    # the slower rank's time
    assert out["seeds"] == [base.seed, base.seed + dp.SEED_STRIDE] and out["call_ids"] == [0, 1]
    assert out["value"] == dp.whole_job_gbs(2, base.n_tokens * base.d * base.elem_bytes, 2.0)


class _FakeShard:
    """Stands in for joint.JointShard on a CPU process group: every stage hands out a matrix that depends on the
    rank and records what sum it was given, so that the order of the stages and the reductions can be checked."""

    def __init__(self, rank):
        self.rank, self.seen = rank, []
        self.U, self.idx = torch.full((2, 2), float(rank)), torch.arange(2)

    def sample_rows(self):
        return torch.full((2, 3), 1.0 + self.rank)

    def sketch(self, S_sum):
        self.seen.append(("S", S_sum.clone()))
        return torch.full((2, 2), 10.0 * (1 + self.rank))

    def orthonormalise(self, round_, W_sum):
        self.seen.append((f"W{round_}", W_sum.clone()))
        return torch.full((2, 2), 100.0 * (1 + self.rank)) if round_ == 0 else self.U

    def project(self):
        return torch.full((2, 3), 1000.0 * (1 + self.rank))

    def finish(self, V_sum):
        self.seen.append(("V", V_sum.clone()))
        return V_sum


def _joint_worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2509_23472_b200 import joint
        shard = _FakeShard(rank)

        def add(parts):
            t = parts[0].clone()
            dist.all_reduce(t, op=dist.ReduceOp.SUM)
            return t
        joint.run_stages([shard], add)
        out[rank] = [(k, float(v.flatten()[0])) for k, v in shard.seen]
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_joint_compression_stages_reduce_the_right_matrix_at_the_right_time():
    """The stage sequence of the token-sharded compression on two gloo ranks: each stage must be handed the SUM
    over the ranks of what the previous stage produced, in the order rows, Gram 1, Gram 2, V."""
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_joint_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = {k: list(v) for k, v in out.items()}
    want = [("S", 3.0), ("W0", 30.0), ("W1", 300.0), ("V", 3000.0)]
    assert res[0] == want and res[1] == want
