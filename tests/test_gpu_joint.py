"""Joint compression of a token-sharded matrix (loract_joint_*): several shards of ONE matrix, run stage by stage on
one device with their partial matrices added in between, against the float64 oracle on the whole matrix.  The
result must be the factorisation of the whole matrix: the same sampled rows, the same projection."""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from oracle import loract_oracle as orc
from paper_2509_23472_b200 import binding as B
from paper_2509_23472_b200 import joint, synth
from tests.parity_util import TOL_ERR, TOL_ORTH, gpu_err, orth_defect, projection_distance, to64, tol_projection

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    entry.build()
    B.lib()
    return torch.device("cuda:0")


@pytest.mark.parametrize("name,sizes,d,r,R", [
    ("llama7b_block", (1536, 1000, 1560), 1024, 128, 256),    # three uneven shards, ragged tiles
    ("llama7b_block", (4096, 4096), 2048, 256, 512),          # two equal shards
    ("llama13b_s1024_r64", (2048, 640, 2048, 1408), 1024, 64, 256),
    ("llama7b_mlp", (2048, 2048), 2752, 512, 768),            # block small-block scheme
])
def test_sharded_factorisation_is_the_factorisation_of_the_whole_matrix(dev, name, sizes, d, r, R):
    n = sum(sizes)
    w = synth.scaled(synth.get_workload(name), n_tokens=n, d=d, rank=r, signal_rank=R)
    X = synth.make_inputs(w, device=dev)["X"]
    shards_X = list(torch.split(X, list(sizes), dim=0))
    out, shards = joint.joint_compress_shards([x.contiguous() for x in shards_X], r, seed=w.seed, call_id=5)
    torch.cuda.synchronize()
    U = torch.cat([o[0] for o in out], dim=0)
    V, idx = out[0][1], out[0][2]
    for o in out[1:]:
        assert torch.equal(o[1], V) and torch.equal(o[2], idx)         # every shard ends with the same V and rows
    for s in shards:
        assert s.device_status() == 0
    Xd = to64(X)
    Uo, Vo, idx_o = orc.decompose(Xd, r, seed=w.seed, call_id=5)
    assert np.array_equal(idx.cpu().numpy().astype(np.int64), idx_o)    # rows sampled from the whole matrix
    X64 = X.double()
    e_gpu, e_ref = gpu_err(X64, U, V), orc.rel_fro_error(Xd, Uo, Vo)
    assert abs(e_gpu - e_ref) <= TOL_ERR["bf16"], (e_gpu, e_ref)
    assert orth_defect(U) <= TOL_ORTH                                   # U of the whole matrix, not of a shard
    proj = projection_distance(X64, U, V, Uo, Vo)
    assert proj <= tol_projection(e_ref, "bf16"), (proj, e_ref)
    # and it agrees with the one-device call on the whole matrix to the same level
    U1, V1, idx1 = B.compress(X, r, seed=w.seed, call_id=5)
    assert torch.equal(idx1, idx)
    assert abs(gpu_err(X64, U1, V1) - e_gpu) <= 2e-3
    print(f"joint {sizes}: err {e_gpu:.5f} oracle {e_ref:.5f} projection distance {proj:.2e}")


def test_gathered_rows_are_byte_identical_and_a_window_zeroes_the_rest(dev):
    # The gather on its own: with the window covering the whole matrix the staged entry returns exactly
    # X[idx, :] (the bytes, not values within a tolerance); with a window of some rows, the sampled rows outside
    # it come back as zeros, so that the sum over the shards is X[idx, :] again.
    n, d, r = 3000, 776, 96
    g = torch.Generator(device=dev)
    g.manual_seed(11)
    X = torch.randn(n, d, generator=g, device=dev).bfloat16()           # the staged entry points take bf16
    idx_o = orc.sample_indices(n, r, seed=9, call_id=2)
    whole = joint.JointShard(X, n, 0, r, seed=9, call_id=2)
    S = whole.sample_rows()
    torch.cuda.synchronize()
    assert np.array_equal(whole.idx.cpu().numpy().astype(np.int64), idx_o)
    expect = X[torch.as_tensor(idx_o, device=dev)]
    assert torch.equal(S.view(torch.uint8), expect.contiguous().view(torch.uint8))
    row0, n_local = 1000, 1200
    part = joint.JointShard(X[row0:row0 + n_local].contiguous(), n, row0, r, seed=9, call_id=2)
    Sp = part.sample_rows()
    torch.cuda.synchronize()
    inside = torch.as_tensor((idx_o >= row0) & (idx_o < row0 + n_local), device=dev)
    assert 0 < int(inside.sum()) < r                                    # the case has rows on both sides
    assert torch.equal(Sp[inside].view(torch.uint8), expect[inside].contiguous().view(torch.uint8))
    assert not bool(Sp[~inside].view(torch.uint8).any())


def test_joint_rejects_bad_arguments_before_launching(dev):
    X = torch.zeros(512, 256, dtype=torch.bfloat16, device=dev)
    before = B.kernel_launch_count()
    with pytest.raises(B.LoractError):
        joint.JointShard(X, 256, 0, 64).sample_rows()          # the whole matrix cannot be smaller than the shard
    with pytest.raises(B.LoractError):
        joint.JointShard(X, 2048, 1800, 64).sample_rows()      # the shard would end past the last row
    with pytest.raises(B.LoractError):
        joint.JointShard(X.float(), 512, 0, 64)                # bf16 only
    assert B.kernel_launch_count() == before
