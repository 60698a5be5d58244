"""Parity at the full sizes of the five configurations, in the launch configuration the benchmark times.
The oracle runs the whole of Algorithm 1 in float64 on the host for each (tens of seconds in total)."""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from paper_2509_23472_b200 import binding as B
from paper_2509_23472_b200 import synth
from tests.parity_util import check_compress, gpu_err, orth_defect, to64, TOL_ERR, TOL_ORTH, TOL_WGRAD
from oracle import loract_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    entry.build()
    return torch.device("cuda:0")


SWEEP = [f"llama13b_s{s}_r{r}" for s in (1024, 2048, 4096, 8192) for r in (64, 128, 256, 512)]


@pytest.mark.parametrize("name", ["llama7b_block", "llama7b_mlp"] + SWEEP)
def test_full_size_configuration(dev, name):
    w = synth.get_workload(name)
    inp = synth.make_inputs(w, device=dev)
    res = check_compress(inp["X"], w.rank, w.seed, G=inp["G"])
    print(f"{name}: err gpu {res['err']:.5f} oracle {res['ref']['err']:.5f} projection distance {res['proj']:.2e} "
          f"orth {res['orth']:.1e} wgrad {res['wgrad_rel']:.1e}")
    del res, inp
    torch.cuda.empty_cache()


def test_vit_prenorm_full_size(dev):
    w = synth.WORKLOADS["vit_b16_prenorm"]
    inp = synth.make_inputs(w, device=dev)
    X, gamma, beta, G = inp["X"], inp["gamma"], inp["beta"], inp["G"]
    A, rstd, mean, U, V, idx = B.compress_prenorm(X, gamma, beta, 1e-5, B.NORM_LAYER, w.rank, seed=w.seed)
    caster = (lambda a: torch.from_numpy(a).bfloat16().double().numpy())
    Ao, rstd_o, mean_o, Uo, Vo, idx_o = orc.compress_prenorm(to64(X), to64(gamma), to64(beta), 1e-5, "layer",
                                                             w.rank, seed=w.seed, in_dtype=caster)
    assert np.array_equal(idx.cpu().numpy().astype(np.int64), idx_o)
    assert np.allclose(to64(rstd), rstd_o, rtol=2e-5)
    err_o = orc.rel_fro_error(Ao, Uo, Vo)
    err_g = gpu_err(A.double(), U, V)
    assert abs(err_g - err_o) <= TOL_ERR["bf16"], (err_g, err_o)
    assert orth_defect(U) <= TOL_ORTH
    dW = B.weight_grad(U, V, G)                      # q, k, v LoRA-A gradients in one call (g = 48)
    ref = orc.weight_grad(Uo, Vo, to64(G))
    assert np.linalg.norm(to64(dW) - ref) / np.linalg.norm(ref) <= TOL_WGRAD
    print(f"vit prenorm: err gpu {err_g:.5f} oracle {err_o:.5f}")
