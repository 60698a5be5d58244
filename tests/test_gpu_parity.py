"""GPU parity tests: the CUDA path against the float64 oracle, through the C ABI, on the same seeded inputs.

Bars: sampled indices bit-exact; |err_gpu - err_oracle| <= 2e-2 (bf16) / 1e-4 (fp32) for the relative
Frobenius reconstruction error; max|U^T U - I| <= 1e-3; weight-gradient relative error <= 2e-2.
"""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from oracle import loract_oracle as orc
from paper_2509_23472_b200 import binding as B
from paper_2509_23472_b200 import synth
from tests.parity_util import (TOL_ERR, TOL_ORTH, TOL_WGRAD, check_compress, gpu_err, oracle_run, orth_bound,
                               orth_defect, to64)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    entry.build()
    B.lib()
    return torch.device("cuda:0")


# ------------------------------------------------------------------ sampler
@pytest.mark.parametrize("n,r,seed,call", [(512, 64, 0, 0), (12608, 96, 1, 7), (16384, 256, 2, 0),
                                           (32768, 512, 9, 1 << 33), (512, 512, 3, 0), (96, 96, 5, 5),
                                           (100000, 16, (1 << 40) + 5, 3), (17, 16, 0, 0)])
def test_sampled_rows_are_bit_identical_to_the_oracle(dev, n, r, seed, call):
    desc = B.desc_for(n, max(r, 64), r, torch.bfloat16, seed, call)
    idx = B.sample_indices(desc, dev).cpu().numpy().astype(np.int64)
    assert np.array_equal(idx, orc.sample_indices(n, r, seed, call))


# ------------------------------------------------------------------ the small fp32 configuration, full size
def test_small_f32_configuration_full(dev):
    w = synth.WORKLOADS["small_f32"]
    inp = synth.make_inputs(w, device=dev)
    res = check_compress(inp["X"], w.rank, w.seed, G=inp["G"], dtype_key="f32")
    # the reconstruction entry point returns U V
    Xr = B.reconstruct(res["U"], res["V"])
    ref = res["U"].double() @ res["V"].double()
    assert float((Xr.double() - ref).abs().max()) <= 1e-5 * float(ref.abs().max())
    # the residual is orthogonal to the basis and V = U^T X, as for the oracle
    X64 = inp["X"].double()
    assert float((res["U"].double().t() @ (X64 - ref)).abs().max()) <= 1e-3
    assert res["wgrad_rel"] <= 1e-3


# ------------------------------------------------------------------ reduced bf16 shapes: several tiles + ragged tails
@pytest.mark.parametrize("name,n,d,r,R", [
    ("llama7b_block", 1000, 520, 48, 96),      # ragged token tile, d not a multiple of 64
    ("llama7b_block", 2176, 1024, 128, 256),   # 17 token tiles
    ("vit_b16_prenorm", 788, 768, 96, 128),    # 4 images x 197 tokens
    ("llama7b_mlp", 1536, 2752, 272, 512),     # r not a multiple of 64, two accumulator tiles
    ("llama7b_block", 384, 4096, 256, 512),    # short and wide
    ("llama7b_block", 4100, 264, 16, 32),      # smallest rank
])
def test_reduced_bf16_shapes(dev, name, n, d, r, R):
    w = synth.scaled(synth.WORKLOADS[name], n_tokens=n, d=d, rank=r, signal_rank=R)
    inp = synth.make_inputs(w, device=dev)
    res = check_compress(inp["X"], r, w.seed, call_id=3, G=inp["G"])
    Xr = B.reconstruct(res["U"], res["V"])
    ref = res["U"].double() @ res["V"].double()
    assert float(torch.linalg.norm(Xr.double() - ref) / torch.linalg.norm(ref)) <= 4e-3   # bf16 output rounding
    # V is the projection coefficient matrix of the stored U
    Vref = res["U"].double().t() @ inp["X"].double()
    assert float(torch.linalg.norm(res["V"].double() - Vref) / torch.linalg.norm(Vref)) <= 4e-3


def test_row_stride_larger_than_d_and_determinism(dev):
    w = synth.scaled(synth.WORKLOADS["llama7b_block"], n_tokens=900, d=512, rank=64, signal_rank=128)
    X = synth.make_inputs(w, device=dev)["X"]
    wide = torch.zeros(900, 640, dtype=X.dtype, device=dev)
    wide[:, :512] = X
    Xs = wide[:, :512]                       # ldx = 640
    U1, V1, i1 = B.compress(Xs, 64, seed=5)
    U2, V2, i2 = B.compress(X, 64, seed=5)
    U3, V3, i3 = B.compress(X, 64, seed=5)
    assert torch.equal(i1, i2) and torch.equal(U1, U2) and torch.equal(V1, V2)
    assert torch.equal(U2, U3) and torch.equal(V2, V3)           # run-to-run bitwise determinism
    out = torch.full((900, 640), 7.0, dtype=X.dtype, device=dev)
    B.reconstruct(U1, V1, out=out[:, :512])
    assert torch.all(out[:, 512:] == 7.0)                        # nothing written past d


# ------------------------------------------------------------------ edge cases
def test_all_rows_sampled_is_exact_up_to_storage_rounding(dev):
    w = synth.scaled(synth.WORKLOADS["llama7b_block"], n_tokens=64, d=512, rank=64, signal_rank=128)
    X = synth.make_inputs(w, device=dev)["X"]
    res = check_compress(X, 64, seed=1, full_rank=False)     # r = N: the projection is the identity
    assert sorted(res["idx"].cpu().tolist()) == list(range(64))
    assert res["err"] <= 6e-3      # only the bf16 rounding of U and V is left


def test_exactly_low_rank_input_is_recovered(dev):
    # rank(A) <= k: the projection error is zero in exact arithmetic (proof of Theorem 3.3)
    X64 = synth.exact_low_rank(1500, 384, 24, seed=3, device=dev)
    Xf = X64.float()
    res = check_compress(Xf, 32, seed=2, dtype_key="f32", require_status=None, full_rank=False)
    assert res["err"] <= 2e-5
    Xb = X64.bfloat16()            # rounding makes it full rank again at the 2^-9 level
    res = check_compress(Xb, 32, seed=2, require_status=None, full_rank=False)
    assert gpu_err(X64, res["U"], res["V"]) <= 8e-3


@pytest.mark.parametrize("n,d,r", [(16, 16, 16), (64, 16, 16), (16, 64, 16), (32, 32, 16), (128, 128, 16),
                                   (48, 48, 48), (130, 72, 16)])
def test_smallest_problems(dev, n, d, r):
    gen = torch.Generator(device=dev); gen.manual_seed(n + d)
    X = torch.randn(n, d, generator=gen, device=dev).bfloat16()
    res = check_compress(X, r, seed=0, require_status=None, full_rank=r < min(n, d))
    if r == min(n, d):
        assert res["err"] <= 8e-3          # full rank kept: only storage rounding is left


def test_zero_input_returns_finite_factors(dev):
    X = torch.zeros(300, 128, dtype=torch.bfloat16, device=dev)
    U, V, idx = B.compress(X, 32, seed=0)
    assert torch.isfinite(U.float()).all() and torch.isfinite(V.float()).all()
    assert float(B.reconstruct(U, V).float().abs().max()) == 0.0


# ------------------------------------------------------------------ weight gradient
@pytest.mark.parametrize("g,pad", [(16, 0), (48, 0), (96, 32), (8, 0), (256, 0)])
def test_weight_grad_shapes_and_accumulate(dev, g, pad):
    w = synth.scaled(synth.WORKLOADS["llama7b_block"], n_tokens=3000, d=768, rank=64, signal_rank=128)
    X = synth.make_inputs(w, device=dev)["X"]
    U, V, _ = B.compress(X, 64, seed=1)
    gen = torch.Generator(device=dev); gen.manual_seed(g)
    Gw = torch.randn(3000, g + pad, generator=gen, device=dev).bfloat16()
    G = Gw[:, :g]
    ref = orc.weight_grad(to64(U), to64(V), to64(G))        # the oracle's formula on the same factors
    dW = B.weight_grad(U, V, G)
    assert dW.shape == (768, g) and dW.dtype == torch.float32
    assert np.linalg.norm(to64(dW) - ref) / np.linalg.norm(ref) <= 1e-3
    dW2 = B.weight_grad(U, V, G, dW=dW.clone(), accumulate=True)
    assert np.linalg.norm(to64(dW2) - 2 * ref) / np.linalg.norm(ref) <= 2e-3
    # against the gradient at the uncompressed activation it is only as good as the compression
    full = to64(X).T @ to64(G)
    assert np.linalg.norm(to64(dW) - full) / np.linalg.norm(full) <= 1.0


# ------------------------------------------------------------------ pre-norm unit
@pytest.mark.parametrize("kind,dtype", [("layer", torch.bfloat16), ("rms", torch.bfloat16), ("rms", torch.float32)])
def test_prenorm_entry(dev, kind, dtype):
    base = synth.WORKLOADS["vit_b16_prenorm"]
    w = synth.scaled(base, n_tokens=4 * 197, d=768, rank=96 if dtype == torch.bfloat16 else 64, signal_rank=128)
    inp = synth.make_inputs(w, device=dev)
    X = inp["X"].to(dtype)
    gamma = inp["gamma"].to(dtype)
    beta = inp["beta"].to(dtype) if kind == "layer" else None
    eps = 1e-5 if kind == "layer" else 1e-6
    code = B.NORM_LAYER if kind == "layer" else B.NORM_RMS
    A, rstd, mean, U, V, idx = B.compress_prenorm(X, gamma, beta, eps, code, w.rank, seed=w.seed)
    Ao, rstd_o, mean_o = orc.norm_forward(to64(X), to64(gamma), None if beta is None else to64(beta), eps, kind)
    assert np.allclose(to64(rstd), rstd_o, rtol=2e-5)
    if kind == "layer":
        assert np.allclose(to64(mean), mean_o, rtol=1e-4, atol=1e-6)
    ulp = 2.0 ** -8 if dtype == torch.bfloat16 else 2.0 ** -22
    assert np.max(np.abs(to64(A) - Ao) / (np.abs(Ao) + 1e-3)) <= 2 * ulp
    # the factor pair compresses the normalised input: same rows, same error level as the oracle on its own A
    caster = (lambda a: torch.from_numpy(a).to(dtype).double().numpy())
    _, _, _, Uo, Vo, idx_o = orc.compress_prenorm(to64(X), to64(gamma), None if beta is None else to64(beta), eps,
                                                  kind, w.rank, seed=w.seed, in_dtype=caster)
    assert np.array_equal(idx.cpu().numpy().astype(np.int64), idx_o)
    err_o = orc.rel_fro_error(caster(Ao), Uo, Vo)
    err_g = gpu_err(A.double(), U, V)
    assert abs(err_g - err_o) <= TOL_ERR["bf16" if dtype == torch.bfloat16 else "f32"]
    assert orth_defect(U) <= orth_bound(U)
    # without A_out the normalised matrix lives in the workspace only: same factors
    A2, _, _, U2, V2, _ = B.compress_prenorm(X, gamma, beta, eps, code, w.rank, seed=w.seed, want_A=False)
    assert A2 is None and torch.equal(U2, U) and torch.equal(V2, V)
    # one compression serves every consumer: q/k/v gradients in one call equal three separate calls
    G = inp["G"].to(dtype)
    dW = B.weight_grad(U, V, G)
    parts = [B.weight_grad(U, V, G[:, 16 * i:16 * (i + 1)].contiguous()) for i in range(3)]
    assert torch.allclose(dW, torch.cat(parts, dim=1), rtol=1e-4, atol=1e-4 * float(dW.abs().max()))
    ref = orc.weight_grad(Uo, Vo, to64(G))
    assert np.linalg.norm(to64(dW) - ref) / np.linalg.norm(ref) <= TOL_WGRAD


# ------------------------------------------------------------------ RSVD comparator
def test_rsvd_comparator(dev):
    """Oversample 8, one power iteration, cut to rank r: the comparator as the workloads define it."""
    from paper_2509_23472_b200 import report
    w = synth.scaled(synth.llama13b_sweep_point(1024, 64), n_tokens=2048, d=1024, rank=64, signal_rank=256)
    X = synth.make_inputs(w, device=dev)["X"]
    Q, Bm = B.rsvd(X, 64, oversample=8, power_iters=1, seed=3)
    assert Q.shape == (2048, 72) and Bm.shape == (72, 1024)
    assert orth_defect(Q) <= TOL_ORTH
    X64 = X.double()
    Xd = to64(X)
    e_l = gpu_err(X64, Q, Bm)
    errs = [orc.rel_fro_error(Xd, *orc.rsvd(Xd, 64, 8, 1, seed=s, truncate=False)) for s in range(2)]
    assert e_l >= orc.rel_fro_error(Xd, *orc.truncated_svd(Xd, 72)) - 1e-3     # Eckart-Young at rank l
    assert abs(e_l - np.mean(errs)) <= 2e-2          # different Gaussian draws, same error level
    # cut to rank r: the equal-rank error, against the oracle's truncated form
    Qr, Br = report.truncate_to_rank(Q, Bm, 64)
    assert Qr.shape == (2048, 64) and Br.shape == (64, 1024)
    e_r = gpu_err(X64, Qr, Br)
    errs_r = [orc.rel_fro_error(Xd, *orc.rsvd(Xd, 64, 8, 1, seed=s, truncate=True)) for s in range(2)]
    opt = orc.rel_fro_error(Xd, *orc.truncated_svd(Xd, 64))
    assert e_r >= opt - 1e-3                          # Eckart-Young at rank r
    assert e_r >= e_l - 1e-3                          # cutting columns cannot help
    assert abs(e_r - np.mean(errs_r)) <= 2e-2
    # a power iteration does not hurt
    Q0, B0 = B.rsvd(X, 64, oversample=8, power_iters=0, seed=3)
    assert e_l <= gpu_err(X64, Q0, B0) + 2e-3


@pytest.mark.parametrize("r", [128, 256, 512])
def test_rsvd_comparator_oversampled_ranks(dev, r):
    # l = r + 8 at the ranks of the sweep: 136 (one accumulator tile, ragged), 264 and 520 (block small-block scheme)
    w = synth.scaled(synth.llama13b_sweep_point(1024, r), n_tokens=3072, d=1024, rank=r, signal_rank=768 if r == 512 else 512)
    X = synth.make_inputs(w, device=dev)["X"]
    Q, Bm = B.rsvd(X, r, oversample=8, power_iters=1, seed=4)
    assert Q.shape == (3072, r + 8)
    assert orth_defect(Q) <= TOL_ORTH
    Xd = to64(X)
    e_gpu = gpu_err(X.double(), Q, Bm)
    e_orc = orc.rel_fro_error(Xd, *orc.rsvd(Xd, r, 8, 1, seed=0, truncate=False))
    assert abs(e_gpu - e_orc) <= TOL_ERR["bf16"], (e_gpu, e_orc)


def test_rsvd_comparator_at_the_largest_test_matrix(dev):
    # l = 512 Gaussian test vectors (the largest the library takes: the two-level small-block route) and one
    # power iteration, on the long-context sweep's spectrum at a reduced width.  The iteration's test matrix
    # Q^T X is brought back to near-orthonormal rows before it multiplies X again; without that the sketch
    # carries the cube of the spectrum into a Gram matrix and the factors come out non-finite.
    w = synth.scaled(synth.llama13b_sweep_point(1024, 512), n_tokens=4096, d=2048, rank=512, signal_rank=768)
    X = synth.make_inputs(w, device=dev)["X"]
    Q, Bm = B.rsvd(X, 512, oversample=0, power_iters=1, seed=5)
    assert Q.shape == (4096, 512) and bool(torch.isfinite(Q.float()).all()) and bool(torch.isfinite(Bm.float()).all())
    assert orth_defect(Q) <= TOL_ORTH
    Xd = to64(X)
    e_gpu = gpu_err(X.double(), Q, Bm)
    e_orc = orc.rel_fro_error(Xd, *orc.rsvd(Xd, 512, 0, 1, seed=0, truncate=False))
    assert abs(e_gpu - e_orc) <= TOL_ERR["bf16"]


# ------------------------------------------------------------------ power iterations (the loop of Algorithm 1)
@pytest.mark.parametrize("t", [1, 2])
def test_power_iterations_match_the_oracle_and_help_on_a_flat_spectrum(dev, t):
    # a slowly decaying spectrum with strong noise: the regime in which the loop of Algorithm 1 pays
    w = synth.scaled(synth.get_workload("llama13b_s1024_r64"), n_tokens=2048, d=1024, rank=64, signal_rank=256)
    X = synth.make_inputs(w, device=dev)["X"]
    X64 = X.double()
    Xd = to64(X)
    errs = {}
    for tt in (0, t):
        U, V, idx = B.compress(X, 64, seed=w.seed, power_iters=tt)
        torch.cuda.synchronize()
        Uo, Vo, io = orc.decompose(Xd, 64, t=tt, seed=w.seed)
        assert np.array_equal(idx.cpu().numpy().astype(np.int64), io)
        e_gpu, e_ref = gpu_err(X64, U, V), orc.rel_fro_error(Xd, Uo, Vo)
        assert abs(e_gpu - e_ref) <= TOL_ERR["bf16"], (tt, e_gpu, e_ref)
        assert orth_defect(U) <= orth_bound(U)
        errs[tt] = (e_gpu, e_ref)
    # the loop must not make things worse, on either side (it improves the oracle's error on this input)
    assert errs[t][1] <= errs[0][1] + 1e-12
    assert errs[t][0] <= errs[0][0] + 2e-3


def test_power_iterations_fp32(dev):
    w = synth.scaled(synth.WORKLOADS["small_f32"], n_tokens=384, d=256, rank=32, signal_rank=96)
    X = synth.make_inputs(w, device=dev)["X"]
    Xd = to64(X)
    U, V, idx = B.compress(X, 32, seed=w.seed, power_iters=2)
    torch.cuda.synchronize()
    Uo, Vo, io = orc.decompose(Xd, 32, t=2, seed=w.seed)
    assert np.array_equal(idx.cpu().numpy().astype(np.int64), io)
    assert abs(gpu_err(X.double(), U, V) - orc.rel_fro_error(Xd, Uo, Vo)) <= TOL_ERR["f32"]
    assert orth_defect(U) <= TOL_ORTH


# ------------------------------------------------------------------ coherent inputs
def test_private_outlier_tokens_need_one_power_iteration(dev):
    """A few token rows carry large components nobody else has (high coherence).  Uniform row sampling at
    t = 0 misses them on both sides; one pass of the loop of Algorithm 1 (t = 1) recovers them, on both sides."""
    w = synth.scaled(synth.get_workload("llama13b_s1024_r64"), n_tokens=2048, d=1024, rank=64, signal_rank=48)
    X = synth.plant_private_outliers(synth.make_inputs(w, device=dev)["X"], n_out=8, scale=400.0, seed=123)
    X64, Xd = X.double(), to64(X)
    got = {}
    for t in (0, 1):
        U, V, idx = B.compress(X, 64, seed=w.seed, power_iters=t)
        torch.cuda.synchronize()
        Uo, Vo, io = orc.decompose(Xd, 64, t=t, seed=w.seed)
        assert np.array_equal(idx.cpu().numpy().astype(np.int64), io)
        got[t] = (gpu_err(X64, U, V), orc.rel_fro_error(Xd, Uo, Vo))
        assert abs(got[t][0] - got[t][1]) <= TOL_ERR["bf16"], (t, got[t])
        assert orth_defect(U) <= orth_bound(U, spiky=True)   # t = 1: basis vectors sit on single rows
    assert got[0][1] > 0.5 and got[0][0] > 0.5          # the sample cannot see the private components
    assert got[1][1] < 0.1 and got[1][0] < 0.1 + TOL_ERR["bf16"]   # one iteration finds them


# ------------------------------------------------------------------ pre-norm unit, backward (Section 3.3)
@pytest.mark.parametrize("n,d,r", [(1024, 512, 64), (1000, 768, 96), (4096, 1024, 256), (2048, 1024, 512)])
def test_prenorm_backward_matches_the_three_gradient_equations(dev, n, d, r):
    w = synth.scaled(synth.WORKLOADS["llama7b_block"], n_tokens=n, d=d, rank=r, signal_rank=min(2 * r, d // 2))
    w = synth.Workload(**{**w.__dict__, "prenorm": "rms"})
    inp = synth.make_inputs(w, device=dev)
    X, gamma = inp["X"], inp["gamma"]
    A, rstd, _, U, V, idx = B.compress_prenorm(X, gamma, None, 1e-6, B.NORM_RMS, r, seed=w.seed)
    g = torch.Generator(device=dev)
    g.manual_seed(77)
    gA = torch.randn(n, d, generator=g, device=dev).to(X.dtype)
    gX = B.prenorm_backward(U, V, gamma, rstd, gA)
    torch.cuda.synchronize()
    # the oracle's equations on the same stored factors: this isolates the backward step
    A_tilde = to64(U) @ to64(V)
    want = orc.prenorm_backward_rms(A_tilde, to64(gamma), to64(rstd), to64(gA))
    rel = np.linalg.norm(to64(gX) - want) / np.linalg.norm(want)
    assert rel <= 1e-2, rel                     # bf16 output: 2^-9 per entry
    # and against the exact (uncompressed) gradient the difference is the compression error, not more
    exact = orc.prenorm_backward_rms(to64(A), to64(gamma), to64(rstd), to64(gA))
    err_A = np.linalg.norm(A_tilde - to64(A)) / np.linalg.norm(to64(A))
    rel_exact = np.linalg.norm(to64(gX) - exact) / np.linalg.norm(exact)
    assert rel_exact <= 2.0 * err_A + 1e-2, (rel_exact, err_A)


# ------------------------------------------------------------------ element-wise consumer (Section 3.1)
@pytest.mark.parametrize("kind,name", [(B.ACT_SILU, "silu"), (B.ACT_GELU, "gelu")])
@pytest.mark.parametrize("n,d,r", [(1024, 512, 64), (1000, 776, 96), (4096, 2048, 256), (2048, 1024, 512)])
def test_activation_backward_matches_the_gradient_equation(dev, kind, name, n, d, r):
    """grad_X = grad_Z * f'(A~) with A~ = U V never stored: the device against the oracle's equation on the same
    stored factors (this isolates the consumer), and against the exact gradient at the uncompressed input."""
    w = synth.scaled(synth.WORKLOADS["llama7b_block"], n_tokens=n, d=d, rank=r, signal_rank=min(2 * r, d // 2))
    X = synth.make_inputs(w, device=dev)["X"]
    X = (X.float() * (2.0 / float(X.float().std()))).to(X.dtype)      # entries of a few units: f' is not flat there
    U, V, _ = B.compress(X, r, seed=w.seed)
    g = torch.Generator(device=dev)
    g.manual_seed(91)
    gZ = torch.randn(n, d, generator=g, device=dev).to(X.dtype)
    gX = B.activation_backward(U, V, gZ, kind)
    torch.cuda.synchronize()
    assert gX.shape == (n, d) and gX.dtype == X.dtype
    A_tilde = to64(U) @ to64(V)
    want = orc.activation_backward(A_tilde, to64(gZ), name)
    rel = np.linalg.norm(to64(gX) - want) / np.linalg.norm(want)
    assert rel <= 1e-2, rel                     # bf16 output: 2^-9 per entry
    exact = orc.activation_backward(to64(X), to64(gZ), name)
    err_A = np.linalg.norm(A_tilde - to64(X)) / np.linalg.norm(to64(X))
    rel_exact = np.linalg.norm(to64(gX) - exact) / np.linalg.norm(exact)
    assert rel_exact <= 2.0 * err_A + 1e-2, (rel_exact, err_A)   # |f''| <= 1/2: the compression error, not more
    # a row stride larger than d, and nothing written past d
    wide_in = torch.zeros(n, d + 64, dtype=X.dtype, device=dev)
    wide_in[:, :d] = gZ
    out = B.activation_backward(U, V, wide_in[:, :d], kind)
    assert out.stride(0) == d + 64 and torch.equal(out, gX)
