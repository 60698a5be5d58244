"""GPU tests of the tensor-core contraction behind the sketch and the projection of Algorithm 1, the Gram products and
Reconstruct: C = sum_t A_t B_t with bf16 operands and fp32 accumulation, for every operand major, with
ragged shapes, split-K partials and the bf16 hi/lo output -- in both forms of the kernel (one CTA per
128-row tile, and a pair of CTAs per 256-row tile).  The reference is the definition, evaluated in float64
on the same bf16 inputs."""
import pytest
import torch

import __graft_entry__ as entry
from paper_2509_23472_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    entry.build()
    B.lib()
    yield torch.device("cuda:0")
    B.debug_set_pair_mode(True)


def operands(M, N, K, a_mn, b_mn, n_terms, dev, seed):
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    As = [torch.randn((K, M) if a_mn else (M, K), generator=g, device=dev).bfloat16() for _ in range(n_terms)]
    Bs = [torch.randn((K, N) if b_mn else (N, K), generator=g, device=dev).bfloat16() for _ in range(n_terms)]
    ref = torch.zeros(M, N, dtype=torch.float64, device=dev)
    for a, b in zip(As, Bs):
        a64 = a.double().t() if a_mn else a.double()
        b64 = b.double() if b_mn else b.double().t()
        ref += a64 @ b64
    return As, Bs, ref


SHAPES = [(256, 256, 512), (384, 128, 200), (1000, 96, 264), (512, 256, 64), (300, 64, 1032), (128, 256, 256),
          (2048, 512, 320)]


@pytest.mark.parametrize("pair", [False, True])
@pytest.mark.parametrize("a_mn,b_mn", [(False, False), (True, True), (False, True), (True, False)])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_contraction_matches_the_definition(dev, pair, a_mn, b_mn, M, N, K):
    # leading dimensions must be multiples of 8 elements
    if (a_mn and M % 8) or (b_mn and N % 8) or K % 8:
        pytest.skip("stride rule")
    B.debug_set_pair_mode(pair)
    As, Bs, ref = operands(M, N, K, a_mn, b_mn, 1, dev, seed=M + N + K)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    C = B.debug_gemm(As, Bs, M, N, K, a_mn, b_mn, out_mode=B.OUT_F32, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    scale = float(ref.abs().max())
    assert float((C.double() - ref).abs().max()) <= 2e-5 * scale * max(1.0, (K / 64) ** 0.5)


@pytest.mark.parametrize("pair", [False, True])
def test_three_terms_split_k_and_pair_output(dev, pair):
    B.debug_set_pair_mode(pair)
    M, N, K = 256, 256, 4096
    As, Bs, ref = operands(M, N, K, True, True, 3, dev, seed=11)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    P = B.debug_gemm(As, Bs, M, N, K, True, True, out_mode=B.OUT_F32, splits=8, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and P.shape == (8, M, N)
    scale = float(ref.abs().max())
    assert float((P.double().sum(0) - ref).abs().max()) <= 1e-4 * scale
    # bf16 hi/lo output: hi + lo carries 16 bits of the fp32 result
    M2, N2, K2 = 1024, 256, 256
    As, Bs, ref = operands(M2, N2, K2, False, False, 3, dev, seed=12)
    hi, lo = B.debug_gemm(As, Bs, M2, N2, K2, False, False, out_mode=B.OUT_SPLIT, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = hi.double() + lo.double()
    assert float((got - ref).abs().max()) <= 2.0 ** -15 * float(ref.abs().max()) + 1e-4 * float(ref.abs().max())


def test_both_forms_agree_bit_for_bit_on_a_gram_product(dev):
    # same products, same order of accumulation along K inside a tile: the two forms must agree exactly
    M = N = 256
    K = 2048
    As, Bs, _ = operands(M, N, K, True, True, 1, dev, seed=5)
    B.debug_set_pair_mode(False)
    C1 = B.debug_gemm(As, Bs, M, N, K, True, True, out_mode=B.OUT_F32)
    B.debug_set_pair_mode(True)
    C2 = B.debug_gemm(As, Bs, M, N, K, True, True, out_mode=B.OUT_F32)
    torch.cuda.synchronize()
    assert float((C1 - C2).abs().max()) <= 1e-5 * float(C1.abs().max())


@pytest.mark.parametrize("M,N,K,out_mode", [
    (8192, 4096, 256, "bf16"),     # 32 x 16 tiles of 256 x 256, four K blocks: two or three column tiles per pair
    (7000, 1288, 96, "f32"),       # ragged rows, ragged last column tile, K not a multiple of 64
    (4100, 2560, 512, "bf16"),     # eight K blocks: B takes 128 KB, so a four-stage ring and one staging box per warp
    (3000, 1032, 384, "f32"),      # six K blocks, fp32 boxes, ragged rows and columns
    (40000, 256, 48, "f32"),       # one column tile, many row tiles
])
def test_persistent_form_for_short_contractions_with_a_large_output(dev, M, N, K, out_mode):
    # The shape of Reconstruct (A K-major, B N-major, K <= 512, far more tiles than SMs) is served by the
    # persistent pair kernel: B resident, A streamed, double-buffered accumulator.  Checked against the
    # definition and, bit for bit, against the one-tile-per-CTA form (same products in the same order).
    As, Bs, ref = operands(M, N, K, False, True, 1, dev, seed=M + K)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    mode = B.OUT_BF16 if out_mode == "bf16" else B.OUT_F32
    B.debug_set_pair_mode(True)
    C = B.debug_gemm(As, Bs, M, N, K, False, True, out_mode=mode, status=status)
    B.debug_set_pair_mode(False)
    C1 = B.debug_gemm(As, Bs, M, N, K, False, True, out_mode=mode, status=status)
    B.debug_set_pair_mode(True)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    scale = float(ref.abs().max())
    tol = (2.0 ** -8 if out_mode == "bf16" else 2e-5 * max(1.0, (K / 64) ** 0.5)) * scale
    assert float((C.double() - ref).abs().max()) <= tol
    assert torch.equal(C, C1)


@pytest.mark.parametrize("a_mn,b_mn,M,N,K,splits", [(True, True, 256, 256, 4096, 8),      # Gram of a hi/lo pair
                                                    (False, False, 1024, 256, 256, 1),   # apply L^-T
                                                    (False, True, 256, 1024, 256, 1)])   # Omega = L^-1 T
@pytest.mark.parametrize("pattern", ["hl3", "a2", "b2"])
def test_terms_that_share_operands(dev, a_mn, b_mn, M, N, K, splits, pattern):
    # hi/lo products repeat operands: (Ah Bh + Ah Bl + Al Bh), (A0 B + A1 B), (A B0 + A B1).  The two-CTA form
    # then loads every distinct operand once per K block and issues all the products from that stage; the result
    # must be the definition, and agree with the one-CTA form (which runs the terms one after the other) to
    # fp32 rounding of a different order of additions.
    g = torch.Generator(device=dev)
    g.manual_seed(17)
    mk_a = lambda: torch.randn((K, M) if a_mn else (M, K), generator=g, device=dev).bfloat16()
    mk_b = lambda: torch.randn((K, N) if b_mn else (N, K), generator=g, device=dev).bfloat16()
    A0, A1, B0, B1 = mk_a(), (mk_a().float() * 2.0 ** -8).bfloat16(), mk_b(), (mk_b().float() * 2.0 ** -8).bfloat16()
    if pattern == "hl3":
        As, Bs = [A0, A0, A1], [B0, B1, B0]
    elif pattern == "a2":
        As, Bs = [A0, A1], [B0, B0]
    else:
        As, Bs = [A0, A0], [B0, B1]
    ref = torch.zeros(M, N, dtype=torch.float64, device=dev)
    for a, b in zip(As, Bs):
        ref += (a.double().t() if a_mn else a.double()) @ (b.double() if b_mn else b.double().t())
    out = {}
    for pair in (True, False):
        B.debug_set_pair_mode(pair)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        C = B.debug_gemm(As, Bs, M, N, K, a_mn, b_mn, out_mode=B.OUT_F32, splits=splits, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        out[pair] = C.double().sum(0) if splits > 1 else C.double()
    B.debug_set_pair_mode(True)
    scale = float(ref.abs().max())
    assert float((out[True] - ref).abs().max()) <= 1e-4 * scale
    assert float((out[True] - out[False]).abs().max()) <= 1e-5 * scale


@pytest.mark.parametrize("engine", [0, 1])
@pytest.mark.parametrize("pair", [False, True])
@pytest.mark.parametrize("r,n,splits,halve", [(256, 4096, 8, 1), (96, 1000, 3, 1), (256, 2048, 1, 2), (128, 520, 2, 1)])
def test_halved_accumulator_and_the_symmetric_gram_matrix_it_is_for(dev, engine, pair, r, n, splits, halve):
    # C = (t_0 + ... + t_{h-1}) / 2 + t_h + ...: checked against that definition in float64, for both kernels
    # (and split over K: every split halves its own partial sum).  Then the use it is made for: with the
    # pair {Yh^T Yh, Yh^T Yl} the partial sums D give D + D^T = Yh^T Yh + Yh^T Yl + Yl^T Yh, the three-term
    # Gram matrix of Y = Yh + Yl, exactly symmetric.
    if engine == 0 and pair:
        pytest.skip("the CUDA-core kernel has one form")
    B.debug_set_pair_mode(pair)
    g = torch.Generator(device=dev)
    g.manual_seed(r + n)
    Y = torch.randn(n, r, generator=g, device=dev)
    Yh = Y.bfloat16()
    Yl = (Y - Yh.float()).bfloat16()
    Z = torch.randn(n, r, generator=g, device=dev).bfloat16()
    terms_a, terms_b = ([Yh, Yh], [Yh, Yl]) if halve == 1 else ([Yh, Z, Yh], [Yh, Yh, Yl])
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    C = B.debug_gemm(terms_a, terms_b, r, r, n, True, True, out_mode=B.OUT_F32, engine=engine, splits=splits,
                     status=status, halve_at_term=halve)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    parts = C if splits > 1 else C[None]
    prods = [a.double().t() @ b.double() for a, b in zip(terms_a, terms_b)]
    ref = sum(prods[:halve]) / 2 + sum(prods[halve:])
    scale = float(ref.abs().max())
    assert float((parts.double().sum(0) - ref).abs().max()) <= 2e-5 * scale * max(1.0, (n / 64) ** 0.5)
    if halve == 1:
        W = B.debug_reduce_sym(parts.contiguous())
        torch.cuda.synchronize()
        assert torch.equal(W, W.t())
        S = parts.sum(0)                     # the kernel adds the partials in index order, as torch does here
        assert torch.equal(W, S + S.t()) or float((W - (S + S.t())).abs().max()) <= 1e-6 * scale
        gram = Yh.double().t() @ Yh.double() + Yh.double().t() @ Yl.double() + Yl.double().t() @ Yh.double()
        assert float((W.double() - gram).abs().max()) <= 4e-5 * scale * max(1.0, (n / 64) ** 0.5)
        full = (Yh.double() + Yl.double()).t() @ (Yh.double() + Yl.double())
        assert float((W.double() - full).abs().max()) <= 6e-5 * scale * max(1.0, (n / 64) ** 0.5)
    B.debug_set_pair_mode(True)


@pytest.mark.parametrize("r,n,splits", [(256, 8192, 128), (96, 1000, 16), (384, 3072, 48), (256, 8192, 32)])
def test_three_term_gram_matrix_of_a_split_sketch(dev, r, n, splits):
    # The form the orthonormalisation uses: D = (Yl^T Yl + Yh^T Yh) / 2 + Yh^T Yl per split, W = sum D + (sum D)^T,
    # which is (Yh + Yl)^T (Yh + Yl) with all four products.  Against float64; the diagonal in particular, where
    # leaving Yl^T Yl out would show as a relative deficit of about 2^-18 / 3 = 1.3e-6.
    g = torch.Generator(device=dev)
    g.manual_seed(3 * r + n)
    Y = torch.randn(n, r, generator=g, device=dev) * torch.logspace(0, -2, r, device=dev)
    Yh = Y.bfloat16()
    Yl = (Y - Yh.float()).bfloat16()
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    P = B.debug_gemm([Yl, Yh, Yh], [Yl, Yh, Yl], r, r, n, True, True, out_mode=B.OUT_F32, engine=1, splits=splits,
                     status=status, halve_at_term=2)
    W = B.debug_reduce_sym(P.contiguous())
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(W, W.t())
    Yd = Yh.double() + Yl.double()
    full = Yd.t() @ Yd
    sc = full.diagonal().sqrt()
    rel = (W.double() - full) / (sc[:, None] * sc[None, :])
    chain = -(-n // 64 // splits) * 12          # tensor-core instructions that add into one accumulator
    # the tensor cores truncate: up to an ulp (2^-23 relative) per instruction of the chain, one-signed on the diagonal
    # (about a quarter of that on average)
    assert float(rel.abs().max()) <= 2.0 ** -23 * chain + 2e-7
    without_ll = float((Yl.double() ** 2).sum(0).div(full.diagonal()).mean())
    assert without_ll > 1e-6                                            # the term is not negligible ...
    if chain == 12:                                                     # ... and with short chains one can see that it is in W
        assert float(rel.diagonal().mean()) > -(2.0 ** -24) * chain - 1e-7
