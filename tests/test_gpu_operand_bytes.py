"""Operand bytes: the 8-bit form of the 4-bit codes that a quantizer can write in the same
pass and a GEMM can fetch instead of widening the codes again.  They carry the integers the
codes stand for (INT4: 16 * q, LUQ: +-2^(c-1)), so they are checked against the oracle's
dequantization of its own codes, and every GEMM must give bit-identical results with and
without them."""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import binding, inputs

from test_gpu_parity import assert_gemm_close, luq_inputs, scalar, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def want_bytes(codes: np.ndarray, n: int, kind: str) -> np.ndarray:
    """int8 operand bytes from the oracle's reading of the codes (unit scale)."""
    v = oracle.dequant(codes, n, 1.0, kind) * (16.0 if kind == "int4" else 1.0)
    assert np.abs(v).max(initial=0) <= 127 and (v == np.rint(v)).all()
    return v.astype(np.int8)


def fresh_bytes(numel: int) -> torch.Tensor:
    return torch.full((numel,), 0x5A, dtype=torch.int8, device="cuda")   # a pattern no code maps to


@pytest.mark.parametrize("n", [2, 6, 8, 10, 1000, 4098, 65536, (1 << 20) + 2, 3_000_004])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_int4_operand_bytes(ctx, n, dtype):
    x = np.random.default_rng(n).standard_normal(n).astype(np.float32)
    x[: min(n, 4)] = np.array([0.0, -0.0, x.max(), -np.abs(x).max()], dtype=np.float32)[: min(n, 4)]
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    mx, _ = oracle.amax(x)
    want, s_want, _ = oracle.quant_int4(x, mx)
    xd = to_dev(x)
    ob = fresh_bytes(n + 16)
    codes, scale = ctx.quant_int4(xd, ctx.amax(xd), operand=ob)
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    assert scale.item() == s_want
    np.testing.assert_array_equal(ob[:n].cpu().numpy(), want_bytes(want, n, "int4"))
    assert (ob[n:] == 0x5A).all().item()           # nothing written past the tensor
    assert ctx.status() == 0


@pytest.mark.parametrize("n", [2, 6, 10, 1000, 4098, 65536, (1 << 20) + 2, 3_000_004])
@pytest.mark.parametrize("dtype,ns", [("f32", 1), ("f32", 2), ("bf16", 1), ("bf16", 3)])
def test_luq_operand_bytes(ctx, n, dtype, ns):
    x = luq_inputs(n, 8000 + n)
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    mx, _ = oracle.amax(x)
    seed = 999 + n
    want, a_want, _ = oracle.quant_luq(x, mx, seed, ns)
    xd = to_dev(x)
    ob = fresh_bytes(ns * n + 16)
    codes, alpha = ctx.quant_grad(xd, ctx.amax(xd), seed, ns, operand=ob)
    np.testing.assert_array_equal(codes.cpu().numpy().reshape(ns, -1), want)
    assert alpha.item() == a_want
    got = ob[: ns * n].cpu().numpy().reshape(ns, n)
    for s in range(ns):
        np.testing.assert_array_equal(got[s], want_bytes(want[s], n, "luq"))
    assert (ob[ns * n:] == 0x5A).all().item()
    assert ctx.status() == 0


def test_luq_operand_bytes_in_range_levels(ctx):
    """A tensor spread over every level (no warp is all-underflow) exercises the general route."""
    n = 300_000
    rng = np.random.default_rng(5)
    x = (np.exp2(rng.uniform(-6, 0, n)) * np.where(rng.random(n) < 0.5, -1, 1)).astype(np.float32)
    mx, _ = oracle.amax(x)
    want, _, _ = oracle.quant_luq(x, mx, 11, 2)
    assert set(np.unique(oracle.unpack(want[0], n) & 7)) == {0, 1, 2, 3, 4, 5}
    ob = fresh_bytes(2 * n)
    xd = to_dev(x)
    codes, _ = ctx.quant_grad(xd, ctx.amax(xd), 11, 2, operand=ob)
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    got = ob.cpu().numpy().reshape(2, n)
    for s in range(2):
        np.testing.assert_array_equal(got[s], want_bytes(want[s], n, "luq"))
    assert set(np.unique(got)) == {-16, -8, -4, -2, -1, 0, 1, 2, 4, 8, 16}


def test_operand_bytes_of_the_scale_variants(ctx):
    n, ns = 70_002, 2
    x = luq_inputs(n, 77)
    xd = to_dev(x)
    mx, _ = oracle.amax(x)
    want, _, _ = oracle.quant_luq_pw2(x, mx, 5, ns)
    ob = fresh_bytes(ns * n)
    codes, _ = ctx.quant_grad_pw2(xd, ctx.amax(xd), 5, ns, operand=ob)
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    for s in range(ns):
        np.testing.assert_array_equal(ob.cpu().numpy().reshape(ns, n)[s], want_bytes(want[s], n, "luq"))
    for pw2 in (False, True):
        m_hat = np.float32(mx) * np.float32(0.3)              # a lagging estimate: the top levels clip
        want, _, _, _, _ = oracle.quant_luq_hindsight(x, m_hat, 0.1, seed=6, n_samples=ns, pw2=pw2)
        ob = fresh_bytes(ns * n)
        codes, _, _ = ctx.quant_grad_hindsight(xd, scalar(float(m_hat)), 0.1, 6, ns, pw2, operand=ob)
        np.testing.assert_array_equal(codes.cpu().numpy(), want)
        for s in range(ns):
            np.testing.assert_array_equal(ob.cpu().numpy().reshape(ns, n)[s], want_bytes(want[s], n, "luq"))
    assert ctx.status() == 0


def test_operand_bytes_of_unusable_scales_are_zero(ctx):
    x = to_dev(np.zeros(5000, dtype=np.float32))
    ob = fresh_bytes(5000)
    ctx.quant_int4(x, ctx.amax(x), operand=ob)
    assert not ob.any().item()
    ob = fresh_bytes(10000)
    ctx.quant_grad(x, ctx.amax(x), 1, 2, operand=ob)
    assert not ob.any().item()
    assert ctx.status() == 0


def test_operand_argument_errors(ctx):
    x = to_dev(np.ones(4096, dtype=np.float32))
    ob = fresh_bytes(4096 + 16)
    with pytest.raises(binding.LuqError):        # not 16-byte aligned
        ctx.quant_int4(x, ctx.amax(x), operand=ob[1:])
    with pytest.raises(TypeError):               # too small
        ctx.quant_grad(x, ctx.amax(x), 1, 2, operand=ob)
    with pytest.raises(TypeError):               # wrong type
        ctx.quant_int4(x, ctx.amax(x), operand=ob.view(torch.uint8))


def layer_with_bytes(ctx, A, W, G, seed, ns):
    M, K = A.shape
    N = W.shape[0]
    Ad, Wd, Gd = to_dev(A), to_dev(W), to_dev(G)
    ba, bw, bg = fresh_bytes(M * K), fresh_bytes(N * K), fresh_bytes(ns * M * N)
    ca, sa = ctx.quant_int4(Ad, ctx.amax(Ad), operand=ba)
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd), operand=bw)
    cg, al = ctx.quant_grad(Gd, ctx.amax(Gd), seed, ns, operand=bg)
    return (ca, sa, ba), (cw, sw, bw), (cg, al, bg)


GEMM_SHAPES = [
    (1024, 1024, 1024, 2),   # every product: long contraction, several tiles both ways
    (1152, 1056, 800, 1),    # ragged tiles, contraction not a multiple of the block
    (300, 160, 96, 1),       # small: the bytes are passed but the codes are read
    (4096, 2304, 256, 1),    # ResNet-like layer: mixed use
]


@pytest.mark.parametrize("M,K,N,ns", GEMM_SHAPES)
def test_gemms_identical_with_and_without_operand_bytes(ctx, M, K, N, ns):
    A, W, G = inputs.small_layer(M, K, N, 900 + M)
    (ca, sa, ba), (cw, sw, bw), (cg, al, bg) = layer_with_bytes(ctx, A, W, G, seed=M, ns=ns)
    Z0 = ctx.gemm_fwd(ca, sa, cw, sw, M, N, K)
    Z1 = ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, a_operand=ba, w_operand=bw)
    Z2 = ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, w_operand=bw)
    dA0 = ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K)
    dA1 = ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=bg, w_operand=bw)
    dA2 = ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=bg)
    dW0 = ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K)
    dW1 = ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, g_operand=bg, a_operand=ba)
    dW2 = ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, a_operand=ba)
    assert ctx.status() == 0
    for x0, x1, x2 in ((Z0, Z1, Z2), (dA0, dA1, dA2), (dW0, dW1, dW2)):
        assert torch.equal(x0, x1) and torch.equal(x0, x2)
    oa, ow, og = ca.cpu().numpy(), cw.cpu().numpy(), cg.cpu().numpy().reshape(ns, -1)

    def grid(n_rows, n_cols):       # a lattice of entries, as paired index lists
        r, c = np.meshgrid(np.arange(0, n_rows, max(n_rows // 31, 1)), np.arange(0, n_cols, max(n_cols // 29, 1)))
        return r.reshape(-1), c.reshape(-1)

    r, c = grid(M, N)
    assert_gemm_close(Z1.cpu().numpy()[r, c], oracle.gemm_entries("fwd", oa, sa.item(), 1, ow, sw.item(), M, N, K, r, c))
    r, c = grid(M, K)
    assert_gemm_close(dA1.cpu().numpy()[r, c],
                      oracle.gemm_entries("bwd", og, al.item(), ns, ow, sw.item(), M, N, K, r, c))
    r, c = grid(N, K)
    assert_gemm_close(dW1.cpu().numpy()[r, c],
                      oracle.gemm_entries("wgrad", og, al.item(), ns, oa, sa.item(), M, N, K, r, c))


@pytest.mark.parametrize("mma_kind", [0, 2])
@pytest.mark.parametrize("M,K,N,ns", [(1000, 160, 416, 1),    # forward: 2 stages, 13 column chunks (one tile and a part)
                                      (777, 640, 96, 1),      # backward: 1 stage, ragged rows, 2.5 column tiles
                                      (1300, 2304, 256, 2),   # backward: 4 stages (two samples), 9 column tiles
                                      (256, 352, 224, 1)])    # all three: 3, 2 and 2 stages; the update product unsplit (4 tiles)
def test_whole_row_epilogue_of_short_contractions(ctx, M, K, N, ns, mma_kind):
    """A product with at most four contraction stages, fp32 output and both operands' bytes stores whole
    output rows (one 3-D copy per 32-row strip).  Same integers, same scales: bit-identical with the
    box epilogue of the codes path, ragged rows and partial column tiles included."""
    A, W, G = inputs.small_layer(M, K, N, 1200 + M)
    (ca, sa, ba), (cw, sw, bw), (cg, al, bg) = layer_with_bytes(ctx, A, W, G, seed=M, ns=ns)
    ctx.set_option(binding.OPT_MMA_KIND, mma_kind)
    try:
        pairs = []
        if K <= 512:
            pairs.append((ctx.gemm_fwd(ca, sa, cw, sw, M, N, K), ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, a_operand=ba, w_operand=bw)))
        dA_rows = None
        if ns * N <= 512:
            dA_rows = ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=bg, w_operand=bw)
            pairs.append((ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K), dA_rows))
        if ns * M <= 512:
            pairs.append((ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K),
                          ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, g_operand=bg, a_operand=ba)))
        assert pairs
        for plain, rows in pairs:
            assert torch.equal(plain, rows)
        if dA_rows is not None and mma_kind == 2:
            # the bytes are what is multiplied: all-zero gradient bytes give an all-zero product
            out = torch.full((M, K), 7.0, device="cuda")
            ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, out, g_operand=torch.zeros_like(bg), w_operand=bw)
            assert not out.any().item()
            # and nothing is written outside the output: a guard row after it keeps its pattern
            buf = torch.full((M + 40, K), 3.0, device="cuda")
            ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, buf[:M], g_operand=bg, w_operand=bw)
            assert torch.equal(buf[:M], dA_rows)
            assert (buf[M:] == 3.0).all().item()
    finally:
        ctx.set_option(binding.OPT_MMA_KIND, 2)
    assert ctx.status() == 0


def test_gemm_reads_the_bytes_it_is_given(ctx):
    """Where a product fetches operand bytes, it must fetch the caller's: all-zero bytes give an
    all-zero product.  (With e4m3 operands forced, the int8 bytes are ignored.)"""
    M = K = N = 1024
    A, W, G = inputs.small_layer(M, K, N, 17)
    (ca, sa, ba), (cw, sw, bw), (cg, al, bg) = layer_with_bytes(ctx, A, W, G, seed=1, ns=1)
    zeros = torch.zeros_like(bw)
    Z = ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, a_operand=ba, w_operand=zeros)
    assert not Z.any().item()
    ctx.set_option(binding.OPT_MMA_KIND, 0)
    try:
        Z_e4m3 = ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, a_operand=ba, w_operand=zeros)
    finally:
        ctx.set_option(binding.OPT_MMA_KIND, 2)
    assert torch.equal(Z_e4m3, ctx.gemm_fwd(ca, sa, cw, sw, M, N, K))
    assert ctx.status() == 0


@pytest.mark.parametrize("mma_kind", [0, 2])
def test_cta_pair_kernel_matches_the_single_cta_kernel(ctx, mma_kind):
    """LUQ_OPT_PAIRS: products whose operands both arrive as bytes and whose contraction is not split
    run on CTA pairs (256-row tiles, cta_group::2).  Same integers, same epilogue: bit-identical.
    The shape has more tiles than half the SMs (no split) and ragged edges in both directions."""
    M, K, N, ns = 2176, 1024, 2304, 2
    A, W, G = inputs.small_layer(M, K, N, 123)
    (ca, sa, ba), (cw, sw, bw), (cg, al, bg) = layer_with_bytes(ctx, A, W, G, seed=5, ns=ns)
    ctx.set_option(binding.OPT_MMA_KIND, mma_kind)
    ctx.set_option(binding.OPT_PAIRS, 0)
    try:
        single = (ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, a_operand=ba, w_operand=bw),
                  ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=bg, w_operand=bw),
                  ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, g_operand=bg, a_operand=ba))
        launches = ctx.launches
        ctx.set_option(binding.OPT_PAIRS, 1)
        paired = (ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, a_operand=ba, w_operand=bw),
                  ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=bg, w_operand=bw),
                  ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, g_operand=bg, a_operand=ba))
        ctx.set_option(binding.OPT_PAIRS, 2)      # the default: pairs where measured faster (backward, update)
        auto = (ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, a_operand=ba, w_operand=bw),
                ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=bg, w_operand=bw),
                ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, g_operand=bg, a_operand=ba))
    finally:
        ctx.set_option(binding.OPT_PAIRS, 2)
        ctx.set_option(binding.OPT_MMA_KIND, 2)
    assert ctx.status() == 0
    for s, p, a in zip(single, paired, auto):
        assert torch.equal(s, p) and torch.equal(s, a)
    oa, ow, og = ca.cpu().numpy(), cw.cpu().numpy(), cg.cpu().numpy().reshape(ns, -1)
    r = np.array([0, 127, 128, 255, 256, 1000, M - 1, M - 1, 0], dtype=np.int64)
    c = np.array([0, 255, 256, 1, N - 1, 777, N - 1, 0, N - 1], dtype=np.int64)
    assert_gemm_close(paired[0].cpu().numpy()[r, c],
                      oracle.gemm_entries("fwd", oa, sa.item(), 1, ow, sw.item(), M, N, K, r, c))
    ck = np.minimum(c, K - 1)
    assert_gemm_close(paired[1].cpu().numpy()[r, ck],
                      oracle.gemm_entries("bwd", og, al.item(), ns, ow, sw.item(), M, N, K, r, ck))
    rn = np.minimum(r, N - 1)
    assert_gemm_close(paired[2].cpu().numpy()[rn, ck],
                      oracle.gemm_entries("wgrad", og, al.item(), ns, oa, sa.item(), M, N, K, rn, ck))
