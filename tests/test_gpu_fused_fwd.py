"""The forward product that quantizes its activations on the way in (luq_quant_int4_gemm_fwd):
the INT4 codes and the scale it writes must be those of the oracle's quantizer bit for bit, and Z
within 1e-5 of the oracle's product of those codes, for ragged shapes in every dimension, both
input types, with and without W's operand bytes, few CTAs walking many tiles, and for the shapes
where the call falls back to the two separate kernels."""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import binding, inputs

from test_gpu_parity import assert_gemm_close, scalar, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture()
def ctx():
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


SHAPES = [
    (128, 128, 256),      # one tile, one operand stage
    (300, 160, 96),       # ragged rows, K = 2.5 raw stages, one partial slab of W
    (1000, 32, 32),       # minimum contraction: the second raw stage lies beyond K
    (130, 416, 200),      # K leaves half a raw stage
    (257, 96, 132),       # one row into the third tile
    (2000, 2304, 256),    # the ResNet layer's K and N
    (4224, 640, 256),     # 33 tiles
]


def run_case(ctx, M, K, N, dtype, with_bytes, clip_factor=1.0, seed=0):
    A, W, _ = inputs.small_layer(M, K, N, 700 + M + K + seed)
    if dtype == "bf16":
        A, W = inputs.to_bf16_bits(A), inputs.to_bf16_bits(W)
    Ad, Wd = to_dev(A), to_dev(W)
    bw = torch.empty(N * K, dtype=torch.int8, device="cuda") if with_bytes else None
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd), operand=bw)
    clip = ctx.amax(Ad) * clip_factor
    ca = torch.full((M * K // 2 + 64,), 0xEE, dtype=torch.uint8, device="cuda")      # guard bytes behind the codes
    Z = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    ca_out, sa, Z_out = ctx.quant_int4_gemm_fwd(Ad, clip, cw, sw, M, N, K, a_codes=ca, out=Z, w_operand=bw)
    oa, osa, _ = oracle.quant_int4(A, np.float32(clip.item()))
    ow, osw, _ = oracle.quant_int4(W, oracle.amax(W)[0])
    np.testing.assert_array_equal(cw.cpu().numpy(), ow)
    got = ca.cpu().numpy()
    np.testing.assert_array_equal(got[:M * K // 2], oa)
    assert (got[M * K // 2:] == 0xEE).all()
    assert sa.item() == osa and sw.item() == osw
    assert_gemm_close(Z.cpu().numpy(), oracle.gemm_fwd(oa, osa, ow, osw, M, N, K))
    return ca, sa, Z


@pytest.mark.parametrize("with_bytes", [True, False])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("M,K,N", SHAPES)
def test_fused_forward_matches_oracle(ctx, M, K, N, dtype, with_bytes):
    launches = ctx.launches
    run_case(ctx, M, K, N, dtype, with_bytes)
    # amax(W), quant(W), amax(A), [expansion of W's codes], ONE kernel for quantizer + product
    assert ctx.launches - launches == (4 if with_bytes else 5)
    assert ctx.status() == 0


@pytest.mark.parametrize("limit", [1, 2, 5])
def test_few_ctas_walk_many_tiles(ctx, limit):
    """Rings, accumulator buffers and code boxes wrap many times inside one CTA."""
    ctx.set_option(binding.OPT_SM_LIMIT, limit)
    try:
        ca, sa, Z = run_case(ctx, 1700, 352, 256, "f32", True, seed=limit)
        # equal to the two separate kernels, bit for bit
        A, W, _ = inputs.small_layer(1700, 352, 256, 700 + 1700 + 352 + limit)
        Ad, Wd = to_dev(A), to_dev(W)
        cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd))
        c2, s2 = ctx.quant_int4(Ad, ctx.amax(Ad))
        Z2 = ctx.gemm_fwd(c2, s2, cw, sw, 1700, 256, 352)
        assert torch.equal(ca[:c2.numel()], c2) and torch.equal(Z, Z2)
    finally:
        ctx.set_option(binding.OPT_SM_LIMIT, 0)


@pytest.mark.parametrize("limit", [1, 2])
def test_repeated_calls_give_the_same_codes(ctx, limit):
    """A raw slot goes back to its producer while the warp that read it still converts: a refill that
    overtook the reads would show as wrong codes in some calls (seen once in about 150 with an
    earlier hand-over), so the same small problem is run many times on few, fast CTAs."""
    M, K, N = 1700, 352, 256
    ctx.set_option(binding.OPT_SM_LIMIT, limit)
    try:
        ca, sa, Z = run_case(ctx, M, K, N, "f32", True, seed=limit)       # checked against the oracle
        ca, Z = ca.clone(), Z.clone()
        A, W, _ = inputs.small_layer(M, K, N, 700 + M + K + limit)
        Ad, Wd = to_dev(A), to_dev(W)
        bw = torch.empty(N * K, dtype=torch.int8, device="cuda")
        cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd), operand=bw)
        clip = ctx.amax(Ad)
        for _ in range(400):
            c2 = torch.full_like(ca, 0xEE)
            _, _, Z2 = ctx.quant_int4_gemm_fwd(Ad, clip, cw, sw, M, N, K, a_codes=c2, w_operand=bw)
            assert torch.equal(c2, ca) and torch.equal(Z2, Z)
    finally:
        ctx.set_option(binding.OPT_SM_LIMIT, 0)


def test_caller_clip_specials_and_unusable_clips(ctx):
    M, K, N = 384, 128, 64
    # a clip below the maximum saturates at +-7, as in the streaming quantizer
    run_case(ctx, M, K, N, "f32", True, clip_factor=0.37)
    A, W, _ = inputs.small_layer(M, K, N, 5)
    A[3, 5] = np.nan; A[100, 127] = np.inf; A[383, 0] = -np.inf; A[7, 7] = -0.0
    Ad, Wd = to_dev(A), to_dev(W)
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd))
    ca, sa, Z = ctx.quant_int4_gemm_fwd(Ad, scalar(2.5), cw, sw, M, N, K)
    oa, osa, _ = oracle.quant_int4(A, np.float32(2.5))
    np.testing.assert_array_equal(ca.cpu().numpy(), oa)
    assert sa.item() == osa
    assert_gemm_close(Z.cpu().numpy(), oracle.gemm_fwd(oa, osa, cw.cpu().numpy(), sw.item(), M, N, K))
    assert ctx.status() == 0
    for clip, flag in ((0.0, 0), (float("inf"), binding.STATUS_NONFINITE), (float("nan"), binding.STATUS_NONFINITE),
                       (2.0 ** -120, binding.STATUS_RANGE), (2.0 ** 110, binding.STATUS_RANGE)):
        ca, sa, Z = ctx.quant_int4_gemm_fwd(Ad, scalar(clip), cw, sw, M, N, K)
        assert sa.item() == 0 and not ca.any().item() and not Z.any().item()
        assert ctx.status() == flag


def test_shapes_outside_the_fusion_run_the_two_kernels(ctx):
    for (M, K, N), opt in (((300, 160, 512), None), ((256, 128, 96), (binding.OPT_MMA_KIND, 0))):
        if opt:
            ctx.set_option(*opt)
        try:
            launches = ctx.launches
            run_case(ctx, M, K, N, "f32", True)
            assert ctx.launches - launches == 5     # amax(W), quant(W), amax(A), quant(A), product
        finally:
            if opt:
                ctx.set_option(binding.OPT_MMA_KIND, 2)
    with pytest.raises(binding.LuqError):
        ctx.quant_int4_gemm_fwd(torch.zeros(64, 48, device="cuda"), scalar(1.0),
                                torch.zeros(32 * 24, dtype=torch.uint8, device="cuda"), scalar(1.0), 64, 32, 48)
    # empty batch: nothing to do, no error
    ca, sa, Z = ctx.quant_int4_gemm_fwd(torch.zeros(0, 64, device="cuda"), scalar(1.0),
                                        torch.zeros(32 * 32, dtype=torch.uint8, device="cuda"), scalar(1.0), 0, 32, 64)
    assert Z.numel() == 0


HINDSIGHT_SHAPES = [(300, 160, 96), (1000, 32, 32), (257, 96, 132), (4224, 640, 256)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("M,K,N", HINDSIGHT_SHAPES)
def test_in_hindsight_form_over_a_sequence_of_steps(ctx, M, K, N, dtype):
    """The kernel that quantizes with a running estimate, measures max|A| itself and replaces the estimate:
    codes, scale, measured maximum, next estimate against the oracle bit for bit over steps whose scale
    jumps (the estimate lags: some steps saturate); Z within 1e-5 of the oracle's product."""
    eta = 0.1
    A0, W, _ = inputs.small_layer(M, K, N, 4000 + M + K)
    if dtype == "bf16":
        W = inputs.to_bf16_bits(W)
    Wd = to_dev(W)
    bw = torch.empty(N * K, dtype=torch.int8, device="cuda")
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd), operand=bw)
    ow = cw.cpu().numpy()
    first = inputs.to_bf16_bits(A0) if dtype == "bf16" else A0
    est_o = oracle.amax(first)[0]
    est_d = scalar(float(est_o))
    saturated = 0
    for step, sc in enumerate([1.0, 0.3, 6.0, 0.05, 2.0]):
        A = (A0 * np.float32(sc)).astype(np.float32)
        A[step % M, step % K] = np.float32(-0.0)
        if dtype == "bf16":
            A = inputs.to_bf16_bits(A)
        want, s_want, fl, meas_want, next_want = oracle.quant_int4_hindsight(A, est_o, eta)
        launches = ctx.launches
        ca, sa, measured, Z = ctx.quant_int4_hindsight_gemm_fwd(to_dev(A), est_d, eta, cw, sw, M, N, K, w_operand=bw)
        assert ctx.launches - launches == 1
        assert fl == 0 and sa.item() == s_want and measured.item() == meas_want and est_d.item() == next_want
        np.testing.assert_array_equal(ca.cpu().numpy(), want)
        assert_gemm_close(Z.cpu().numpy(), oracle.gemm_fwd(want, s_want, ow, sw.item(), M, N, K))
        saturated += int(meas_want > est_o)
        est_o = next_want
    assert saturated >= 1
    # the same step through the two separate kernels: identical results
    e1, e2 = scalar(float(est_o)), scalar(float(est_o))
    Ad = to_dev(A)
    ca1, sa1, m1, Z1 = ctx.quant_int4_hindsight_gemm_fwd(Ad, e1, eta, cw, sw, M, N, K, w_operand=bw)
    ca2, sa2, m2 = ctx.quant_int4_hindsight(Ad, e2, eta)
    Z2 = ctx.gemm_fwd(ca2, sa2, cw, sw, M, N, K, w_operand=bw)
    assert torch.equal(ca1, ca2) and torch.equal(Z1, Z2)
    assert (sa1.item(), m1.item(), e1.item()) == (sa2.item(), m2.item(), e2.item())


def test_in_hindsight_form_specials(ctx):
    M, K, N = 384, 128, 64
    A, W, _ = inputs.small_layer(M, K, N, 5)
    Wd = to_dev(W)
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd))
    # an estimate of zero quantizes everything to zero and is replaced by the measurement
    est = scalar(0.0)
    ca, sa, measured, Z = ctx.quant_int4_hindsight_gemm_fwd(to_dev(A), est, 0.1, cw, sw, M, N, K)
    assert not ca.any().item() and sa.item() == 0 and not Z.any().item()
    assert measured.item() == oracle.amax(A)[0] == est.item()
    assert ctx.status() == 0
    # an Inf among the activations: the measurement is Inf, the flag is raised, the estimate stays
    B = A.copy(); B[17, 3] = np.inf; B[200, 100] = np.nan
    est = scalar(1.5)
    ca, sa, measured, Z = ctx.quant_int4_hindsight_gemm_fwd(to_dev(B), est, 0.1, cw, sw, M, N, K)
    want, s_want, fl, meas_want, next_want = oracle.quant_int4_hindsight(B, np.float32(1.5), 0.1)
    np.testing.assert_array_equal(ca.cpu().numpy(), want)
    assert est.item() == 1.5 == next_want and not np.isfinite(measured.item())
    assert ctx.status() == binding.STATUS_NONFINITE
    # a layer too wide for the fusion runs the two kernels, with the same results
    M2, K2, N2 = 256, 64, 512
    A2, W2, _ = inputs.small_layer(M2, K2, N2, 9)
    W2d = to_dev(W2)
    cw2, sw2 = ctx.quant_int4(W2d, ctx.amax(W2d))
    est = scalar(0.8)
    launches = ctx.launches
    ca, sa, measured, Z = ctx.quant_int4_hindsight_gemm_fwd(to_dev(A2), est, 0.25, cw2, sw2, M2, N2, K2)
    assert ctx.launches - launches >= 2
    want, s_want, fl, meas_want, next_want = oracle.quant_int4_hindsight(A2, np.float32(0.8), 0.25)
    np.testing.assert_array_equal(ca.cpu().numpy(), want)
    assert (sa.item(), measured.item(), est.item()) == (s_want, meas_want, next_want)
    assert_gemm_close(Z.cpu().numpy(), oracle.gemm_fwd(want, s_want, cw2.cpu().numpy(), sw2.item(), M2, N2, K2))
    with pytest.raises(binding.LuqError):
        ctx.quant_int4_hindsight_gemm_fwd(to_dev(A), scalar(1.0), 1.5, cw, sw, M, N, K)
