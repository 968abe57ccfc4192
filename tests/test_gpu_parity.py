"""Parity of the CUDA path against the CPU oracle, through the C ABI.

Codes must match bit for bit; GEMM outputs within 1e-5 relative (products and
sums are exact integers, only the two scale roundings of the epilogue differ
from the float64 oracle) and exact zeros must be exact zeros.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import binding, inputs

pytestmark = pytest.mark.gpu

RTOL = 1e-5


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


def to_dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:  # bf16 bit patterns
        return torch.from_numpy(a.view(np.int16).copy()).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def scalar(v) -> torch.Tensor:
    return torch.tensor([v], dtype=torch.float32, device="cuda")


def assert_gemm_close(got: np.ndarray, ref: np.ndarray):
    """1e-5 relative, entry by entry, against the float64 oracle; entries the oracle has
    exactly zero must be exactly zero."""
    got = got.astype(np.float64)
    zero = ref == 0
    assert (got[zero] == 0).all(), "entries that are exactly zero in the oracle must be exactly zero"
    err = np.abs(got - ref)
    rel = err[~zero] / np.abs(ref[~zero])
    assert (err <= RTOL * np.abs(ref)).all(), f"max relative error {rel.max() if rel.size else 0.0:.3e}"


# ------------------------------------------------------------------ amax ----

@pytest.mark.parametrize("n", [1, 2, 3, 5, 8, 1023, 4096, 65537, (1 << 20) + 6, 5_000_011])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_amax_matches_oracle(ctx, n, dtype):
    x = inputs.lognormal_gradient((n,), -10.0, 3.0, 0.2, 1000 + n)
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    want, fl = oracle.amax(x)
    got = ctx.amax(to_dev(x)).cpu().numpy()[0]
    assert fl == 0 and got == want and got.dtype == np.float32
    assert ctx.status() == 0


def test_amax_zero_empty_and_nonfinite(ctx):
    assert ctx.amax(torch.zeros(1000, device="cuda")).item() == 0.0
    assert ctx.amax(torch.zeros(0, device="cuda")).item() == 0.0
    assert ctx.status() == 0
    for bad in (float("inf"), float("-inf"), float("nan")):
        x = torch.randn(100000, device="cuda")
        x[77777] = bad
        got = ctx.amax(x).item()
        assert not np.isfinite(got)
        assert ctx.status() == binding.STATUS_NONFINITE
        assert ctx.status() == 0  # reading clears


# ------------------------------------------------------------------ INT4 ----

@pytest.mark.parametrize("n", [2, 6, 8, 10, 1000, 4098, 65536, (1 << 20) + 2, 3_000_004])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_quant_int4_bit_exact(ctx, n, dtype):
    x = inputs.normal((n,), 1.0, 2000 + n, relu=(n % 4 == 0))
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    clip, _ = oracle.amax(x)
    want, s_want, fl = oracle.quant_int4(x, clip)
    xd = to_dev(x)
    codes, scale = ctx.quant_int4(xd, ctx.amax(xd))
    assert fl == 0 and scale.item() == s_want
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    assert ctx.status() == 0


def test_quant_int4_caller_clip_ties_and_specials(ctx):
    x = np.array([0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5, 6.5, 100.0, -100.0, 7.49, 7.51, 0.0, -0.0, np.nan, np.inf,
                  -np.inf, 1e-30], dtype=np.float32)
    want, s_want, _ = oracle.quant_int4(x, np.float32(7.0))
    codes, scale = ctx.quant_int4(to_dev(x), scalar(7.0))
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    assert scale.item() == s_want == 1.0
    # window of consecutive floats around a rounding boundary
    clip = np.float32(3.0)
    start = np.array([2.5 * 3.0 / 7.0], dtype=np.float32).view(np.uint32)[0]
    x = (np.arange(-2000, 2000, dtype=np.int64) + int(start)).astype(np.uint32).view(np.float32)
    want, _, _ = oracle.quant_int4(x, clip)
    codes, _ = ctx.quant_int4(to_dev(x), scalar(3.0))
    np.testing.assert_array_equal(codes.cpu().numpy(), want)


def test_quant_zero_and_unusable_scale(ctx):
    x = torch.randn(4096, device="cuda")
    for clip, flag in ((0.0, 0), (float("inf"), binding.STATUS_NONFINITE), (float("nan"), binding.STATUS_NONFINITE),
                       (2.0 ** -120, binding.STATUS_RANGE), (2.0 ** 110, binding.STATUS_RANGE)):
        codes, scale = ctx.quant_int4(x, scalar(clip))
        assert scale.item() == 0 and not codes.any().item()
        assert ctx.status() == flag
        codes, alpha = ctx.quant_grad(x, scalar(clip), seed=1, n_samples=2)
        assert alpha.item() == 0 and not codes.any().item()
        assert ctx.status() == flag
    z = torch.zeros(4096, device="cuda")
    codes, alpha = ctx.quant_grad(z, ctx.amax(z), seed=1)
    assert alpha.item() == 0 and not codes.any().item() and ctx.status() == 0


def test_argument_errors(ctx):
    x = torch.randn(64, device="cuda")
    with pytest.raises(binding.LuqError):
        ctx.quant_grad(x, scalar(1.0), seed=0, n_samples=0)
    with pytest.raises(binding.LuqError):
        ctx.quant_grad(x, scalar(1.0), seed=0, n_samples=9)
    with pytest.raises(binding.LuqError):
        ctx.quant_int4(x[:63], scalar(1.0))          # odd element count
    with pytest.raises(binding.LuqError):
        ctx.quant_int4(x[1:33], scalar(1.0))         # misaligned pointer
    c = torch.zeros(64 * 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.LuqError):
        ctx.gemm_fwd(c, scalar(1.0), c, scalar(1.0), 64, 32, 16)   # K not a multiple of 32


# ------------------------------------------------------------------- LUQ ----

def luq_inputs(n, seed):
    x = inputs.log_uniform_magnitudes(n, -30, 3, seed)
    mx = np.abs(x).max()
    al = mx / 16
    special = [0.0, -0.0, mx, -mx, al, -al, 2 * al, 4 * al, 8 * al, 1e-38, -1e-45, al * (1 - 2 ** -24), al * (1 + 2 ** -23)]
    k = min(len(special), n)
    x[:k] = np.array(special[:k], dtype=np.float32)
    if n > 20:
        x[20] = np.float32(mx)
    return x


@pytest.mark.parametrize("n", [2, 6, 8, 10, 1000, 4098, 65536, (1 << 20) + 2, 3_000_004])
@pytest.mark.parametrize("dtype,ns", [("f32", 1), ("f32", 2), ("bf16", 1), ("bf16", 3)])
def test_quant_grad_bit_exact(ctx, n, dtype, ns):
    x = luq_inputs(n, 3000 + n)
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    mx, _ = oracle.amax(x)
    seed = 12345 + n
    want, a_want, fl = oracle.quant_luq(x, mx, seed, ns)
    xd = to_dev(x)
    codes, alpha = ctx.quant_grad(xd, ctx.amax(xd), seed, ns)
    assert fl == 0 and alpha.item() == a_want
    np.testing.assert_array_equal(codes.cpu().numpy().reshape(ns, -1), want)
    assert ctx.status() == 0


@pytest.mark.parametrize("exponent", [-103, -99, -80, -62, -59, -45, -20, 60, 95])
@pytest.mark.parametrize("pw2", [False, True])
def test_quant_grad_extreme_scales(ctx, exponent, pw2):
    """Maxima near both ends of the accepted range, and on both sides of the point below which
    the kernel rescales its operands: codes stay bit-exact (inputs reach into the denormals)."""
    n = 300_000
    x = (luq_inputs(n, 400 + exponent).astype(np.float64) * 2.0 ** exponent).astype(np.float32)
    mx, _ = oracle.amax(x)
    xd = to_dev(x)
    if pw2:
        want, a_want, fl = oracle.quant_luq_pw2(x, mx, 5, 2)
        codes, alpha = ctx.quant_grad_pw2(xd, ctx.amax(xd), 5, 2)
    else:
        want, a_want, fl = oracle.quant_luq(x, mx, 5, 2)
        codes, alpha = ctx.quant_grad(xd, ctx.amax(xd), 5, 2)
    assert alpha.item() == a_want
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    assert ctx.status() == fl


def test_quant_grad_seed_semantics_and_clipping(ctx):
    x = luq_inputs(50000, 9)
    xd = to_dev(x)
    mx = ctx.amax(xd)
    big = (1 << 63) + 12345678901234
    for seed in (0, 1, 2 ** 32 - 1, 2 ** 32, big):
        want, _, _ = oracle.quant_luq(x, mx.item(), seed, 2)
        codes, _ = ctx.quant_grad(xd, mx, seed, 2)
        np.testing.assert_array_equal(codes.cpu().numpy(), want)
    # sample s of seed equals sample 0 of seed + s
    c2, _ = ctx.quant_grad(xd, mx, 40, 3)
    c0, _ = ctx.quant_grad(xd, mx, 42, 1)
    assert torch.equal(c2[2], c0[0])
    # a caller max below the true one clips to the top level
    small = scalar(float(mx.item()) / 64)
    want, a_want, _ = oracle.quant_luq(x, small.item(), 5, 1)
    codes, alpha = ctx.quant_grad(xd, small, 5, 1)
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    assert alpha.item() == a_want
    # many scales: on-grid inputs are fixed points for every seed
    rng = np.random.default_rng(3)
    for mxv in np.exp2(rng.uniform(-20, 20, 40)).astype(np.float32):
        al = np.float32(mxv) / np.float32(16)
        grid = np.array([al * 2 ** k for k in range(5)] * 8, dtype=np.float32)
        want, _, _ = oracle.quant_luq(grid, mxv, 7, 1)
        codes, _ = ctx.quant_grad(to_dev(grid), scalar(float(mxv)), 7, 1)
        np.testing.assert_array_equal(codes.cpu().numpy(), want)
        assert list(oracle.unpack(want[0], 5)) == [1, 2, 3, 4, 5]


# ------------------------------------------------------------------ GEMMs ----

def run_layer(ctx, A, W, G, seed, ns):
    """Whole path on the GPU; returns device tensors and the oracle's codes."""
    M, K = A.shape
    N = W.shape[0]
    Ad, Wd, Gd = to_dev(A), to_dev(W), to_dev(G)
    ca, sa = ctx.quant_int4(Ad, ctx.amax(Ad))
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd))
    cg, al = ctx.quant_grad(Gd, ctx.amax(Gd), seed, ns)
    Z = ctx.gemm_fwd(ca, sa, cw, sw, M, N, K)
    dA = ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K)
    dW = ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K)
    oa, osa, _ = oracle.quant_int4(A, oracle.amax(A)[0])
    ow, osw, _ = oracle.quant_int4(W, oracle.amax(W)[0])
    og, oal, _ = oracle.quant_luq(G, oracle.amax(G)[0], seed, ns)
    np.testing.assert_array_equal(ca.cpu().numpy(), oa)
    np.testing.assert_array_equal(cw.cpu().numpy(), ow)
    np.testing.assert_array_equal(cg.cpu().numpy().reshape(ns, -1), og)
    assert (sa.item(), sw.item(), al.item()) == (osa, osw, oal)
    return (Z, dA, dW), (oa, osa), (ow, osw), (og, oal)


SHAPES = [
    (128, 128, 256, 1),    # one tile, one contraction block
    (256, 256, 256, 1),    # config 1 shape
    (300, 160, 96, 1),     # ragged in every dimension
    (130, 416, 544, 2),    # several tiles with tails, two samples
    (1000, 32, 32, 1),     # minimum contraction
    (64, 1024, 288, 3),    # three samples
]


@pytest.mark.parametrize("mma_kind", [0, 1, 2])
@pytest.mark.parametrize("M,K,N,ns", SHAPES)
def test_three_gemms_match_oracle(ctx, M, K, N, ns, mma_kind):
    ctx.set_option(binding.OPT_MMA_KIND, mma_kind)
    try:
        A, W, G = inputs.small_layer(M, K, N, 500 + M + K)
        (Z, dA, dW), (oa, osa), (ow, osw), (og, oal) = run_layer(ctx, A, W, G, seed=M, ns=ns)
        assert ctx.status() == 0
        assert_gemm_close(Z.cpu().numpy(), oracle.gemm_fwd(oa, osa, ow, osw, M, N, K))
        assert_gemm_close(dA.cpu().numpy(), oracle.gemm_bwd(og, oal, ns, ow, osw, M, N, K))
        assert_gemm_close(dW.cpu().numpy(), oracle.gemm_wgrad(og, oal, ns, oa, osa, M, N, K))
    finally:
        ctx.set_option(binding.OPT_MMA_KIND, 2)


@pytest.mark.parametrize("splits", [1, 2, 5])
def test_wgrad_contraction_split(ctx, splits):
    """The update GEMM contracts over the batch; splitting that contraction over
    CTAs must not change the result."""
    M, K, N = 2500, 160, 96
    A, W, G = inputs.small_layer(M, K, N, 77)
    ctx.set_option(binding.OPT_SPLITS, splits)
    try:
        for _ in range(2):  # twice: the workspace must be left clean
            (Z, dA, dW), (oa, osa), (ow, osw), (og, oal) = run_layer(ctx, A, W, G, seed=3, ns=2)
            assert ctx.status() == 0
            assert_gemm_close(dW.cpu().numpy(), oracle.gemm_wgrad(og, oal, 2, oa, osa, M, N, K))
            assert_gemm_close(dA.cpu().numpy(), oracle.gemm_bwd(og, oal, 2, ow, osw, M, N, K))
            assert_gemm_close(Z.cpu().numpy(), oracle.gemm_fwd(oa, osa, ow, osw, M, N, K))
    finally:
        ctx.set_option(binding.OPT_SPLITS, 0)


def test_config1_whole_step(ctx):
    cfg = inputs.CONFIGS["cfg1"]
    A, W, G = inputs.layer_inputs(cfg)
    (Z, dA, dW), (oa, osa), (ow, osw), (og, oal) = run_layer(ctx, A, W, G, cfg.luq_seed, cfg.n_samples)
    M, K, N = cfg.M, cfg.K, cfg.N
    assert_gemm_close(Z.cpu().numpy(), oracle.gemm_fwd(oa, osa, ow, osw, M, N, K))
    assert_gemm_close(dA.cpu().numpy(), oracle.gemm_bwd(og, oal, 1, ow, osw, M, N, K))
    assert_gemm_close(dW.cpu().numpy(), oracle.gemm_wgrad(og, oal, 1, oa, osa, M, N, K))
    assert ctx.status() == 0


def test_empty_contraction_gives_zeros(ctx):
    """K = 0 in the forward product, an empty batch in the update product: the sum over nothing is 0
    in every entry of a non-empty output (not stale memory)."""
    one = scalar(1.0)
    e = torch.zeros(0, dtype=torch.uint8, device="cuda")
    Z = torch.full((64, 32), float("nan"), device="cuda")
    ctx.gemm_fwd(e, one, e, one, 64, 32, 0, out=Z)
    dW = torch.full((32, 64), float("nan"), device="cuda")
    ctx.gemm_wgrad(e, one, 2, e, one, 0, 32, 64, out=dW)
    dA = torch.full((64, 96), float("nan"), device="cuda")
    ctx.gemm_bwd(e, one, 1, e, one, 64, 0, 96, out=dA)
    assert not Z.any().item() and not dW.any().item() and not dA.any().item()
    ctx.set_option(binding.OPT_OUTPUT_BF16, 1)
    try:
        Zh = torch.full((64, 32), float("nan"), dtype=torch.bfloat16, device="cuda")
        ctx.gemm_fwd(e, one, e, one, 64, 32, 0, out=Zh)
        assert not Zh.any().item()
    finally:
        ctx.set_option(binding.OPT_OUTPUT_BF16, 0)
    assert ctx.status() == 0


def test_gemm_large_integer_sums_are_exact(ctx):
    """Worst-case operands (every code at its extreme) over a long contraction:
    the accumulator must hold every integer partial sum exactly."""
    M, N, K = 128, 256, 4096
    a = torch.full((M, K // 2), 0x77, dtype=torch.uint8, device="cuda")     # all +7
    w = torch.full((N, K // 2), 0x77, dtype=torch.uint8, device="cuda")
    w[1::2] = 0x99                                                           # odd rows all -7
    for kind in (0, 1, 2):
        ctx.set_option(binding.OPT_MMA_KIND, kind)
        Z = ctx.gemm_fwd(a, scalar(1.0), w, scalar(1.0), M, N, K).cpu().numpy()
        assert (Z[:, 0::2] == 49 * K).all() and (Z[:, 1::2] == -49 * K).all()
        # sums that need all 24 bits: 49*K + small odd corrections
        a2 = a.clone()
        a2[:, 0] = 0x71                                                     # first element +1 instead of +7
        Z = ctx.gemm_fwd(a2, scalar(1.0), w, scalar(1.0), M, N, K).cpu().numpy()
        assert (Z[:, 0::2] == 49 * K - 42).all()
        # gradient levels up to 16 times weights up to 7 over the whole contraction
        g = torch.full((M, K // 2), 0x55, dtype=torch.uint8, device="cuda")  # all +16 (code 5)
        wk = torch.full((K, N // 2), 0x77, dtype=torch.uint8, device="cuda")
        dA = ctx.gemm_bwd(g, scalar(1.0), 1, wk, scalar(1.0), M, K, N).cpu().numpy()
        assert (dA == 16 * 7 * K).all()
    ctx.set_option(binding.OPT_MMA_KIND, 2)
    assert ctx.status() == 0


def test_division_free_quotient_equals_ieee_division(ctx):
    """The quantizer forms t = |x|/alpha with a reciprocal and two residual
    corrections; it must be the IEEE round-to-nearest quotient for every scale,
    including maxima near the ends of the accepted range [2^-100, 2^100]."""
    rng = np.random.default_rng(123)
    n = 1 << 21
    exps = list(rng.uniform(-99, 99, 40)) + [-100, -99.5, -63, -44.2, -43.9, -40, 0, 40, 99.9]
    total = 0
    for ex in exps:
        mx = np.float32(2.0 ** ex) * np.float32(rng.uniform(1.0, 1.9999))
        if ex <= -100:
            mx = np.float32(2.0 ** -100)
        alpha = np.float32(mx) / np.float32(16)
        # magnitudes from far below alpha up to a few times the maximum, plus values hugging the levels
        t_target = np.exp2(rng.uniform(-45, 5.5, n))
        x = (t_target * float(alpha)).astype(np.float32)
        lv = (alpha * np.float32(2.0) ** rng.integers(0, 5, 4096)).astype(np.float32)
        x[:4096] = lv
        x[4096:8192] = np.nextafter(lv, np.float32(0))
        x[8192:12288] = np.nextafter(lv, np.float32(np.inf))
        x[12288:16384] = (lv * np.float32(1.5)).astype(np.float32)
        x *= np.where(rng.random(n) < 0.5, -1, 1).astype(np.float32)
        with np.errstate(over="ignore", under="ignore"):
            ref = (np.abs(x) / alpha).astype(np.float32)
        got = ctx.debug_quotient(to_dev(x), scalar(float(mx))).cpu().numpy()
        check = (ref >= np.float32(2.0 ** -60)) & (ref <= np.float32(64.0))
        np.testing.assert_array_equal(got[check].view(np.uint32), ref[check].view(np.uint32))
        small = ref < np.float32(2.0 ** -60)
        assert (got[small] < 2.0 ** -40).all()
        total += int(check.sum())
    assert total > 50_000_000
    assert ctx.status() == 0


# ----------------------------------------- power-of-two scale, in-hindsight maximum ----

@pytest.mark.parametrize("n", [10, 4098, (1 << 20) + 2])
@pytest.mark.parametrize("dtype,ns", [("f32", 1), ("f32", 2), ("bf16", 3)])
def test_quant_grad_pw2_bit_exact(ctx, n, dtype, ns):
    x = luq_inputs(n, 5000 + n)
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    mx, _ = oracle.amax(x)
    want, a_want, fl = oracle.quant_luq_pw2(x, mx, 77 + n, ns)
    xd = to_dev(x)
    codes, alpha = ctx.quant_grad_pw2(xd, ctx.amax(xd), 77 + n, ns)
    assert fl == 0 and alpha.item() == a_want
    np.testing.assert_array_equal(codes.cpu().numpy().reshape(ns, -1), want)
    # a maximum that already is a power of two is used as it is; one just above it doubles
    for m in (np.float32(0.25), np.nextafter(np.float32(0.25), np.float32(1))):
        want, a_want, _ = oracle.quant_luq_pw2(x, m, 3, 1)
        codes, alpha = ctx.quant_grad_pw2(xd, scalar(float(m)), 3, 1)
        assert alpha.item() == a_want
        np.testing.assert_array_equal(codes.cpu().numpy(), want)
    assert ctx.status() == 0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("pw2", [False, True])
def test_hindsight_sequence_matches_oracle(ctx, dtype, pw2):
    """Six steps with tensors whose scale jumps around: the estimate lags, some steps clip.
    Codes, alpha, the measured maximum and the estimate must match the oracle bit for bit."""
    n, eta, ns = 200_006, 0.1, 2
    scales = [1.0, 0.4, 5.0, 0.05, 2.0, 1.0]
    base = inputs.log_uniform_magnitudes(n, -20, 2, 31)
    first = (base * np.float32(scales[0])).astype(np.float32)
    m_hat_o = oracle.amax(inputs.to_bf16_bits(first) if dtype == "bf16" else first)[0]
    m_hat_d = scalar(float(m_hat_o))
    clipped = 0
    for step, sc in enumerate(scales):
        x = (base * np.float32(sc)).astype(np.float32)
        x[step] = np.float32(0.0)
        if dtype == "bf16":
            x = inputs.to_bf16_bits(x)
        want, a_want, fl, meas_want, next_want = oracle.quant_luq_hindsight(x, m_hat_o, eta, seed=step, n_samples=ns, pw2=pw2)
        codes, alpha, measured = ctx.quant_grad_hindsight(to_dev(x), m_hat_d, eta, step, ns, pw2)
        assert fl == 0 and alpha.item() == a_want and measured.item() == meas_want
        assert m_hat_d.item() == next_want
        np.testing.assert_array_equal(codes.cpu().numpy().reshape(ns, -1), want)
        clipped += int(meas_want > m_hat_o)
        m_hat_o = next_want
    assert clipped >= 2
    assert ctx.status() == 0


def test_hindsight_unusable_estimate_recovers(ctx):
    x = luq_inputs(50_000, 4)
    xd = to_dev(x)
    m_hat = scalar(0.0)
    codes, alpha, measured = ctx.quant_grad_hindsight(xd, m_hat, 0.1, 1)
    assert alpha.item() == 0 and not codes.any().item()
    assert measured.item() == oracle.amax(x)[0]
    assert m_hat.item() == oracle.hindsight_next(measured.item(), 0.0, 0.1)
    assert ctx.status() == 0
    codes, alpha, _ = ctx.quant_grad_hindsight(xd, m_hat, 0.1, 2)
    assert alpha.item() > 0 and codes.any().item()
    with pytest.raises(binding.LuqError):
        ctx.quant_grad_hindsight(xd, m_hat, 1.5, 1)
    assert ctx.status() == 0


# ------------------------------- other grids from the same kernels: level count, nearest power ----

@pytest.mark.parametrize("kmax", [1, 2, 3, 5, 6])
@pytest.mark.parametrize("dtype,ns", [("f32", 1), ("bf16", 2)])
def test_quant_grad_other_level_counts(ctx, kmax, dtype, ns):
    n = 500_002
    x = inputs.log_uniform_magnitudes(n, -12, 1, 60 + kmax)       # every level of every grid occurs
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    mx, _ = oracle.amax(x)
    xd = to_dev(x)
    ctx.set_option(binding.OPT_LEVELS, kmax)
    try:
        want, a_want, _ = oracle.quant_luq(x, mx, 21, ns, kmax=kmax)
        ob = torch.empty(ns * n, dtype=torch.int8, device="cuda")
        codes, alpha = ctx.quant_grad(xd, ctx.amax(xd), 21, ns, operand=ob)
        assert alpha.item() == a_want == oracle.luq_alpha(mx, kmax)
        np.testing.assert_array_equal(codes.cpu().numpy(), want)
        assert set(np.unique(oracle.unpack(want[0], n) & 7)) == set(range(kmax + 2))
        got = ob.cpu().numpy().reshape(ns, n)
        for s in range(ns):
            np.testing.assert_array_equal(got[s], oracle.dequant(want[s], n, 1.0, "luq").astype(np.int8))
        want, a_want, _ = oracle.quant_luq_pw2(x, mx, 22, ns, kmax=kmax)
        codes, alpha = ctx.quant_grad_pw2(xd, ctx.amax(xd), 22, ns)
        assert alpha.item() == a_want
        np.testing.assert_array_equal(codes.cpu().numpy(), want)
        _, codes, alpha = ctx.amax_quant_grad(xd, 21, ns)
        np.testing.assert_array_equal(codes.cpu().numpy(), oracle.quant_luq(x, mx, 21, ns, kmax=kmax)[0])
    finally:
        ctx.set_option(binding.OPT_LEVELS, 4)
    with pytest.raises(binding.LuqError):
        ctx.set_option(binding.OPT_LEVELS, 7)
    assert ctx.status() == 0


def test_gemms_with_the_widest_grid(ctx):
    """kmax = 6: gradient levels up to 64 alpha; the GEMMs must still be exact."""
    M, K, N, ns = 384, 256, 288, 2
    A, W, G = inputs.small_layer(M, K, N, 91)
    ctx.set_option(binding.OPT_LEVELS, 6)
    try:
        Ad, Wd, Gd = to_dev(A), to_dev(W), to_dev(G)
        ca, sa = ctx.quant_int4(Ad, ctx.amax(Ad))
        cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd))
        cg, al = ctx.quant_grad(Gd, ctx.amax(Gd), 3, ns)
        og, oal, _ = oracle.quant_luq(G, oracle.amax(G)[0], 3, ns, kmax=6)
        np.testing.assert_array_equal(cg.cpu().numpy(), og)
        assert (oracle.unpack(og[0], M * N) & 7).max() == 7
        for kind in (0, 1):
            ctx.set_option(binding.OPT_MMA_KIND, kind)
            dA = ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K)
            dW = ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K)
            assert_gemm_close(dA.cpu().numpy(), oracle.gemm_bwd(og, oal, ns, cw.cpu().numpy(), sw.item(), M, N, K))
            assert_gemm_close(dW.cpu().numpy(), oracle.gemm_wgrad(og, oal, ns, ca.cpu().numpy(), sa.item(), M, N, K))
    finally:
        ctx.set_option(binding.OPT_MMA_KIND, 2)
        ctx.set_option(binding.OPT_LEVELS, 4)
    assert ctx.status() == 0


@pytest.mark.parametrize("n", [10, 4098, (1 << 20) + 2])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("kmax", [2, 4])
def test_quant_grad_nearest_power_bit_exact(ctx, n, dtype, kmax):
    x = luq_inputs(n, 700 + n)
    mx0 = np.abs(x).max()
    # values on and around the midpoints of the bins, where the deterministic decision flips
    al = np.float32(mx0) / np.float32(2 ** kmax)
    mids = np.array([al * 0.5, al * 1.5, al * 3, al * 6], dtype=np.float32)
    k = min(n - 2, 12)
    x[-k:] = np.concatenate([mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(np.inf))])[:k]
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    mx, _ = oracle.amax(x)
    xd = to_dev(x)
    ctx.set_option(binding.OPT_LEVELS, kmax)
    try:
        want, a_want, _ = oracle.quant_fp_nearest(x, mx, kmax)
        ob = torch.empty(n, dtype=torch.int8, device="cuda")
        codes, alpha = ctx.quant_grad_nearest(xd, ctx.amax(xd), operand=ob)
        assert alpha.item() == a_want
        np.testing.assert_array_equal(codes.cpu().numpy(), want)
        np.testing.assert_array_equal(ob.cpu().numpy(), oracle.dequant(want[0], n, 1.0, "luq").astype(np.int8))
    finally:
        ctx.set_option(binding.OPT_LEVELS, 4)
    assert ctx.status() == 0


def test_back_to_back_steps_equal_a_synchronised_step(ctx):
    """Every kernel may become resident while its predecessor drains; nothing may be read or written
    before the predecessor has finished.  Thirty steps queued without a host synchronisation, buffers
    re-used, must leave exactly what one synchronised step leaves."""
    M, K, N, ns = 1152, 1056, 800, 2
    A, W, G = inputs.small_layer(M, K, N, 5)
    Ad, Wd, Gd = to_dev(A), to_dev(W), to_dev(G)
    dev = Ad.device
    f32 = lambda *s: torch.empty(s, dtype=torch.float32, device=dev)   # noqa: E731
    u8 = lambda *s: torch.empty(s, dtype=torch.uint8, device=dev)      # noqa: E731
    i8 = lambda n: torch.empty(n, dtype=torch.int8, device=dev)        # noqa: E731
    mA, mW, mG, sA, sW, aG = (f32(1) for _ in range(6))
    cA, cW, cG = u8(M * K // 2), u8(N * K // 2), u8(ns, M * N // 2)
    bW, bG = i8(N * K), i8(ns * M * N)
    Z, dA, dW = f32(M, N), f32(M, K), f32(N, K)

    def step(seed):
        ctx.amax(Ad, mA); ctx.amax(Wd, mW)
        ctx.quant_int4(Ad, mA, cA, sA); ctx.quant_int4(Wd, mW, cW, sW, bW)
        ctx.gemm_fwd(cA, sA, cW, sW, M, N, K, Z, None, bW)
        ctx.amax(Gd, mG); ctx.quant_grad(Gd, mG, seed, ns, cG, aG, bG)
        ctx.gemm_bwd(cG, aG, ns, cW, sW, M, N, K, dA, bG, bW)
        ctx.gemm_wgrad(cG, aG, ns, cA, sA, M, N, K, dW, bG, None)

    step(29)
    torch.cuda.synchronize()
    want = [t.clone() for t in (cA, cW, cG, Z, dA, dW, mA, mW, mG, sA, sW, aG)]
    for t in (cA, cW, cG, Z, dA, dW):
        t.zero_()
    for seed in range(30):          # different seeds: every step really rewrites the gradient codes
        step(seed)
    torch.cuda.synchronize()
    for got, ref in zip((cA, cW, cG, Z, dA, dW, mA, mW, mG, sA, sW, aG), want):
        assert torch.equal(got, ref)
    assert ctx.status() == 0


def test_an_expired_wait_is_reported_and_the_context_stays_usable(ctx):
    """The library's waits are bounded: when one runs out the kernel raises a status bit and returns.
    The diagnostic kernel waits on a barrier nothing arrives on (no fault, no hang)."""
    x = to_dev(luq_inputs(100_000, 8))
    before, _ = ctx.quant_grad(x, ctx.amax(x), 3, 1)
    assert ctx.status() == 0
    ctx.debug_expire_wait()
    assert ctx.status() == binding.STATUS_TIMEOUT
    assert ctx.status() == 0                       # reading the status clears it
    after, _ = ctx.quant_grad(x, ctx.amax(x), 3, 1)
    _, fused, _ = ctx.amax_quant_grad(x, 3, 1)     # also the kernels that share the scratch counters
    assert torch.equal(before, after) and torch.equal(before, fused)
    assert ctx.status() == 0


def test_a_step_can_be_captured_in_a_cuda_graph(ctx):
    """No call of the path allocates or synchronises with the host, so a whole step can be captured
    once and replayed; the replay must leave what the direct calls leave."""
    cfg = inputs.CONFIGS["cfg1"]
    A, W, G = inputs.layer_inputs(cfg)
    M, K, N, ns = cfg.M, cfg.K, cfg.N, 2
    Ad, Wd, Gd = to_dev(A), to_dev(W), to_dev(G)
    f32 = lambda *s: torch.empty(s, dtype=torch.float32, device="cuda")   # noqa: E731
    u8 = lambda *s: torch.empty(s, dtype=torch.uint8, device="cuda")      # noqa: E731
    mA, mW, mG, sA, sW, aG = (f32(1) for _ in range(6))
    cA, cW, cG = u8(M * K // 2), u8(N * K // 2), u8(ns, M * N // 2)
    bW, bG = torch.empty(N * K, dtype=torch.int8, device="cuda"), torch.empty(ns * M * N, dtype=torch.int8, device="cuda")
    Z, dA, dW = f32(M, N), f32(M, K), f32(N, K)

    def step():
        ctx.amax_multi([Ad, Wd], [mA, mW])
        ctx.quant_int4_multi([Ad, Wd], [mA, mW], [cA, cW], [sA, sW], [None, bW])
        ctx.gemm_fwd(cA, sA, cW, sW, M, N, K, Z, None, bW)
        ctx.amax_quant_grad(Gd, 5, ns, mG, cG, aG, bG)
        ctx.gemm_bwd(cG, aG, ns, cW, sW, M, N, K, dA, bG, bW)
        ctx.gemm_wgrad(cG, aG, ns, cA, sA, M, N, K, dW, bG, None)

    step()
    torch.cuda.synchronize()
    want = [t.clone() for t in (cA, cW, cG, Z, dA, dW)]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()                                   # warm up on the capture stream
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
        for t in (cA, cW, cG, Z, dA, dW):
            t.zero_()
        for _ in range(3):
            graph.replay()
    torch.cuda.synchronize()
    for got, ref in zip((cA, cW, cG, Z, dA, dW), want):
        assert torch.equal(got, ref)
    assert ctx.status() == 0
