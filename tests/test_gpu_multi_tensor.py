"""Several tensors in one launch: maxima, codes, scales and operand bytes against the CPU oracle,
and equal to the one-tensor calls, whatever the mix of sizes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import binding, inputs

from test_gpu_parity import to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


SIZE_SETS = [(2,), (65536, 10), (3_000_004, 4098), (10, 1 << 20, 6, 5_000_012), (20_000_000, 590_000),
             (1000, 1000, 1000, 1000)]


@pytest.mark.parametrize("sizes", SIZE_SETS)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_multi_tensor_calls_equal_the_single_ones(ctx, sizes, dtype):
    rng = np.random.default_rng(sum(sizes))
    hosts = []
    for i, n in enumerate(sizes):
        x = (rng.standard_normal(n) * 10.0 ** (i - 1)).astype(np.float32)
        x[n // 3] = np.float32(-(7.5 + i) * 10.0 ** (i - 1))            # a distinct maximum per tensor
        hosts.append(inputs.to_bf16_bits(x) if dtype == "bf16" else x)
    xs = [to_dev(h) for h in hosts]
    for _ in range(2):                                                    # twice: scratch regions left clean
        maxima = ctx.amax_multi(xs)
        for h, x, m in zip(hosts, xs, maxima):
            assert m.item() == oracle.amax(h)[0] == ctx.amax(x).item()
    operands = [torch.full((x.numel(),), 0x5A, dtype=torch.int8, device="cuda") if i % 2 == 0 else None
                for i, x in enumerate(xs)]
    codes, scales = ctx.quant_int4_multi(xs, maxima, operands=operands)
    for h, x, m, c, s, o in zip(hosts, xs, maxima, codes, scales, operands):
        want, s_want, _ = oracle.quant_int4(h, m.item())
        np.testing.assert_array_equal(c.cpu().numpy(), want)
        assert s.item() == s_want
        if o is not None:
            q = oracle.unpack(want, x.numel()).astype(np.int64)       # the oracle's codes, as integers
            q = np.where(q >= 8, q - 16, q)
            np.testing.assert_array_equal(o.cpu().numpy(), (16 * q).astype(np.int8))
            ob = torch.empty_like(o)
            ctx.quant_int4(x, m, operand=ob)
            assert torch.equal(o, ob)
    assert ctx.status() == 0


def test_multi_tensor_special_values_and_errors(ctx):
    z = to_dev(np.zeros(1000, dtype=np.float32))
    bad = np.ones(5000, dtype=np.float32)
    bad[17] = np.inf
    good = to_dev(np.arange(2000, dtype=np.float32))
    maxima = ctx.amax_multi([z, to_dev(bad), good])
    assert maxima[0].item() == 0 and np.isinf(maxima[1].item()) and maxima[2].item() == 1999
    assert ctx.status() & binding.STATUS_NONFINITE
    codes, scales = ctx.quant_int4_multi([z, to_dev(bad), good], maxima)
    assert scales[0].item() == 0 and scales[1].item() == 0 and not codes[0].any().item() and not codes[1].any().item()
    want, s_want, _ = oracle.quant_int4(np.arange(2000, dtype=np.float32), np.float32(1999))
    np.testing.assert_array_equal(codes[2].cpu().numpy(), want)
    assert ctx.status() & binding.STATUS_NONFINITE
    with pytest.raises(binding.LuqError):
        ctx.amax_multi([good] * 5)                                        # at most four tensors
    # the one-tensor kernels share the context's scratch words with these: still clean
    assert ctx.amax(good).item() == 1999
    assert ctx.status() == 0
