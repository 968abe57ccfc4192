"""The autograd wrapper is argument marshalling: its outputs and gradients must be exactly what the
C-ABI calls give, and those are checked against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import autograd, inputs

from test_gpu_parity import assert_gemm_close

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N", [288, 224])    # two columns of output tiles / one (A quantized inside the forward product)
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_function_matches_the_oracle(dtype, N):
    M, K, ns, seed = 384, 256, 2, 17
    A, W, G = inputs.small_layer(M, K, N, 4)
    a = torch.from_numpy(A).cuda().to(dtype).requires_grad_(True)
    w = torch.from_numpy(W).cuda().to(dtype).requires_grad_(True)
    g = torch.from_numpy(G).cuda().to(dtype)
    z = autograd.luq_linear(a, w, seed, ns)
    z.backward(g)
    # the oracle on the same (possibly bf16-rounded) inputs
    to_np = (lambda t: t.detach().float().cpu().numpy()) if dtype == torch.float32 else \
        (lambda t: t.detach().view(torch.int16).cpu().numpy().view(np.uint16))
    An, Wn, Gn = to_np(a), to_np(w), to_np(g)
    oa, sa, _ = oracle.quant_int4(An, oracle.amax(An)[0])
    ow, sw, _ = oracle.quant_int4(Wn, oracle.amax(Wn)[0])
    og, al, _ = oracle.quant_luq(Gn, oracle.amax(Gn)[0], seed, ns)
    refs = (oracle.gemm_fwd(oa, sa, ow, sw, M, N, K), oracle.gemm_bwd(og, al, ns, ow, sw, M, N, K),
            oracle.gemm_wgrad(og, al, ns, oa, sa, M, N, K))
    for got, ref in zip((z, a.grad, w.grad), refs):
        assert got.dtype == dtype
        got = got.detach().float().cpu().numpy().astype(np.float64)
        if dtype == torch.float32:
            assert_gemm_close(got, ref)
        else:   # the result is rounded once more, to bf16
            assert (np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref)).all()


def test_module_trains_a_small_regression():
    torch.manual_seed(0)
    K, N, M = 128, 64, 512
    target = torch.randn(N, K, device="cuda") / K ** 0.5
    layer = autograd.LuqLinear(K, N, n_samples=2, seed=100, device="cuda")
    opt = torch.optim.SGD(layer.parameters(), lr=0.2)
    losses = []
    for _ in range(60):
        x = torch.randn(M, K, device="cuda")
        loss = (layer(x) - x @ target.T).pow(2).sum(1).mean()     # gradient 2 (W - target) for white inputs
        opt.zero_grad()
        loss.backward()
        opt.step()
        losses.append(loss.item())
    assert layer.calls == 60
    assert losses[-1] < 0.2 * losses[0]          # the 4-bit forward noise sets the floor; no divergence
    assert autograd.context(torch.device("cuda", 0)).status() == 0


@pytest.mark.parametrize("N", [288, 224])
def test_function_with_in_hindsight_estimates_matches_the_oracle(N):
    M, K, ns, seed, eta = 384, 256, 2, 23, 0.1
    A, W, G = inputs.small_layer(M, K, N, 6)
    a = torch.from_numpy(A).cuda().requires_grad_(True)
    w = torch.from_numpy(W).cuda().requires_grad_(True)
    g = torch.from_numpy(G).cuda()
    start = np.array([oracle.amax(A)[0] * 0.7, oracle.amax(W)[0] * 1.2, oracle.amax(G)[0] * 0.5], dtype=np.float32)
    est = torch.from_numpy(start.copy()).cuda()
    z = autograd.luq_linear(a, w, seed, ns, est, eta)
    z.backward(g)
    oa, sa, _, ma, na = oracle.quant_int4_hindsight(A, start[0], eta)
    ow, sw, _, mw, nw = oracle.quant_int4_hindsight(W, start[1], eta)
    og, al, _, mg, ng = oracle.quant_luq_hindsight(G, start[2], eta, seed, ns)
    np.testing.assert_array_equal(est.cpu().numpy(), np.array([na, nw, ng], dtype=np.float32))
    assert_gemm_close(z.detach().cpu().numpy(), oracle.gemm_fwd(oa, float(sa), ow, float(sw), M, N, K))
    assert_gemm_close(a.grad.cpu().numpy(), oracle.gemm_bwd(og, float(al), ns, ow, float(sw), M, N, K))
    assert_gemm_close(w.grad.cpu().numpy(), oracle.gemm_wgrad(og, float(al), ns, oa, float(sa), M, N, K))


def test_module_trains_with_in_hindsight_maxima():
    torch.manual_seed(0)
    K, N, M = 128, 64, 512
    target = torch.randn(N, K, device="cuda") / K ** 0.5
    layer = autograd.LuqLinear(K, N, n_samples=2, seed=100, device="cuda", hindsight=True)
    opt = torch.optim.SGD(layer.parameters(), lr=0.2)
    losses = []
    for _ in range(60):
        x = torch.randn(M, K, device="cuda")
        loss = (layer(x) - x @ target.T).pow(2).sum(1).mean()
        opt.zero_grad()
        loss.backward()
        opt.step()
        losses.append(loss.item())
    assert (layer.estimates > 0).all().item()
    assert losses[-1] < 0.2 * losses[0]
    assert autograd.context(torch.device("cuda", 0)).status() == 0


def test_stacked_layers_get_gradients_on_the_first_step_and_restored_estimates_are_kept():
    """Every estimate is primed with its tensor's own maximum the first time the tensor is seen - the
    gradient's in the first backward pass - so the first layer of a stack receives a gradient on step 1;
    a module restored from a state dict keeps the estimates it was saved with."""
    torch.manual_seed(1)
    K = 128
    layers = torch.nn.Sequential(*[autograd.LuqLinear(K, K, seed=10 * i, device="cuda", hindsight=True)
                                   for i in range(3)])
    x = torch.randn(256, K, device="cuda")
    layers(x).pow(2).mean().backward()
    for layer in layers:
        assert layer.weight.grad.abs().max().item() > 0
        assert (layer.estimates > 0).all().item() and layer._primed == [True, True, True]
    saved = {k: v.clone() for k, v in layers.state_dict().items()}
    fresh = torch.nn.Sequential(*[autograd.LuqLinear(K, K, seed=10 * i, device="cuda", hindsight=True)
                                  for i in range(3)])
    fresh.load_state_dict(saved)
    for layer, old in zip(fresh, layers):
        assert layer._primed == [True, True, True]
        assert torch.equal(layer.estimates, old.estimates)
    before = [layer.estimates.clone() for layer in fresh]
    fresh(x * 0.5).pow(2).mean().backward()
    eta = 0.1
    for layer, b in zip(fresh, before):
        # A's estimate followed the recursion from the restored value: it was not measured afresh
        assert layer.estimates[0].item() != b[0].item()
        assert layer.estimates[0].item() > 0.5 * b[0].item() * (1 - eta)
    first = fresh[0]
    want = oracle.hindsight_next(oracle.amax((x * 0.5).cpu().numpy())[0], before[0][0].item(), eta)
    assert first.estimates[0].item() == want
    assert autograd.context(torch.device("cuda", 0)).status() == 0
