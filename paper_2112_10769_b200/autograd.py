"""A linear layer trained with the 4-bit path, as a ``torch.autograd.Function``.

Argument marshalling only: every step runs in the library's kernels (Sec. 3, Eqs. Forward /
Backward / Update; Sec. 4 LUQ; Sec. 5.1 SMP).

    forward    Z  = Q_INT(A) . Q_INT(W)^T
    backward   dA = mean_s Q_FP,s(G) . Q_INT(W)
    update     dW = mean_s Q_FP,s(G)^T . Q_INT(A)

``A`` is ``[M, K]`` (leading dimensions are flattened), ``W`` is ``[N, K]`` as in ``torch.nn.Linear``.
The INT4 codes of the forward pass are kept for the backward pass (the paper's update GEMM re-uses the
quantized activations), together with the 8-bit operand bytes of W and G that the GEMMs re-read.
Shapes must satisfy the GEMMs' divisibility rules (K and N multiples of 32).

With ``estimates`` (a float32 tensor of three running maxima: A, W, G) the quantizers take the
in-hindsight route of Sec. 7: each tensor is quantized in one pass with the estimate made from earlier
steps while its own maximum is measured and folded into the estimate - no max pass over any tensor.
"""
from __future__ import annotations

import torch

from . import binding

_contexts: dict[int, binding.Context] = {}


def context(device: torch.device) -> binding.Context:
    """One library context per device, created on first use."""
    index = device.index if device.index is not None else torch.cuda.current_device()
    if index not in _contexts:
        _contexts[index] = binding.Context(index)
    return _contexts[index]


class LuqLinearFunction(torch.autograd.Function):
    @staticmethod
    def forward(ctx, a: torch.Tensor, w: torch.Tensor, seed: int, n_samples: int,
                estimates: torch.Tensor | None = None, eta: float = 0.1, primed: list | None = None):
        lib = context(a.device)
        a2 = a.reshape(-1, a.shape[-1]).contiguous()
        w2 = w.contiguous()
        M, K = a2.shape
        N = w2.shape[0]
        w_bytes = torch.empty(N * K, dtype=torch.int8, device=a.device)
        # A is quantized inside the forward product where the layer allows it (one column of output tiles,
        # N <= 256); elsewhere the same calls run the quantizer and the product one after the other
        if estimates is None:
            cw, sw = lib.quant_int4(w2, lib.amax(w2), operand=w_bytes)
            ca, sa, z = lib.quant_int4_gemm_fwd(a2, lib.amax(a2), cw, sw, M, N, K, w_operand=w_bytes)
        else:
            if primed is not None:
                # a tensor seen for the first time has no history: its estimate starts as its own maximum
                if not primed[0]:
                    lib.amax(a2, estimates[0:1]); primed[0] = True
                if not primed[1]:
                    lib.amax(w2, estimates[1:2]); primed[1] = True
            cw, sw, _ = lib.quant_int4_hindsight(w2, estimates[1:2], eta, operand=w_bytes)
            ca, sa, _, z = lib.quant_int4_hindsight_gemm_fwd(a2, estimates[0:1], eta, cw, sw, M, N, K, w_operand=w_bytes)
        ctx.save_for_backward(ca, sa, cw, sw, w_bytes)
        ctx.dims = (M, N, K, a.shape, a.dtype, w.dtype)
        ctx.seed, ctx.n_samples = int(seed), int(n_samples)
        ctx.estimates, ctx.eta, ctx.primed = estimates, float(eta), primed
        return z.reshape(*a.shape[:-1], N).to(a.dtype)

    @staticmethod
    def backward(ctx, grad_out: torch.Tensor):
        ca, sa, cw, sw, w_bytes = ctx.saved_tensors
        M, N, K, a_shape, a_dtype, w_dtype = ctx.dims
        ns = ctx.n_samples
        lib = context(grad_out.device)
        g2 = grad_out.reshape(M, N).contiguous()
        # several samples (Sec. 5.1): one operand plane holding their sum while that sum fits int8 - the two
        # products then cost what one sample's cost, with the same result (LUQ_OPT_SUM_SAMPLES)
        lib.set_option(binding.OPT_SUM_SAMPLES, int(ns > 1 and (ns << binding.kmax()) <= 127))
        g_bytes = torch.empty(lib._planes(ns) * M * N, dtype=torch.int8, device=g2.device)
        if ctx.estimates is None:
            cg, alpha = lib.quant_grad(g2, lib.amax(g2), ctx.seed, ns, operand=g_bytes)
        else:
            if ctx.primed is not None and not ctx.primed[2]:
                # first backward pass: without this the gradient would be quantized with an estimate of
                # zero, i.e. to all zeros, and every layer below would receive (and measure) nothing
                lib.amax(g2, ctx.estimates[2:3]); ctx.primed[2] = True
            cg, alpha, _ = lib.quant_grad_hindsight(g2, ctx.estimates[2:3], ctx.eta, ctx.seed, ns, operand=g_bytes)
        da = dw = None
        if ctx.needs_input_grad[0]:
            da = lib.gemm_bwd(cg, alpha, ns, cw, sw, M, N, K, g_operand=g_bytes, w_operand=w_bytes)
            da = da.reshape(a_shape).to(a_dtype)
        if ctx.needs_input_grad[1]:
            dw = lib.gemm_wgrad(cg, alpha, ns, ca, sa, M, N, K, g_operand=g_bytes).to(w_dtype)
        return da, dw, None, None, None, None, None


def luq_linear(a: torch.Tensor, w: torch.Tensor, seed: int, n_samples: int = 1,
               estimates: torch.Tensor | None = None, eta: float = 0.1, primed: list | None = None) -> torch.Tensor:
    """``a @ w.T`` with INT4 operands forward and LUQ-FP4 gradients backward.  ``seed`` keys the
    stochastic rounding of this call's backward pass: give every layer and step its own.
    ``estimates``: three running maxima (A, W, G) for the in-hindsight route; updated in place.
    ``primed``: a list of three booleans, updated in place - an estimate whose flag is False is first
    set to its tensor's own maximum (one extra max pass, the first time only).  Without it the caller
    initialises the estimates."""
    return LuqLinearFunction.apply(a, w, seed, n_samples, estimates, eta, primed)


class LuqLinear(torch.nn.Module):
    """``torch.nn.Linear`` without bias whose three GEMMs run on the 4-bit path.  The seed of the
    gradient quantizer advances with every forward call."""

    def __init__(self, in_features: int, out_features: int, n_samples: int = 1, seed: int = 0,
                 device=None, dtype=torch.float32, hindsight: bool = False, eta: float = 0.1):
        super().__init__()
        # in-hindsight maxima of A, W and G (Sec. 7): each is measured once, the first time its tensor is
        # seen (A and W in the first forward pass, G in the first backward pass), then estimated.  An
        # estimate is "primed" when it is positive; the flags mirror that on the host and are rebuilt
        # from the buffer when a state dict is loaded, so restored estimates are kept.
        self.hindsight, self.eta = hindsight, eta
        self.register_buffer("estimates", torch.zeros(3, device=device, dtype=torch.float32))
        self._primed = [False, False, False]
        w = torch.empty(out_features, in_features, device=device, dtype=dtype)
        torch.nn.init.kaiming_uniform_(w, a=5 ** 0.5)
        self.weight = torch.nn.Parameter(w)
        self.n_samples = n_samples
        self.base_seed = seed
        self.calls = 0

    def forward(self, a: torch.Tensor) -> torch.Tensor:
        seed = self.base_seed + self.calls * self.n_samples     # sample s of a call uses seed + s
        self.calls += 1
        if not self.hindsight:
            return luq_linear(a, self.weight, seed, self.n_samples)
        return luq_linear(a, self.weight, seed, self.n_samples, self.estimates, self.eta, self._primed)

    def _load_from_state_dict(self, state_dict, prefix, *args, **kwargs):
        super()._load_from_state_dict(state_dict, prefix, *args, **kwargs)
        if prefix + "estimates" in state_dict:
            self._primed[:] = [bool(v > 0) for v in self.estimates.tolist()]
