"""ctypes binding of the C-ABI library declared in ``include/luq.h``.

Argument marshalling only: every step of the path runs in the CUDA kernels of
``libluq_b200.so``.  PyTorch supplies device memory and the current stream.
There is no fallback: if the library has not been built (``python -m
paper_2112_10769_b200.build``) or no sm_100 GPU is present, calls raise.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# LUQ_LIB selects another build of the same library, e.g. the bounds-checking one (libluq_b200_debug.so)
LIB_PATH = os.environ.get("LUQ_LIB") or os.path.join(_HERE, "libluq_b200.so")

LUQ_F32, LUQ_BF16 = 0, 1
STATUS_NONFINITE, STATUS_RANGE, STATUS_TIMEOUT, STATUS_BOUNDS = 1, 2, 4, 8
OPT_MMA_KIND, OPT_SPLITS, OPT_PAIRS, OPT_LEVELS, OPT_UNSIGNED_ACTIVATIONS, OPT_OUTPUT_BF16 = 1, 2, 3, 4, 5, 6
OPT_GRADIENT_INT4 = 7
OPT_SM_LIMIT = 8
OPT_SUM_SAMPLES = 9
SCHEME_FP4, SCHEME_FP4_SR, SCHEME_FP4_SU, SCHEME_LUQ, SCHEME_INT4_SR = 0, 1, 2, 3, 4
ERR_ARG, ERR_CUDA, ERR_UNSUPPORTED, ERR_WORKSPACE = -1, -2, -3, -4

SYMBOLS = ("luq_create", "luq_destroy", "luq_set_option", "luq_kmax", "luq_debug_build", "luq_amax", "luq_quant_int4",
           "luq_amax_multi", "luq_quant_int4_multi", "luq_quant_int4_hindsight_gemm_fwd", "luq_quant_uint4", "luq_amax_quant_int4", "luq_quant_int4_hindsight", "luq_quant_grad", "luq_amax_quant_grad", "luq_quant_grad_nearest", "luq_quant_grad_ablation", "luq_quant_grad_pw2",
           "luq_quant_grad_hindsight", "luq_debug_quotient", "luq_debug_expire_wait", "luq_debug_bounds_probe", "luq_gemm_fwd", "luq_quant_int4_gemm_fwd", "luq_gemm_bwd", "luq_gemm_wgrad",
           "luq_gemm_wgrad_static", "luq_status", "luq_launch_count", "luq_strerror")

_lib = None


class LuqError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {load().luq_strerror(code).decode()} ({code})")


def load() -> ctypes.CDLL:
    """Loads the compiled library; raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2112_10769_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, i64, u64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int64, ctypes.c_uint64
        L.luq_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int]
        L.luq_destroy.argtypes = [vp]
        L.luq_set_option.argtypes = [vp, ctypes.c_int, ctypes.c_int]
        L.luq_kmax.argtypes = []
        L.luq_debug_build.argtypes = []
        L.luq_amax.argtypes = [vp, vp, ctypes.c_int, sz, vp, vp]
        L.luq_quant_int4.argtypes = [vp, vp, ctypes.c_int, sz, sz, vp, vp, vp, vp, vp]
        L.luq_amax_multi.argtypes = [vp, ctypes.c_int, vp, ctypes.c_int, vp, vp, vp]
        L.luq_quant_int4_multi.argtypes = [vp, ctypes.c_int, vp, ctypes.c_int, vp, vp, vp, vp, vp, vp]
        L.luq_quant_uint4.argtypes = [vp, vp, ctypes.c_int, sz, sz, vp, vp, vp, vp, vp]
        L.luq_amax_quant_int4.argtypes = [vp, vp, ctypes.c_int, sz, sz, vp, vp, vp, vp, vp]
        L.luq_amax_quant_grad.argtypes = [vp, vp, ctypes.c_int, sz, sz, u64, ctypes.c_int, vp, vp, vp, vp, vp]
        L.luq_quant_grad.argtypes = [vp, vp, ctypes.c_int, sz, sz, vp, u64, ctypes.c_int, vp, vp, vp, vp]
        L.luq_quant_int4_hindsight.argtypes = [vp, vp, ctypes.c_int, sz, sz, vp, ctypes.c_float, vp, vp, vp, vp, vp]
        L.luq_quant_grad_nearest.argtypes = [vp, vp, ctypes.c_int, sz, sz, vp, vp, vp, vp, vp]
        L.luq_quant_grad_ablation.argtypes = [vp, vp, ctypes.c_int, sz, sz, vp, u64, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp]
        L.luq_quant_grad_pw2.argtypes = [vp, vp, ctypes.c_int, sz, sz, vp, u64, ctypes.c_int, vp, vp, vp, vp]
        L.luq_quant_grad_hindsight.argtypes = [vp, vp, ctypes.c_int, sz, sz, vp, ctypes.c_float, ctypes.c_int, u64,
                                               ctypes.c_int, vp, vp, vp, vp, vp]
        L.luq_debug_expire_wait.argtypes = [vp, vp]
        L.luq_debug_bounds_probe.argtypes = [vp, vp]
        L.luq_debug_quotient.argtypes = [vp, vp, sz, vp, vp, vp]
        L.luq_gemm_fwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, vp]
        L.luq_quant_int4_gemm_fwd.argtypes = [vp, vp, ctypes.c_int, vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, vp]
        L.luq_quant_int4_hindsight_gemm_fwd.argtypes = [vp, vp, ctypes.c_int, vp, ctypes.c_float, vp, vp, vp, vp, vp, vp, vp,
                                                        i64, i64, i64, vp]
        L.luq_gemm_bwd.argtypes = [vp, vp, vp, ctypes.c_int, vp, vp, vp, vp, vp, i64, i64, i64, vp]
        L.luq_gemm_wgrad.argtypes = [vp, vp, vp, ctypes.c_int, vp, vp, vp, vp, vp, i64, i64, i64, vp]
        L.luq_gemm_wgrad_static.argtypes = [vp, vp, ctypes.c_int, vp, vp, vp, i64, i64, i64, vp]
        L.luq_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int)]
        L.luq_launch_count.argtypes = [vp]
        L.luq_launch_count.restype = i64
        L.luq_strerror.argtypes = [ctypes.c_int]
        L.luq_strerror.restype = ctypes.c_char_p
        _lib = L
    return _lib


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return LUQ_F32
    if t.dtype == torch.bfloat16:
        return LUQ_BF16
    raise TypeError("inputs are float32 or bfloat16")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _opt(t, numel: int):
    """Pointer of an optional int8 operand-byte tensor (None -> NULL), size and type checked."""
    if t is None:
        return None
    if t.dtype != torch.int8 or t.numel() < numel or not t.is_contiguous():
        raise TypeError(f"operand bytes: contiguous int8 tensor of at least {numel} elements expected")
    return t.data_ptr()


def _check(rc: int, what: str):
    if rc != 0:
        raise LuqError(rc, what)


class Context:
    """Owns one luq_ctx (status word + split workspace) on a device."""

    def __init__(self, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: this library has no CPU path")
        self.device = device
        h = ctypes.c_void_p()
        _check(load().luq_create(ctypes.byref(h), device), "luq_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            load().luq_destroy(self.handle)
            self.handle = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def set_option(self, option: int, value: int):
        _check(load().luq_set_option(self.handle, option, value), "luq_set_option")
        if option == OPT_OUTPUT_BF16:
            self.out_dtype = torch.bfloat16 if value else torch.float32
        if option == OPT_SUM_SAMPLES:
            self.sum_samples = bool(value)

    def _planes(self, n_samples: int) -> int:
        """Operand planes the LUQ quantizers write / the gradient products read: one per sample, or one in all."""
        return 1 if getattr(self, "sum_samples", False) else n_samples

    def _out(self, out, rows: int, cols: int, device):
        """Output tensor of a GEMM: the caller's (type checked) or a new one of the context's output type."""
        dtype = getattr(self, "out_dtype", torch.float32)
        if out is None:
            return torch.empty((rows, cols), dtype=dtype, device=device)
        if out.dtype != dtype or out.numel() < rows * cols or not out.is_contiguous():
            raise TypeError(f"GEMM output: contiguous {dtype} tensor of {rows} x {cols} expected")
        return out

    @property
    def launches(self) -> int:
        return int(load().luq_launch_count(self.handle))

    # ---- the path ----------------------------------------------------------
    def amax(self, x: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
        out = torch.empty(1, dtype=torch.float32, device=x.device) if out is None else out
        _check(load().luq_amax(self.handle, x.data_ptr(), _dtype_code(x), x.numel(), out.data_ptr(), _stream()),
               "luq_amax")
        return out

    # `operand` (optional, int8, one byte per element and sample): filled with the tensor-core
    # operand bytes in the same pass; hand it to the GEMMs together with the codes.
    def quant_int4(self, x: torch.Tensor, clip: torch.Tensor, codes: torch.Tensor | None = None,
                   scale: torch.Tensor | None = None, operand: torch.Tensor | None = None):
        rows, cols = (x.shape[0], x.numel() // max(x.shape[0], 1)) if x.dim() > 1 else (1, x.numel())
        codes = torch.empty(x.numel() // 2, dtype=torch.uint8, device=x.device) if codes is None else codes
        scale = torch.empty(1, dtype=torch.float32, device=x.device) if scale is None else scale
        _check(load().luq_quant_int4(self.handle, x.data_ptr(), _dtype_code(x), rows, cols, clip.data_ptr(),
                                     codes.data_ptr(), scale.data_ptr(), _opt(operand, x.numel()), _stream()),
               "luq_quant_int4")
        return codes, scale

    # ---- several tensors in one launch (host arrays of device pointers) -----------------------
    @staticmethod
    def _ptr_array(tensors):
        return (ctypes.c_void_p * len(tensors))(*[None if t is None else t.data_ptr() for t in tensors])

    def amax_multi(self, xs, outs=None):
        """max|x| of up to four tensors of one element type in one launch."""
        outs = [torch.empty(1, dtype=torch.float32, device=x.device) for x in xs] if outs is None else outs
        n = (ctypes.c_size_t * len(xs))(*[x.numel() for x in xs])
        _check(load().luq_amax_multi(self.handle, len(xs), self._ptr_array(xs), _dtype_code(xs[0]), n,
                                     self._ptr_array(outs), _stream()), "luq_amax_multi")
        return outs

    def quant_int4_multi(self, xs, clips, codes=None, scales=None, operands=None):
        """quant_int4 of up to four tensors of one element type in one launch; operands[i] may be None."""
        codes = [torch.empty(x.numel() // 2, dtype=torch.uint8, device=x.device) for x in xs] if codes is None else codes
        scales = [torch.empty(1, dtype=torch.float32, device=x.device) for x in xs] if scales is None else scales
        operands = [None] * len(xs) if operands is None else operands
        for x, o in zip(xs, operands):
            _opt(o, x.numel())
        n = (ctypes.c_size_t * len(xs))(*[x.numel() for x in xs])
        _check(load().luq_quant_int4_multi(self.handle, len(xs), self._ptr_array(xs), _dtype_code(xs[0]), n,
                                           self._ptr_array(clips), self._ptr_array(codes), self._ptr_array(scales),
                                           self._ptr_array(operands), _stream()), "luq_quant_int4_multi")
        return codes, scales

    def quant_uint4(self, x: torch.Tensor, clip: torch.Tensor, codes: torch.Tensor | None = None,
                    scale: torch.Tensor | None = None, operand: torch.Tensor | None = None):
        """Unsigned INT4 (0..15, scale = clip / 15) for non-negative tensors."""
        rows, cols = (x.shape[0], x.numel() // max(x.shape[0], 1)) if x.dim() > 1 else (1, x.numel())
        codes = torch.empty(x.numel() // 2, dtype=torch.uint8, device=x.device) if codes is None else codes
        scale = torch.empty(1, dtype=torch.float32, device=x.device) if scale is None else scale
        _check(load().luq_quant_uint4(self.handle, x.data_ptr(), _dtype_code(x), rows, cols, clip.data_ptr(),
                                      codes.data_ptr(), scale.data_ptr(), _opt(operand, x.numel()), _stream()),
               "luq_quant_uint4")
        return codes, scale

    def quant_int4_hindsight(self, x: torch.Tensor, c_hat: torch.Tensor, eta: float, codes: torch.Tensor | None = None,
                             scale: torch.Tensor | None = None, measured: torch.Tensor | None = None,
                             operand: torch.Tensor | None = None):
        """One pass: INT4 codes with the clip estimate in `c_hat`, this tensor's maximum into `measured`,
        `c_hat` replaced by the estimate for the next step.  Returns (codes, scale, measured)."""
        rows, cols = (x.shape[0], x.numel() // max(x.shape[0], 1)) if x.dim() > 1 else (1, x.numel())
        codes = torch.empty(x.numel() // 2, dtype=torch.uint8, device=x.device) if codes is None else codes
        scale = torch.empty(1, dtype=torch.float32, device=x.device) if scale is None else scale
        measured = torch.empty(1, dtype=torch.float32, device=x.device) if measured is None else measured
        _check(load().luq_quant_int4_hindsight(self.handle, x.data_ptr(), _dtype_code(x), rows, cols, c_hat.data_ptr(),
                                               eta, codes.data_ptr(), scale.data_ptr(), measured.data_ptr(),
                                               _opt(operand, x.numel()), _stream()), "luq_quant_int4_hindsight")
        return codes, scale, measured

    def amax_quant_int4(self, x: torch.Tensor, amax: torch.Tensor | None = None, codes: torch.Tensor | None = None,
                        scale: torch.Tensor | None = None, operand: torch.Tensor | None = None):
        """amax + quant_int4 in one kernel; returns (amax, codes, scale)."""
        rows, cols = (x.shape[0], x.numel() // max(x.shape[0], 1)) if x.dim() > 1 else (1, x.numel())
        amax = torch.empty(1, dtype=torch.float32, device=x.device) if amax is None else amax
        codes = torch.empty(x.numel() // 2, dtype=torch.uint8, device=x.device) if codes is None else codes
        scale = torch.empty(1, dtype=torch.float32, device=x.device) if scale is None else scale
        _check(load().luq_amax_quant_int4(self.handle, x.data_ptr(), _dtype_code(x), rows, cols, amax.data_ptr(),
                                          codes.data_ptr(), scale.data_ptr(), _opt(operand, x.numel()), _stream()),
               "luq_amax_quant_int4")
        return amax, codes, scale

    def amax_quant_grad(self, g: torch.Tensor, seed: int, n_samples: int = 1, amax: torch.Tensor | None = None,
                        codes: torch.Tensor | None = None, alpha: torch.Tensor | None = None,
                        operand: torch.Tensor | None = None):
        """amax + quant_grad in one kernel; returns (amax, codes, alpha)."""
        rows, cols = (g.shape[0], g.numel() // max(g.shape[0], 1)) if g.dim() > 1 else (1, g.numel())
        amax = torch.empty(1, dtype=torch.float32, device=g.device) if amax is None else amax
        if codes is None:
            codes = torch.empty((n_samples, g.numel() // 2), dtype=torch.uint8, device=g.device)
        alpha = torch.empty(1, dtype=torch.float32, device=g.device) if alpha is None else alpha
        _check(load().luq_amax_quant_grad(self.handle, g.data_ptr(), _dtype_code(g), rows, cols,
                                          seed & (2 ** 64 - 1), n_samples, amax.data_ptr(), codes.data_ptr(),
                                          alpha.data_ptr(), _opt(operand, self._planes(n_samples) * g.numel()), _stream()),
               "luq_amax_quant_grad")
        return amax, codes, alpha

    def quant_grad(self, g: torch.Tensor, amax: torch.Tensor, seed: int, n_samples: int = 1,
                   codes: torch.Tensor | None = None, alpha: torch.Tensor | None = None,
                   operand: torch.Tensor | None = None):
        rows, cols = (g.shape[0], g.numel() // max(g.shape[0], 1)) if g.dim() > 1 else (1, g.numel())
        if codes is None:
            codes = torch.empty((n_samples, g.numel() // 2), dtype=torch.uint8, device=g.device)
        alpha = torch.empty(1, dtype=torch.float32, device=g.device) if alpha is None else alpha
        _check(load().luq_quant_grad(self.handle, g.data_ptr(), _dtype_code(g), rows, cols, amax.data_ptr(),
                                     seed & (2 ** 64 - 1), n_samples, codes.data_ptr(), alpha.data_ptr(),
                                     _opt(operand, self._planes(n_samples) * g.numel()), _stream()), "luq_quant_grad")
        return codes, alpha

    def quant_grad_nearest(self, g: torch.Tensor, amax: torch.Tensor, codes: torch.Tensor | None = None,
                           alpha: torch.Tensor | None = None, operand: torch.Tensor | None = None):
        """Deterministic round-to-nearest-power on the LUQ grid (the biased FP4 baseline)."""
        rows, cols = (g.shape[0], g.numel() // max(g.shape[0], 1)) if g.dim() > 1 else (1, g.numel())
        codes = torch.empty((1, g.numel() // 2), dtype=torch.uint8, device=g.device) if codes is None else codes
        alpha = torch.empty(1, dtype=torch.float32, device=g.device) if alpha is None else alpha
        _check(load().luq_quant_grad_nearest(self.handle, g.data_ptr(), _dtype_code(g), rows, cols, amax.data_ptr(),
                                             codes.data_ptr(), alpha.data_ptr(), _opt(operand, g.numel()),
                                             _stream()), "luq_quant_grad_nearest")
        return codes, alpha

    def quant_grad_ablation(self, g: torch.Tensor, amax: torch.Tensor, seed: int, scheme: int, n_samples: int = 1,
                            codes: torch.Tensor | None = None, scale: torch.Tensor | None = None,
                            operand: torch.Tensor | None = None):
        """The ablation's other gradient quantizers (SCHEME_*): one region of the LUQ grid deterministic,
        or the uniform INT4 grid with stochastic rounding.  Returns (codes[n_samples, n/2], scale)."""
        rows, cols = (g.shape[0], g.numel() // max(g.shape[0], 1)) if g.dim() > 1 else (1, g.numel())
        if codes is None:
            codes = torch.empty((n_samples, g.numel() // 2), dtype=torch.uint8, device=g.device)
        scale = torch.empty(1, dtype=torch.float32, device=g.device) if scale is None else scale
        _check(load().luq_quant_grad_ablation(self.handle, g.data_ptr(), _dtype_code(g), rows, cols, amax.data_ptr(),
                                              seed, n_samples, scheme, codes.data_ptr(), scale.data_ptr(),
                                              _opt(operand, n_samples * g.numel()), _stream()),
               "luq_quant_grad_ablation")
        return codes, scale

    def quant_grad_pw2(self, g: torch.Tensor, amax: torch.Tensor, seed: int, n_samples: int = 1,
                       codes: torch.Tensor | None = None, alpha: torch.Tensor | None = None,
                       operand: torch.Tensor | None = None):
        rows, cols = (g.shape[0], g.numel() // max(g.shape[0], 1)) if g.dim() > 1 else (1, g.numel())
        if codes is None:
            codes = torch.empty((n_samples, g.numel() // 2), dtype=torch.uint8, device=g.device)
        alpha = torch.empty(1, dtype=torch.float32, device=g.device) if alpha is None else alpha
        _check(load().luq_quant_grad_pw2(self.handle, g.data_ptr(), _dtype_code(g), rows, cols, amax.data_ptr(),
                                         seed & (2 ** 64 - 1), n_samples, codes.data_ptr(), alpha.data_ptr(),
                                         _opt(operand, self._planes(n_samples) * g.numel()), _stream()), "luq_quant_grad_pw2")
        return codes, alpha

    def quant_grad_hindsight(self, g: torch.Tensor, m_hat: torch.Tensor, eta: float, seed: int, n_samples: int = 1,
                             pw2: bool = False, codes: torch.Tensor | None = None,
                             alpha: torch.Tensor | None = None, measured: torch.Tensor | None = None,
                             operand: torch.Tensor | None = None):
        """One pass: quantize with the estimate in `m_hat`, measure this tensor's maximum into
        `measured`, replace `m_hat` by the estimate for the next step."""
        rows, cols = (g.shape[0], g.numel() // max(g.shape[0], 1)) if g.dim() > 1 else (1, g.numel())
        if codes is None:
            codes = torch.empty((n_samples, g.numel() // 2), dtype=torch.uint8, device=g.device)
        alpha = torch.empty(1, dtype=torch.float32, device=g.device) if alpha is None else alpha
        measured = torch.empty(1, dtype=torch.float32, device=g.device) if measured is None else measured
        _check(load().luq_quant_grad_hindsight(self.handle, g.data_ptr(), _dtype_code(g), rows, cols,
                                               m_hat.data_ptr(), eta, int(pw2), seed & (2 ** 64 - 1), n_samples,
                                               codes.data_ptr(), alpha.data_ptr(), measured.data_ptr(),
                                               _opt(operand, self._planes(n_samples) * g.numel()), _stream()),
               "luq_quant_grad_hindsight")
        return codes, alpha, measured

    def debug_expire_wait(self):
        """Launches a kernel whose bounded wait runs out; status() then reports STATUS_TIMEOUT."""
        _check(load().luq_debug_expire_wait(self.handle, _stream()), "luq_debug_expire_wait")

    def debug_bounds_probe(self):
        """Puts an out-of-region address to the checking build's bounds check (nothing is accessed)."""
        _check(load().luq_debug_bounds_probe(self.handle, _stream()), "luq_debug_bounds_probe")

    def debug_quotient(self, x: torch.Tensor, amax: torch.Tensor) -> torch.Tensor:
        out = torch.empty_like(x, dtype=torch.float32)
        _check(load().luq_debug_quotient(self.handle, x.data_ptr(), x.numel(), amax.data_ptr(), out.data_ptr(),
                                         _stream()), "luq_debug_quotient")
        return out

    def gemm_fwd(self, a_codes, sa, w_codes, sw, M: int, N: int, K: int, out: torch.Tensor | None = None,
                 a_operand: torch.Tensor | None = None, w_operand: torch.Tensor | None = None):
        out = self._out(out, M, N, a_codes.device)
        _check(load().luq_gemm_fwd(self.handle, a_codes.data_ptr(), sa.data_ptr(), _opt(a_operand, M * K),
                                   w_codes.data_ptr(), sw.data_ptr(), _opt(w_operand, N * K), out.data_ptr(),
                                   M, N, K, _stream()), "luq_gemm_fwd")
        return out

    def quant_int4_gemm_fwd(self, a: torch.Tensor, clip: torch.Tensor, w_codes, sw, M: int, N: int, K: int,
                            a_codes: torch.Tensor | None = None, sa: torch.Tensor | None = None,
                            out: torch.Tensor | None = None, w_operand: torch.Tensor | None = None):
        """quant_int4(a) and gemm_fwd in one kernel (layers with N <= 256); returns (a_codes, sa, Z)."""
        if a.numel() != M * K or not a.is_contiguous():
            raise TypeError(f"activations: contiguous tensor of {M} x {K} expected")
        a_codes = torch.empty(M * K // 2, dtype=torch.uint8, device=a.device) if a_codes is None else a_codes
        sa = torch.empty(1, dtype=torch.float32, device=a.device) if sa is None else sa
        out = self._out(out, M, N, a.device)
        _check(load().luq_quant_int4_gemm_fwd(self.handle, a.data_ptr(), _dtype_code(a), clip.data_ptr(),
                                              a_codes.data_ptr(), sa.data_ptr(), w_codes.data_ptr(), sw.data_ptr(),
                                              _opt(w_operand, N * K), out.data_ptr(), M, N, K, _stream()),
               "luq_quant_int4_gemm_fwd")
        return a_codes, sa, out

    def quant_int4_hindsight_gemm_fwd(self, a: torch.Tensor, c_hat: torch.Tensor, eta: float, w_codes, sw,
                                      M: int, N: int, K: int, a_codes: torch.Tensor | None = None,
                                      sa: torch.Tensor | None = None, measured: torch.Tensor | None = None,
                                      out: torch.Tensor | None = None, w_operand: torch.Tensor | None = None):
        """quant_int4_hindsight(a) and gemm_fwd in one kernel (layers with N <= 256): quantizes with the
        estimate in `c_hat`, measures max|a| into `measured`, replaces `c_hat` by the estimate for the next
        step; returns (a_codes, sa, measured, Z)."""
        if a.numel() != M * K or not a.is_contiguous():
            raise TypeError(f"activations: contiguous tensor of {M} x {K} expected")
        a_codes = torch.empty(M * K // 2, dtype=torch.uint8, device=a.device) if a_codes is None else a_codes
        sa = torch.empty(1, dtype=torch.float32, device=a.device) if sa is None else sa
        measured = torch.empty(1, dtype=torch.float32, device=a.device) if measured is None else measured
        out = self._out(out, M, N, a.device)
        _check(load().luq_quant_int4_hindsight_gemm_fwd(self.handle, a.data_ptr(), _dtype_code(a), c_hat.data_ptr(), eta,
                                                        a_codes.data_ptr(), sa.data_ptr(), measured.data_ptr(),
                                                        w_codes.data_ptr(), sw.data_ptr(), _opt(w_operand, N * K),
                                                        out.data_ptr(), M, N, K, _stream()),
               "luq_quant_int4_hindsight_gemm_fwd")
        return a_codes, sa, measured, out

    def gemm_bwd(self, g_codes, alpha, n_samples: int, w_codes, sw, M: int, N: int, K: int,
                 out: torch.Tensor | None = None, g_operand: torch.Tensor | None = None,
                 w_operand: torch.Tensor | None = None):
        out = self._out(out, M, K, g_codes.device)
        _check(load().luq_gemm_bwd(self.handle, g_codes.data_ptr(), alpha.data_ptr(), n_samples,
                                   _opt(g_operand, self._planes(n_samples) * M * N), w_codes.data_ptr(), sw.data_ptr(),
                                   _opt(w_operand, N * K), out.data_ptr(), M, N, K, _stream()), "luq_gemm_bwd")
        return out

    def gemm_wgrad(self, g_codes, alpha, n_samples: int, a_codes, sa, M: int, N: int, K: int,
                   out: torch.Tensor | None = None, g_operand: torch.Tensor | None = None,
                   a_operand: torch.Tensor | None = None):
        out = self._out(out, N, K, g_codes.device)
        _check(load().luq_gemm_wgrad(self.handle, g_codes.data_ptr(), alpha.data_ptr(), n_samples,
                                     _opt(g_operand, self._planes(n_samples) * M * N), a_codes.data_ptr(), sa.data_ptr(),
                                     _opt(a_operand, M * K), out.data_ptr(), M, N, K, _stream()), "luq_gemm_wgrad")
        return out

    def status(self) -> int:
        """Synchronises the current stream; returns and clears the device status bits."""
        flags = ctypes.c_int(0)
        _check(load().luq_status(self.handle, _stream(), ctypes.byref(flags)), "luq_status")
        return flags.value


def gemm_wgrad_static(g_codes, alpha, n_samples: int, a_codes, sa, M: int, N: int, K: int,
                      out: torch.Tensor) -> torch.Tensor:
    """Update GEMM through the entry point that allocates nothing: no context, the
    split workspace is a fixed array inside the library.  `out` must be supplied by
    the caller (this wrapper does not allocate either).  Runs on the current device."""
    _check(load().luq_gemm_wgrad_static(g_codes.data_ptr(), alpha.data_ptr(), n_samples, a_codes.data_ptr(),
                                        sa.data_ptr(), out.data_ptr(), M, N, K, _stream()),
           "luq_gemm_wgrad_static")
    return out


def kmax() -> int:
    return int(load().luq_kmax())


def debug_build() -> bool:
    """True if the loaded library is the bounds-checking build (-DLUQ_DEBUG)."""
    return bool(load().luq_debug_build())
