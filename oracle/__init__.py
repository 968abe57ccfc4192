"""CPU oracle for the 4-bit training hot path.  TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front end over ``luq_oracle.c`` (plain scalar C, compiled with
gcc) plus ``literal.py`` (a pure-Python, exact-rational transcription of the
paper's two-stage quantizer used to pin the C code).  Nothing here is imported
by the CUDA library or its Python binding; only tests, the smoke check and the
benchmark's CPU-baseline leg may use it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "luq_oracle.c")
_LIB = os.path.join(_HERE, "libluq_oracle.so")
_lock = threading.Lock()
_lib = None

FLAG_NONFINITE = 1
FLAG_RANGE = 2
KMAX_DEFAULT = 4  # Eq. alpha with b = 3: alpha = max / 2^(2^(b-1)) = max / 16


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            build()
            L = ctypes.CDLL(_LIB)
            u8p, f32p, f64p = (ctypes.POINTER(ctypes.c_uint8), ctypes.POINTER(ctypes.c_float),
                               ctypes.POINTER(ctypes.c_double))
            u32p, i64p, intp = (ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_int64),
                                ctypes.POINTER(ctypes.c_int))
            sz, i64, dbl = ctypes.c_size_t, ctypes.c_int64, ctypes.c_double
            L.oracle_philox_constants.argtypes = [u32p]
            L.oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
            L.oracle_random_word.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint64]
            L.oracle_random_word.restype = ctypes.c_uint32
            L.oracle_amax.argtypes = [f32p, sz, intp]
            L.oracle_amax.restype = ctypes.c_float
            L.oracle_quant_int4.argtypes = [f32p, sz, ctypes.c_float, u8p, intp]
            L.oracle_quant_int4.restype = ctypes.c_float
            L.oracle_quant_uint4.argtypes = [f32p, sz, ctypes.c_float, u8p, intp]
            L.oracle_quant_uint4.restype = ctypes.c_float
            L.oracle_luq_alpha.argtypes = [ctypes.c_float, ctypes.c_int]
            L.oracle_luq_alpha.restype = ctypes.c_float
            L.oracle_quant_luq.argtypes = [f32p, sz, ctypes.c_float, ctypes.c_int, ctypes.c_uint64,
                                           ctypes.c_int, u8p, intp]
            L.oracle_quant_luq.restype = ctypes.c_float
            L.oracle_quant_luq_window.argtypes = [f32p, sz, ctypes.c_uint64, ctypes.c_float, ctypes.c_int,
                                                  ctypes.c_uint64, ctypes.c_int, u8p, intp]
            L.oracle_quant_luq_window.restype = ctypes.c_float
            L.oracle_quant_fp_nearest.argtypes = [f32p, sz, ctypes.c_float, ctypes.c_int, u8p, intp]
            L.oracle_quant_fp_nearest.restype = ctypes.c_float
            L.oracle_quant_fp_ablation.argtypes = [f32p, sz, ctypes.c_float, ctypes.c_int, ctypes.c_uint64,
                                                   ctypes.c_int, ctypes.c_int, ctypes.c_int, u8p, intp]
            L.oracle_quant_fp_ablation.restype = ctypes.c_float
            L.oracle_quant_int4_sr.argtypes = [f32p, sz, ctypes.c_float, ctypes.c_uint64, ctypes.c_int, u8p, intp]
            L.oracle_quant_int4_sr.restype = ctypes.c_float
            L.oracle_pw2_ceil.argtypes = [ctypes.c_float]
            L.oracle_pw2_ceil.restype = ctypes.c_float
            L.oracle_hindsight_next.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_float]
            L.oracle_hindsight_next.restype = ctypes.c_float
            L.oracle_luq_bins.argtypes = [f32p, sz, ctypes.c_float, ctypes.c_int, f64p, f64p, u32p]
            L.oracle_dequant.argtypes = [u8p, sz, dbl, ctypes.c_int, f64p]
            L.oracle_gemm_fwd.argtypes = [u8p, dbl, u8p, dbl, i64, i64, i64, f64p]
            L.oracle_gemm_bwd.argtypes = [u8p, dbl, ctypes.c_int, u8p, dbl, i64, i64, i64, f64p]
            L.oracle_gemm_wgrad.argtypes = [u8p, dbl, ctypes.c_int, u8p, dbl, i64, i64, i64, f64p]
            L.oracle_gemm_general.argtypes = [ctypes.c_int, u8p, ctypes.c_int, dbl, ctypes.c_int, u8p, ctypes.c_int, dbl,
                                              i64, i64, i64, f64p]
            L.oracle_gemm_int64.argtypes = [ctypes.c_int, u8p, ctypes.c_int, u8p, i64, i64, i64, i64p]
            L.oracle_gemm_entries.argtypes = [ctypes.c_int, u8p, dbl, ctypes.c_int, u8p, dbl,
                                              i64, i64, i64, i64p, i64p, sz, f64p]
            _lib = L
    return _lib


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def widen(x: np.ndarray) -> np.ndarray:
    """fp32 view of the input.  bf16 tensors travel as uint16 bit patterns and
    are widened exactly (bits << 16); fp32 passes through."""
    x = np.ascontiguousarray(x)
    if x.dtype == np.uint16:
        return (x.astype(np.uint32) << 16).view(np.float32)
    if x.dtype != np.float32:
        raise TypeError("oracle inputs are float32 or bf16-as-uint16")
    return x


def philox4x32_10(counter, key) -> np.ndarray:
    c = np.asarray(counter, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c, ctypes.c_uint32), _ptr(k, ctypes.c_uint32), _ptr(out, ctypes.c_uint32))
    return out


def philox_constants() -> np.ndarray:
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox_constants(_ptr(out, ctypes.c_uint32))
    return out


def random_word(seed: int, sample: int, index: int) -> int:
    return int(lib().oracle_random_word(seed & (2**64 - 1), sample, index))


def amax(x: np.ndarray):
    """max|x| over the whole tensor (Eq. alpha).  Returns (value, flags)."""
    xf = widen(x).reshape(-1)
    flags = ctypes.c_int(0)
    v = lib().oracle_amax(_ptr(xf, ctypes.c_float), xf.size, ctypes.byref(flags))
    return np.float32(v), flags.value


def quant_int4(x: np.ndarray, clip):
    """Q_INT with round-to-nearest (Sec. 3.3).  Returns (codes[n/2] uint8, scale, flags)."""
    xf = widen(x).reshape(-1)
    codes = np.zeros((xf.size + 1) // 2, dtype=np.uint8)
    flags = ctypes.c_int(0)
    s = lib().oracle_quant_int4(_ptr(xf, ctypes.c_float), xf.size, np.float32(clip),
                                _ptr(codes, ctypes.c_uint8), ctypes.byref(flags))
    return codes, np.float32(s), flags.value


def quant_uint4(x: np.ndarray, clip):
    """Unsigned INT4 (range [0, clip], s = clip/15) for non-negative tensors.  Returns (codes, scale, flags)."""
    xf = widen(x).reshape(-1)
    codes = np.zeros((xf.size + 1) // 2, dtype=np.uint8)
    flags = ctypes.c_int(0)
    s = lib().oracle_quant_uint4(_ptr(xf, ctypes.c_float), xf.size, np.float32(clip),
                                 _ptr(codes, ctypes.c_uint8), ctypes.byref(flags))
    return codes, np.float32(s), flags.value


def luq_alpha(mx, kmax: int = KMAX_DEFAULT) -> np.float32:
    return np.float32(lib().oracle_luq_alpha(np.float32(mx), kmax))


def quant_luq(x: np.ndarray, mx, seed: int, n_samples: int = 1, kmax: int = KMAX_DEFAULT,
              first_index: int = 0):
    """LUQ = Q_alpha(T_alpha(x)) (Sec. 4).  Returns (codes[n_samples, n/2], alpha, flags).
    `first_index` (even) is the position of x[0] inside the full tensor."""
    xf = widen(x).reshape(-1)
    plane = (xf.size + 1) // 2
    codes = np.zeros((n_samples, plane), dtype=np.uint8)
    flags = ctypes.c_int(0)
    a = lib().oracle_quant_luq_window(_ptr(xf, ctypes.c_float), xf.size, first_index, np.float32(mx), kmax,
                                      seed & (2**64 - 1), n_samples, _ptr(codes, ctypes.c_uint8),
                                      ctypes.byref(flags))
    return codes, np.float32(a), flags.value


def quant_fp_nearest(x: np.ndarray, mx, kmax: int = KMAX_DEFAULT):
    """Deterministic round-to-nearest-power on the LUQ grid (Eq. RC); returns (codes[1, n/2], alpha, flags)."""
    xf = widen(x).reshape(-1)
    codes = np.zeros((1, (xf.size + 1) // 2), dtype=np.uint8)
    flags = ctypes.c_int(0)
    a = lib().oracle_quant_fp_nearest(_ptr(xf, ctypes.c_float), xf.size, np.float32(mx), kmax,
                                      _ptr(codes, ctypes.c_uint8), ctypes.byref(flags))
    return codes, np.float32(a), flags.value


def quant_fp_ablation(x: np.ndarray, mx, seed: int, sr: bool, su: bool, n_samples: int = 1,
                      kmax: int = KMAX_DEFAULT):
    """The ablation's partially unbiased arms on the LUQ grid: `sr` = stochastic rounding inside the
    range, `su` = stochastic underflow below it, the other region deterministic (nearest).
    Returns (codes[n_samples, n/2], alpha, flags)."""
    xf = widen(x).reshape(-1)
    codes = np.zeros((n_samples, (xf.size + 1) // 2), dtype=np.uint8)
    flags = ctypes.c_int(0)
    a = lib().oracle_quant_fp_ablation(_ptr(xf, ctypes.c_float), xf.size, np.float32(mx), kmax, seed, n_samples,
                                       int(bool(sr)), int(bool(su)), _ptr(codes, ctypes.c_uint8), ctypes.byref(flags))
    return codes, np.float32(a), flags.value


def quant_int4_sr(x: np.ndarray, mx, seed: int, n_samples: int = 1):
    """The ablation's "INT4 unbiased" arm: grid -7..7 with step max/7 and stochastic rounding (Eq. SR).
    Returns (codes[n_samples, n/2] as INT4 nibbles, scale, flags)."""
    xf = widen(x).reshape(-1)
    codes = np.zeros((n_samples, (xf.size + 1) // 2), dtype=np.uint8)
    flags = ctypes.c_int(0)
    s = lib().oracle_quant_int4_sr(_ptr(xf, ctypes.c_float), xf.size, np.float32(mx), seed, n_samples,
                                   _ptr(codes, ctypes.c_uint8), ctypes.byref(flags))
    return codes, np.float32(s), flags.value


def pw2_ceil(mx) -> np.float32:
    """2^ceil(log2 mx): the maximum rounded up to a power of two (Appendix A.7)."""
    return np.float32(lib().oracle_pw2_ceil(np.float32(mx)))


def quant_luq_pw2(x: np.ndarray, mx, seed: int, n_samples: int = 1, kmax: int = KMAX_DEFAULT):
    """LUQ_PW2: the same quantizer with alpha = 2^ceil(log2 max) / 2^kmax."""
    return quant_luq(x, pw2_ceil(mx), seed, n_samples, kmax)


def hindsight_next(measured_max, m_hat, eta) -> np.float32:
    """m_hat for the next step: (1 - eta) * max|x| of this step + eta * m_hat of this step."""
    return np.float32(lib().oracle_hindsight_next(np.float32(measured_max), np.float32(m_hat), np.float32(eta)))


def _measured_max(x: np.ndarray):
    """max|x| as a hindsight step measures it: a tensor with an Inf or NaN element has no finite
    maximum, which the recursion must see (it then keeps its estimate)."""
    measured, mflags = amax(x)
    if mflags & FLAG_NONFINITE:
        measured = np.float32(np.inf)
    return measured, mflags


def quant_luq_hindsight(x: np.ndarray, m_hat, eta, seed: int, n_samples: int = 1, pw2: bool = False,
                        kmax: int = KMAX_DEFAULT):
    """One hindsight step: quantize x with the estimate m_hat (not with its own maximum) and return
    (codes, alpha, flags, measured max of x, m_hat for the next step)."""
    mx_used = pw2_ceil(m_hat) if pw2 else np.float32(m_hat)
    codes, alpha, flags = quant_luq(x, mx_used, seed, n_samples, kmax)
    measured, mflags = _measured_max(x)
    return codes, alpha, flags | mflags, measured, hindsight_next(measured, m_hat, eta)


def quant_int4_hindsight(x: np.ndarray, c_hat, eta):
    """One hindsight step for an INT4 tensor (Sec. 7 applied to the forward tensors): quantize x with
    the clip estimate c_hat made from earlier steps (values beyond it saturate at +-7) and return
    (codes, scale, flags, measured max of x, c_hat for the next step)."""
    codes, scale, flags = quant_int4(x, np.float32(c_hat))
    measured, mflags = _measured_max(x)
    return codes, scale, flags | mflags, measured, hindsight_next(measured, c_hat, eta)


def luq_bins(x: np.ndarray, mx, kmax: int = KMAX_DEFAULT):
    """Per element (lo, hi, thr): candidate levels in units of alpha and the
    32-bit threshold; P(hi) = thr / 2^32."""
    xf = widen(x).reshape(-1)
    lo = np.zeros(xf.size, dtype=np.float64)
    hi = np.zeros(xf.size, dtype=np.float64)
    thr = np.zeros(xf.size, dtype=np.uint32)
    lib().oracle_luq_bins(_ptr(xf, ctypes.c_float), xf.size, np.float32(mx), kmax,
                          _ptr(lo, ctypes.c_double), _ptr(hi, ctypes.c_double), _ptr(thr, ctypes.c_uint32))
    return lo, hi, thr


def unpack(codes: np.ndarray, n: int) -> np.ndarray:
    """Nibbles of a packed plane, element 2j low, 2j+1 high."""
    codes = np.ascontiguousarray(codes).reshape(-1)
    out = np.empty(codes.size * 2, dtype=np.uint8)
    out[0::2] = codes & 0xF
    out[1::2] = codes >> 4
    return out[:n]


def dequant(codes: np.ndarray, n: int, scale, kind: str) -> np.ndarray:
    """Values of a packed plane in float64.  kind: 'int4', 'luq' or 'uint4'."""
    codes = np.ascontiguousarray(codes).reshape(-1)
    out = np.zeros(n, dtype=np.float64)
    lib().oracle_dequant(_ptr(codes, ctypes.c_uint8), n, float(scale), {"int4": 0, "luq": 1, "uint4": 2}[kind],
                         _ptr(out, ctypes.c_double))
    return out


def gemm_fwd(a_codes, sa, w_codes, sw, M, N, K) -> np.ndarray:
    """Z = A_d . W_d^T in float64 (Eq. Forward)."""
    a_codes = np.ascontiguousarray(a_codes).reshape(-1)
    w_codes = np.ascontiguousarray(w_codes).reshape(-1)
    Z = np.zeros((M, N), dtype=np.float64)
    lib().oracle_gemm_fwd(_ptr(a_codes, ctypes.c_uint8), float(sa), _ptr(w_codes, ctypes.c_uint8), float(sw),
                          M, N, K, _ptr(Z, ctypes.c_double))
    return Z


def gemm_bwd(g_codes, alpha, n_samples, w_codes, sw, M, N, K) -> np.ndarray:
    """dA = (sum_s G_d,s . W_d) / n_s in float64 (Eq. Backward; Sec. 5.1 averages the samples' results)."""
    g_codes = np.ascontiguousarray(g_codes).reshape(-1)
    w_codes = np.ascontiguousarray(w_codes).reshape(-1)
    dA = np.zeros((M, K), dtype=np.float64)
    lib().oracle_gemm_bwd(_ptr(g_codes, ctypes.c_uint8), float(alpha), n_samples,
                          _ptr(w_codes, ctypes.c_uint8), float(sw), M, N, K, _ptr(dA, ctypes.c_double))
    return dA


def gemm_wgrad(g_codes, alpha, n_samples, a_codes, sa, M, N, K) -> np.ndarray:
    """dW = (sum_s G_d,s^T . A_d) / n_s in float64 (Eq. Update; Sec. 5.1 averages the samples' weight gradients)."""
    g_codes = np.ascontiguousarray(g_codes).reshape(-1)
    a_codes = np.ascontiguousarray(a_codes).reshape(-1)
    dW = np.zeros((N, K), dtype=np.float64)
    lib().oracle_gemm_wgrad(_ptr(g_codes, ctypes.c_uint8), float(alpha), n_samples,
                            _ptr(a_codes, ctypes.c_uint8), float(sa), M, N, K, _ptr(dW, ctypes.c_double))
    return dW


def gemm_general(which: str, x_codes, x_kind: str, sx, n_samples, y_codes, y_kind: str, sy, M, N, K) -> np.ndarray:
    """The three products for operands of any code kind ('int4', 'luq', 'uint4'): `x` is the
    activations (fwd) or the gradient planes (bwd, wgrad), `y` the weights (fwd, bwd) or the
    activations (wgrad).  Same definition as gemm_fwd / gemm_bwd / gemm_wgrad."""
    w = {"fwd": 0, "bwd": 1, "wgrad": 2}[which]
    kinds = {"int4": 0, "luq": 1, "uint4": 2}
    shape = {"fwd": (M, N), "bwd": (M, K), "wgrad": (N, K)}[which]
    x_codes = np.ascontiguousarray(x_codes).reshape(-1)
    y_codes = np.ascontiguousarray(y_codes).reshape(-1)
    out = np.zeros(shape, dtype=np.float64)
    lib().oracle_gemm_general(w, _ptr(x_codes, ctypes.c_uint8), kinds[x_kind], float(sx), n_samples,
                              _ptr(y_codes, ctypes.c_uint8), kinds[y_kind], float(sy), M, N, K,
                              _ptr(out, ctypes.c_double))
    return out


def gemm_int64(which: str, x_codes, n_samples, y_codes, M, N, K) -> np.ndarray:
    """Integer-code products summed in int64 (Appendix A.1 scale factoring)."""
    w = {"fwd": 0, "bwd": 1, "wgrad": 2}[which]
    shape = {"fwd": (M, N), "bwd": (M, K), "wgrad": (N, K)}[which]
    x_codes = np.ascontiguousarray(x_codes).reshape(-1)
    y_codes = np.ascontiguousarray(y_codes).reshape(-1)
    out = np.zeros(shape, dtype=np.int64)
    lib().oracle_gemm_int64(w, _ptr(x_codes, ctypes.c_uint8), n_samples, _ptr(y_codes, ctypes.c_uint8),
                            M, N, K, _ptr(out, ctypes.c_int64))
    return out


def gemm_entries(which: str, x_codes, sx, n_samples, y_codes, sy, M, N, K, rows, cols) -> np.ndarray:
    """Selected entries of one of the three products, each computed on its own."""
    w = {"fwd": 0, "bwd": 1, "wgrad": 2}[which]
    x_codes = np.ascontiguousarray(x_codes).reshape(-1)
    y_codes = np.ascontiguousarray(y_codes).reshape(-1)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    out = np.zeros(rows.size, dtype=np.float64)
    lib().oracle_gemm_entries(w, _ptr(x_codes, ctypes.c_uint8), float(sx), n_samples,
                              _ptr(y_codes, ctypes.c_uint8), float(sy), M, N, K,
                              _ptr(rows, ctypes.c_int64), _ptr(cols, ctypes.c_int64), rows.size,
                              _ptr(out, ctypes.c_double))
    return out


def host_threads() -> int:
    """Threads the OpenMP loops of the C oracle will use."""
    return int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
