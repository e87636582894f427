"""FGMP oracle (TEST INFRASTRUCTURE): ctypes access to the plain-C reference in
``fgmp_oracle.c``.  Only tests, the smoke check and the CPU-baseline leg of the
benchmark may import this package; the CUDA library never does.

The shared object is compiled with gcc on first use (``-ffp-contract=off`` so every
single-precision step is one IEEE operation).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fgmp_oracle.c")
_LIB = os.path.join(_HERE, "libfgmp_oracle.so")

BS = 16


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call([
            "gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
            "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.oracle_e2m1_value.restype = ctypes.c_double
        L.oracle_e2m1_value.argtypes = [ctypes.c_int]
        L.oracle_e4m3_value.restype = ctypes.c_double
        L.oracle_e4m3_value.argtypes = [ctypes.c_int]
        L.oracle_e2m1_encode.restype = ctypes.c_int
        L.oracle_e2m1_encode.argtypes = [ctypes.c_float]
        L.oracle_e4m3_encode.restype = ctypes.c_int
        L.oracle_e4m3_encode.argtypes = [ctypes.c_float]
        L.oracle_clip_search.restype = ctypes.c_int
        L.oracle_clip_search.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float]
        L.oracle_clip_objective.restype = ctypes.c_float
        L.oracle_clip_objective.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_float]
        L.oracle_quantize_activations.restype = None
        L.oracle_quantize_activations.argtypes = [
            ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_float, ctypes.c_int, ctypes.c_float, ctypes.c_int, ctypes.c_float,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.oracle_quantize_weights.restype = ctypes.c_float
        L.oracle_quantize_weights.argtypes = [
            ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64,
            ctypes.c_int64, ctypes.c_int64, ctypes.c_float, ctypes.c_int, ctypes.c_float, ctypes.c_int, ctypes.c_int,
            ctypes.c_double, ctypes.c_float,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p]
        L.oracle_decode.restype = None
        L.oracle_decode.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int64, ctypes.c_int64,
                                                            ctypes.c_float, ctypes.c_int, ctypes.c_float, ctypes.c_void_p]
        L.oracle_linear.restype = None
        L.oracle_linear.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                    ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
        L.oracle_linear_sampled.restype = None
        L.oracle_linear_sampled.argtypes = (
            [ctypes.c_void_p] * 4 + [ctypes.c_float, ctypes.c_int, ctypes.c_float] +
            [ctypes.c_void_p] * 4 + [ctypes.c_float, ctypes.c_int, ctypes.c_float, ctypes.c_int64,
                                     ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.c_void_p, ctypes.c_void_p])
        L.oracle_num_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def _p(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


@dataclass
class Quantized:
    """Canonical arrays of one quantized tensor [rows, K] (see fgmp_oracle.c)."""
    rows: int
    K: int
    codes4: np.ndarray   # uint8 [rows*K/2]
    codes8: np.ndarray   # uint8 [rows*K]
    scales: np.ndarray   # uint8 [rows*K/16]
    mask: np.ndarray     # uint32 [rows*ceil(K/16/32)]
    scores: np.ndarray   # float32 [rows*K/16]
    scale_fp4: float
    ratio: int
    tau_eff: float = float("nan")
    scale_fp8: float = 0.0   # 0: tied to scale_fp4 by 2^ratio; else the FP8 tensor scale given on its own

    def mask_bits(self) -> np.ndarray:
        """bool [rows, K/16]: True = FP8 block."""
        KB = self.K // BS
        MW = (KB + 31) // 32
        w = self.mask.reshape(self.rows, MW)
        bits = (w[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1
        return bits.reshape(self.rows, MW * 32)[:, :KB].astype(bool)


def e2m1_value(code: int) -> float:
    return lib().oracle_e2m1_value(int(code))


def e4m3_value(code: int) -> float:
    return lib().oracle_e4m3_value(int(code))


def e2m1_encode(x: float) -> int:
    return lib().oracle_e2m1_encode(float(np.float32(x)))


def e4m3_encode(x: float) -> int:
    return lib().oracle_e4m3_encode(float(np.float32(x)))


def _alloc(rows: int, K: int):
    KB = K // BS
    MW = (KB + 31) // 32
    return (np.zeros(rows * K // 2, np.uint8), np.zeros(rows * K, np.uint8),
            np.zeros(rows * KB, np.uint8), np.zeros(rows * MW, np.uint32),
            np.zeros(rows * KB, np.float32))


def quantize_activations(x_bf16_bits: np.ndarray, fisher: np.ndarray, scale_fp4: float,
                         ratio: int = 3, mode: int = 0, tau: float = float("inf"), scale_fp8: float = 0.0) -> Quantized:
    """x_bf16_bits: uint16 [M, K] (bf16 bit patterns); fisher: float32 [K]."""
    M, K = x_bf16_bits.shape
    assert K % BS == 0 and x_bf16_bits.dtype == np.uint16
    x = np.ascontiguousarray(x_bf16_bits)
    f = np.ascontiguousarray(fisher, dtype=np.float32)
    c4, c8, sc, mk, scr = _alloc(M, K)
    lib().oracle_quantize_activations(_p(x), K, _p(f), M, K, float(np.float32(scale_fp4)), ratio, float(np.float32(scale_fp8)), mode,
                                      float(np.float32(tau)), _p(c4), _p(c8), _p(sc), _p(mk), _p(scr))
    return Quantized(M, K, c4, c8, sc, mk, scr, float(np.float32(scale_fp4)), ratio, float(tau), float(np.float32(scale_fp8)))


def quantize_weights(w_bf16_bits: np.ndarray, fisher: np.ndarray, scale_fp4: float = 0.0,
                     ratio: int = 3, mode: int = 0, clip: bool = True,
                     fp8_fraction: float = 0.1, tau: float = 0.0, scale_fp8: float = 0.0) -> Quantized:
    """w_bf16_bits: uint16 [N, K]; fisher: float32 [N, K] (per element)."""
    N, K = w_bf16_bits.shape
    assert K % BS == 0 and w_bf16_bits.dtype == np.uint16 and fisher.shape == (N, K)
    w = np.ascontiguousarray(w_bf16_bits)
    f = np.ascontiguousarray(fisher, dtype=np.float32)
    c4, c8, sc, mk, scr = _alloc(N, K)
    teff = ctypes.c_float(0.0)
    s4 = lib().oracle_quantize_weights(_p(w), K, _p(f), K, N, K, float(np.float32(scale_fp4)), ratio, float(np.float32(scale_fp8)), mode,
                                       int(bool(clip)), float(fp8_fraction), float(np.float32(tau)),
                                       _p(c4), _p(c8), _p(sc), _p(mk), _p(scr), ctypes.byref(teff))
    return Quantized(N, K, c4, c8, sc, mk, scr, float(s4), ratio, float(teff.value), float(np.float32(scale_fp8)))


def decode(q: Quantized) -> np.ndarray:
    """float64 [rows, K]: exact values of the quantized tensor."""
    out = np.zeros((q.rows, q.K), np.float64)
    lib().oracle_decode(_p(q.codes4), _p(q.codes8), _p(q.scales), _p(q.mask), q.rows, q.K,
                        float(np.float32(q.scale_fp4)), q.ratio, float(np.float32(q.scale_fp8)), _p(out))
    return out


def linear(a: Quantized, w: Quantized):
    """(Y, S): fp64 [M, N] product of the decoded operands and sum |a||w|."""
    assert a.K == w.K
    A, Wd = decode(a), decode(w)
    Y = np.zeros((a.rows, w.rows), np.float64)
    S = np.zeros_like(Y)
    lib().oracle_linear(_p(A), _p(Wd), a.rows, w.rows, a.K, _p(Y), _p(S))
    return Y, S


def linear_sampled(a: Quantized, w: Quantized, ms: np.ndarray, ns: np.ndarray):
    """(Y, S) at the output coordinates (ms[j], ns[j])."""
    ms = np.ascontiguousarray(ms, dtype=np.int64)
    ns = np.ascontiguousarray(ns, dtype=np.int64)
    Y = np.zeros(len(ms), np.float64)
    S = np.zeros(len(ms), np.float64)
    lib().oracle_linear_sampled(_p(a.codes4), _p(a.codes8), _p(a.scales), _p(a.mask),
                                float(np.float32(a.scale_fp4)), a.ratio, float(np.float32(a.scale_fp8)),
                                _p(w.codes4), _p(w.codes8), _p(w.scales), _p(w.mask),
                                float(np.float32(w.scale_fp4)), w.ratio, float(np.float32(w.scale_fp8)), a.K, len(ms), _p(ms), _p(ns),
                                _p(Y), _p(S))
    return Y, S


def clip_search(v: np.ndarray, f: np.ndarray, scale_fp4: float) -> int:
    v = np.ascontiguousarray(v, dtype=np.float32)
    f = np.ascontiguousarray(f, dtype=np.float32)
    return lib().oracle_clip_search(_p(v), _p(f), float(np.float32(scale_fp4)))


def clip_objective(v: np.ndarray, f: np.ndarray, c: int, scale_fp4: float) -> float:
    v = np.ascontiguousarray(v, dtype=np.float32)
    f = np.ascontiguousarray(f, dtype=np.float32)
    return lib().oracle_clip_objective(_p(v), _p(f), int(c), float(np.float32(scale_fp4)))


def num_threads() -> int:
    return lib().oracle_num_threads()


def global_threshold(score_arrays, fp8_fraction: float) -> float:
    """Global threshold of Eq. 10 (Section 3.2): one tau for several tensors, chosen so that the
    fraction R of the blocks of all of them together exceeds it.  The plain definition: pool the
    scores, k = floor(R * B + 0.5), tau = the fp32 value midway between the k-th largest score and
    the largest score strictly below it (that lower score itself if fp32 has no value between
    them; 0 if there is none below); k = 0 gives +inf, k = B gives -1 (scores are >= 0)."""
    pooled = np.concatenate([np.asarray(a, dtype=np.float32).ravel() for a in score_arrays])
    B = pooled.size
    k = int(np.floor(fp8_fraction * B + 0.5))
    if k <= 0:
        return float("inf")
    if k >= B:
        return -1.0
    s = np.sort(pooled)[::-1]
    hi = s[k - 1]
    below = s[s < hi]
    lo = below.max() if below.size else np.float32(0.0)
    t = np.float32(0.5) * np.float32(hi + lo)
    return float(t) if (lo <= t < hi) else float(lo)


def channel_mean_sq(x_bf16_bits: np.ndarray) -> np.ndarray:
    """Weights of the "Output Error" policy (Eq. 13): the average squared magnitude of every input
    channel of the other operand.  x_bf16_bits: uint16 [rows, K]; float32 [K]: rows added in order,
    one fp32 multiply and one fp32 add per element, one division by the row count."""
    x = (np.ascontiguousarray(x_bf16_bits).astype(np.uint32) << 16).view(np.float32)
    s = np.zeros(x.shape[1], np.float32)
    for r in range(x.shape[0]):
        s = (s + (x[r] * x[r]).astype(np.float32)).astype(np.float32)
    return (s / np.float32(x.shape[0])).astype(np.float32)

