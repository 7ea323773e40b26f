"""CPU oracle for the DPS dual-precision linear path (ctypes wrapper over dps_oracle.c).

TEST INFRASTRUCTURE ONLY.  Nothing in the product package may import this module:
only the tests, the smoke check and the benchmark's cpu-baseline leg use it.  It
shares no code with the CUDA library.

All arrays are numpy arrays on the host.  FP16 tensors travel as ``uint16`` words
(``arr.view(np.uint16)``) so that no conversion happens outside the C file.
Function names follow the paper's vocabulary: the *persistent* plane ``p`` (the
FP8 model kept in the persistent region), the *residual* plane ``r`` (kept in the
shared region), *fast* mode (persistent plane only) and *full* mode (both planes,
original FP16 values) -- sections "Mapper: Semi-Unified Memory Abstraction" and
"Scheduler: Dual-Precision Execution".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

MODE_FAST, MODE_FULL = 0, 1
ENC_AUTO, ENC_E4M3, ENC_E5M2 = 0, 1, 2
ENC_E4M3_RN, ENC_E5M2_RN = 3, 4          # rounded nests (an extension, see dps_oracle.c)
ENC_AUTO_RN = 5                          # split only: the AUTO rule, answering with a rounded nest
OK, ERR_ARG, ERR_DATA = 0, 1, 8

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "dps_oracle.c"
_LIB = _HERE / "libdps_oracle.so"


def build(force: bool = False) -> Path:
    """Compile dps_oracle.c with gcc (OpenMP on) next to its source."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        cmd = ["gcc", "-std=c99", "-O2", "-fPIC", "-shared", "-fopenmp", "-fno-fast-math",
               "-ffp-contract=off", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(str(build()))
        i64, i32, vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p
        L.oracle_half_to_double.restype = ctypes.c_double
        L.oracle_half_to_double.argtypes = [ctypes.c_uint16]
        L.oracle_double_to_half.restype = ctypes.c_uint16
        L.oracle_double_to_half.argtypes = [ctypes.c_double]
        L.oracle_select_encoding.restype = ctypes.c_int
        L.oracle_select_encoding.argtypes = [vp, i64]
        L.oracle_e4m3_legal.restype = ctypes.c_int
        L.oracle_e4m3_legal.argtypes = [vp, i64]
        L.oracle_rounded_legal.restype = ctypes.c_int
        L.oracle_rounded_legal.argtypes = [vp, i64, ctypes.c_int]
        L.oracle_split.restype = ctypes.c_int
        L.oracle_split.argtypes = [vp, vp, vp, i64, ctypes.c_int]
        L.oracle_reconstruct.restype = ctypes.c_int
        L.oracle_reconstruct.argtypes = [vp, vp, vp, i64, ctypes.c_int]
        L.oracle_fast_words.restype = ctypes.c_int
        L.oracle_fast_words.argtypes = [vp, vp, i64, ctypes.c_int]
        L.oracle_linear.restype = ctypes.c_int
        L.oracle_linear.argtypes = [ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, vp, i64, i64, i64,
                                    ctypes.c_int]
        L.oracle_linear_at.restype = ctypes.c_int
        L.oracle_linear_at.argtypes = [ctypes.c_int, ctypes.c_int, vp, vp, vp, i64, i64, i64, vp, vp,
                                       i64, vp]
        L.oracle_moe_linear.restype = ctypes.c_int
        L.oracle_moe_linear.argtypes = [ctypes.c_int, vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, i64,
                                        i64, i32, vp, i64, ctypes.c_int]
        L.oracle_e4m3_to_double.restype = ctypes.c_double
        L.oracle_e4m3_to_double.argtypes = [ctypes.c_uint8]
        L.oracle_float_to_e4m3.restype = ctypes.c_uint8
        L.oracle_float_to_e4m3.argtypes = [ctypes.c_float]
        L.oracle_quantize_activations.restype = ctypes.c_int
        L.oracle_quantize_activations.argtypes = [vp, vp, vp, i64, i64]
        L.oracle_linear_fp8act.restype = ctypes.c_int
        L.oracle_linear_fp8act.argtypes = [ctypes.c_int, vp, vp, vp, vp, i64, i64, i64, ctypes.c_int]
        _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: oracle status {code}")
        self.code = code


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _words(a: np.ndarray) -> np.ndarray:
    """FP16 array (float16 or uint16) -> contiguous uint16 words."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError(f"expected float16/uint16, got {a.dtype}")
    return a


def _bytes(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint8:
        raise TypeError(f"expected uint8, got {a.dtype}")
    return a


def half_to_double(word: int) -> float:
    return lib().oracle_half_to_double(int(word) & 0xFFFF)


def double_to_half(v: float) -> int:
    return lib().oracle_double_to_half(float(v))


def select_encoding(w) -> int:
    """AUTO rule: E4M3 iff every exponent MSB is zero and max|w| <= 1.75, else E5M2."""
    w = _words(w)
    return lib().oracle_select_encoding(_ptr(w), w.size)


def e4m3_legal(w) -> bool:
    w = _words(w)
    return bool(lib().oracle_e4m3_legal(_ptr(w), w.size))


def rounded_legal(w, enc: int) -> bool:
    """Whether a rounded nest (ENC_E4M3_RN / ENC_E5M2_RN) may encode these weights."""
    w = _words(w)
    return bool(lib().oracle_rounded_legal(_ptr(w), w.size, enc))


def split(w, enc: int):
    """FP16 weights -> (p, r, enc_used): the persistent and residual byte planes."""
    w = _words(w)
    if enc == ENC_AUTO:
        enc = select_encoding(w)
    elif enc == ENC_AUTO_RN:                 # the same rule; an illegal answer is refused by the split below
        enc = ENC_E4M3_RN if select_encoding(w) == ENC_E4M3 else ENC_E5M2_RN
    p = np.empty(w.shape, np.uint8)
    r = np.empty(w.shape, np.uint8)
    rc = lib().oracle_split(_ptr(w), _ptr(p), _ptr(r), w.size, enc)
    if rc != OK:
        raise OracleError(rc, "split")
    return p, r, enc


def reconstruct(p, r, enc: int) -> np.ndarray:
    """(p, r) -> the original FP16 words (uint16)."""
    p, r = _bytes(p), _bytes(r)
    w = np.empty(p.shape, np.uint16)
    rc = lib().oracle_reconstruct(_ptr(p), _ptr(r), _ptr(w), p.size, enc)
    if rc != OK:
        raise OracleError(rc, "reconstruct")
    return w


def fast_words(p, enc: int) -> np.ndarray:
    """p alone -> FP16 words of the fast-mode weights."""
    p = _bytes(p)
    w = np.empty(p.shape, np.uint16)
    rc = lib().oracle_fast_words(_ptr(p), _ptr(w), p.size, enc)
    if rc != OK:
        raise OracleError(rc, "fast_words")
    return w


def linear(mode: int, enc: int, x, p, r, threads: int = 1, want_half: bool = False):
    """y_ref[M][N] (float64) = x[M][K] * W_eff[N][K]^T.  r may be None in fast mode."""
    x, p = _words(x), _bytes(p)
    r = None if r is None else _bytes(r)
    if mode == MODE_FULL and r is None:
        raise ValueError("full mode needs the residual plane")
    M, K = x.shape
    N, K2 = p.shape
    if K != K2:
        raise ValueError("K mismatch")
    y = np.zeros((M, N), np.float64)
    yh = np.zeros((M, N), np.uint16) if want_half else None
    rc = lib().oracle_linear(mode, enc, _ptr(x), _ptr(p), _ptr(r), _ptr(y), _ptr(yh), M, N, K, threads)
    if rc != OK:
        raise OracleError(rc, "linear")
    return (y, yh) if want_half else y


def linear_at(mode: int, enc: int, x, p, r, ms, ns) -> np.ndarray:
    """Selected outputs y_ref[ms[i]][ns[i]] (float64)."""
    x, p = _words(x), _bytes(p)
    r = None if r is None else _bytes(r)
    if mode == MODE_FULL and r is None:
        raise ValueError("full mode needs the residual plane")
    M, K = x.shape
    N, _ = p.shape
    ms = np.ascontiguousarray(ms, np.int64)
    ns = np.ascontiguousarray(ns, np.int64)
    out = np.zeros(ms.shape, np.float64)
    rc = lib().oracle_linear_at(mode, enc, _ptr(x), _ptr(p), _ptr(r), M, N, K, _ptr(ms), _ptr(ns),
                                ms.size, _ptr(out))
    if rc != OK:
        raise OracleError(rc, "linear_at")
    return out


def e4m3_to_double(code: int) -> float:
    return float(lib().oracle_e4m3_to_double(int(code) & 0xFF))


def float_to_e4m3(v: float) -> int:
    """binary32 value -> E4M3 code, round to nearest even, saturating at +-448."""
    return int(lib().oracle_float_to_e4m3(float(np.float32(v))))


def quantize_activations(x):
    """FP16 words [M][K] -> (E4M3 codes uint8 [M][K], per-token scale float32 [M])."""
    x = _words(x)
    M, K = x.shape
    q = np.empty((M, K), np.uint8)
    scale = np.empty((M,), np.float32)
    rc = lib().oracle_quantize_activations(_ptr(x), _ptr(q), _ptr(scale), M, K)
    if rc != OK:
        raise OracleError(rc, "quantize_activations")
    return q, scale


def linear_fp8act(enc: int, q, scale, p, threads: int = 1) -> np.ndarray:
    """Fast-mode linear with FP8 activations: y_ref[m][n] = scale[m] * sum_k e4m3(q[m][k]) * W_fast[n][k] (float64)."""
    q, p = _bytes(q), _bytes(p)
    scale = np.ascontiguousarray(scale, np.float32)
    M, K = q.shape
    N, _ = p.shape
    y = np.zeros((M, N), np.float64)
    rc = lib().oracle_linear_fp8act(enc, _ptr(q), _ptr(scale), _ptr(p), _ptr(y), M, N, K, int(threads))
    if rc != OK:
        raise OracleError(rc, "linear_fp8act")
    return y


def moe_linear(mode: int, enc_per_expert, x, token_of_row, expert_of_row, p, r, rows=None,
               threads: int = 1, y_init=None):
    """Grouped linear.  Returns (y_ref [A][N] float64, status); rows with an
    out-of-range expert/token keep the value of y_init (zeros by default) and the
    status is ERR_DATA."""
    x, p = _words(x), _bytes(p)
    r = None if r is None else _bytes(r)
    if mode == MODE_FULL and r is None:
        raise ValueError("full mode needs the residual plane")
    E, N, K = p.shape
    T = x.shape[0]
    enc = np.ascontiguousarray(enc_per_expert, np.int32)
    eor = np.ascontiguousarray(expert_of_row, np.int32)
    tor = None if token_of_row is None else np.ascontiguousarray(token_of_row, np.int32)
    A = eor.size
    y = np.zeros((A, N), np.float64) if y_init is None else np.array(y_init, np.float64)
    sel = None if rows is None else np.ascontiguousarray(rows, np.int64)
    rc = lib().oracle_moe_linear(mode, _ptr(enc), _ptr(x), _ptr(tor), _ptr(eor), _ptr(p), _ptr(r),
                                 _ptr(y), None, A, T, N, K, E, _ptr(sel),
                                 0 if sel is None else sel.size, threads)
    if rc not in (OK, ERR_DATA):
        raise OracleError(rc, "moe_linear")
    return y, rc
