"""Thin ctypes binding over libdps.so: same names as the C ABI, argument marshalling only.

Every computation runs inside the CUDA library.  PyTorch is used for device memory and
streams.  If the library has not been built the import of a function fails loudly; there is
no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional, Sequence, Tuple

import torch

DPS_MODE_FAST, DPS_MODE_FULL = 0, 1
DPS_ENC_AUTO, DPS_ENC_E4M3, DPS_ENC_E5M2 = 0, 1, 2
DPS_ENC_E4M3_RN, DPS_ENC_E5M2_RN = 3, 4      # rounded nests
DPS_ENC_AUTO_RN = 5                          # dps_split_weights only: AUTO's rule, rounded nests
DPS_OK = 0
DPS_ERR_NULL, DPS_ERR_SHAPE, DPS_ERR_MODE, DPS_ERR_ENCODING, DPS_ERR_ALIGN = 1, 2, 3, 4, 5
DPS_ERR_UNSUPPORTED, DPS_ERR_CUDA, DPS_ERR_DATA, DPS_ERR_WORKSPACE = 6, 7, 8, 9

LIB_PATH = Path(__file__).resolve().parent / "libdps.so"

# name -> (restype, argtypes); must list every function include/dps.h declares
_vp, _i64, _i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
ABI = {
    "dps_split_weights": (ctypes.c_int, [_vp, _vp, _vp, _i64, _i64, ctypes.POINTER(_i32), _vp]),
    "dps_reconstruct": (ctypes.c_int, [_vp, _vp, _vp, _i64, _i64, _i32, _vp]),
    "dps_linear": (ctypes.c_int, [_i32, _i32, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp]),
    "dps_moe_linear": (ctypes.c_int, [_i32, ctypes.POINTER(_i32), _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64,
                                      _i64, _i32, _vp, ctypes.c_size_t, _vp]),
    "dps_moe_linear_static": (ctypes.c_int, [_i32, ctypes.POINTER(_i32), _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64,
                                             _i64, _i32, _vp]),
    "dps_moe_workspace_bytes": (ctypes.c_size_t, [_i64, _i32, _i64]),
    "dps_quantize_activations": (ctypes.c_int, [_vp, _vp, _vp, _i64, _i64, _vp]),
    "dps_linear_fp8act": (ctypes.c_int, [_i32, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp]),
    "dps_backup_residual": (ctypes.c_int, [_vp, _vp, ctypes.c_size_t, ctypes.c_size_t, _vp]),
    "dps_restore_residual": (ctypes.c_int, [_vp, _vp, ctypes.c_size_t, ctypes.c_size_t, _vp]),
    "dps_stream_status": (ctypes.c_int, [_vp]),
    "dps_debug_wait_timeout": (ctypes.c_int, [ctypes.c_uint64, _vp]),
    "dps_launch_count": (_i64, []),
    "dps_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "dps_version": (ctypes.c_int, []),
}

_lib = None


class DpsError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {status_string(status)} (dps_status {status})")
        self.status = status


def library() -> ctypes.CDLL:
    """Load libdps.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2609_34380_b200.build` "
                "(there is no fallback path)")
        lib = ctypes.CDLL(str(LIB_PATH))
        for name, (res, args) in ABI.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return library().dps_status_string(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != DPS_OK:
        raise DpsError(status, what)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dev(t: Optional[torch.Tensor], dtype, what: str) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{what} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{what} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{what} must be contiguous")
    return t.data_ptr()


def dps_split_weights(w_fp16: torch.Tensor, enc: int = DPS_ENC_AUTO, w_persist: Optional[torch.Tensor] = None,
                      w_resid: Optional[torch.Tensor] = None, stream=None) -> Tuple[torch.Tensor, torch.Tensor, int]:
    """FP16 W[rows][cols] -> (persistent plane, residual plane, encoding used)."""
    rows, cols = w_fp16.shape
    if w_persist is None:
        w_persist = torch.empty((rows, cols), dtype=torch.uint8, device=w_fp16.device)
    if w_resid is None:
        w_resid = torch.empty((rows, cols), dtype=torch.uint8, device=w_fp16.device)
    enc_io = _i32(int(enc))
    st = library().dps_split_weights(_dev(w_fp16, torch.float16, "w_fp16"), _dev(w_persist, torch.uint8, "w_persist"),
                                     _dev(w_resid, torch.uint8, "w_resid"), rows, cols, ctypes.byref(enc_io),
                                     _stream(stream))
    _check(st, "dps_split_weights")
    return w_persist, w_resid, int(enc_io.value)


def dps_reconstruct(w_persist: torch.Tensor, w_resid: Optional[torch.Tensor], enc: int,
                    w_fp16_out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """(P, R) -> the original FP16 weights; R = None gives the fast-mode weights."""
    rows, cols = w_persist.shape
    if w_fp16_out is None:
        w_fp16_out = torch.empty((rows, cols), dtype=torch.float16, device=w_persist.device)
    st = library().dps_reconstruct(_dev(w_persist, torch.uint8, "w_persist"), _dev(w_resid, torch.uint8, "w_resid"),
                                   _dev(w_fp16_out, torch.float16, "w_fp16_out"), rows, cols, int(enc),
                                   _stream(stream))
    _check(st, "dps_reconstruct")
    return w_fp16_out


def dps_linear(mode: int, enc: int, x: torch.Tensor, w_persist: torch.Tensor, w_resid: Optional[torch.Tensor],
               y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """y[M][N] = x[M][K] * W_eff^T from the planes, in fast or full mode."""
    M, K = x.shape
    N, K2 = w_persist.shape
    if K != K2:
        raise ValueError(f"K mismatch: x has {K}, planes have {K2}")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=x.device)
    st = library().dps_linear(int(mode), int(enc), _dev(x, torch.float16, "x"),
                              _dev(w_persist, torch.uint8, "w_persist"), _dev(w_resid, torch.uint8, "w_resid"),
                              _dev(y, torch.float16, "y"), M, N, K, _stream(stream))
    _check(st, "dps_linear")
    return y


def dps_moe_workspace_bytes(A: int, E: int, K: int) -> int:
    return int(library().dps_moe_workspace_bytes(int(A), int(E), int(K)))


def dps_moe_linear(mode: int, enc_per_expert: Sequence[int], x: torch.Tensor, token_of_row: Optional[torch.Tensor],
                   expert_of_row: torch.Tensor, w_persist: torch.Tensor, w_resid: Optional[torch.Tensor],
                   y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                   stream=None) -> torch.Tensor:
    """Grouped linear: y[a] = x[token_of_row[a]] * W_eff(expert_of_row[a])^T."""
    E, N, K = w_persist.shape
    T, K2 = x.shape
    if K != K2:
        raise ValueError(f"K mismatch: x has {K}, planes have {K2}")
    A = expert_of_row.numel()
    if y is None:
        y = torch.empty((A, N), dtype=torch.float16, device=x.device)
    if workspace is None:
        workspace = torch.empty(max(dps_moe_workspace_bytes(A, E, K), 16), dtype=torch.uint8, device=x.device)
    enc_arr = (_i32 * E)(*[int(e) for e in enc_per_expert])
    st = library().dps_moe_linear(int(mode), enc_arr, _dev(x, torch.float16, "x"),
                                  _dev(token_of_row, torch.int32, "token_of_row"),
                                  _dev(expert_of_row, torch.int32, "expert_of_row"),
                                  _dev(w_persist, torch.uint8, "w_persist"), _dev(w_resid, torch.uint8, "w_resid"),
                                  _dev(y, torch.float16, "y"), A, T, N, K, E,
                                  _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream))
    _check(st, "dps_moe_linear")
    return y


DPS_MOE_STATIC_SCRATCH_BYTES = 16 << 20


def dps_moe_linear_static(mode: int, enc_per_expert: Sequence[int], x: torch.Tensor,
                          token_of_row: Optional[torch.Tensor], expert_of_row: torch.Tensor,
                          w_persist: torch.Tensor, w_resid: Optional[torch.Tensor], y: torch.Tensor,
                          stream=None) -> torch.Tensor:
    """Grouped linear for callers that must not allocate: same result as dps_moe_linear, scratch
    kept in a fixed 16 MiB array inside the library.  The caller passes inputs and the output
    tensor; nothing is allocated here either.  Problems that need more scratch raise DpsError
    (DPS_ERR_WORKSPACE).  Calls share the array, so keep them ordered on the GPU."""
    E, N, K = w_persist.shape
    T, K2 = x.shape
    if K != K2:
        raise ValueError(f"K mismatch: x has {K}, planes have {K2}")
    A = expert_of_row.numel()
    enc_arr = (_i32 * E)(*[int(e) for e in enc_per_expert])
    st = library().dps_moe_linear_static(int(mode), enc_arr, _dev(x, torch.float16, "x"),
                                         _dev(token_of_row, torch.int32, "token_of_row"),
                                         _dev(expert_of_row, torch.int32, "expert_of_row"),
                                         _dev(w_persist, torch.uint8, "w_persist"),
                                         _dev(w_resid, torch.uint8, "w_resid"), _dev(y, torch.float16, "y"), A, T,
                                         N, K, E, _stream(stream))
    _check(st, "dps_moe_linear_static")
    return y


def dps_quantize_activations(x: torch.Tensor, x_fp8: Optional[torch.Tensor] = None,
                             scale: Optional[torch.Tensor] = None, stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """FP16 x[M][K] -> (E4M3 codes uint8 [M][K], per-token scale float32 [M])."""
    M, K = x.shape
    if x_fp8 is None:
        x_fp8 = torch.empty((M, K), dtype=torch.uint8, device=x.device)
    if scale is None:
        scale = torch.empty((M,), dtype=torch.float32, device=x.device)
    st = library().dps_quantize_activations(_dev(x, torch.float16, "x"), _dev(x_fp8, torch.uint8, "x_fp8"),
                                            _dev(scale, torch.float32, "scale"), M, K, _stream(stream))
    _check(st, "dps_quantize_activations")
    return x_fp8, scale


def dps_linear_fp8act(enc: int, x_fp8: torch.Tensor, scale: torch.Tensor, w_persist: torch.Tensor,
                      y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Fast mode with FP8 activations: y[M][N] = scale[m] * x_fp8 * W_fast^T on the FP8 tensor cores."""
    M, K = x_fp8.shape
    N, K2 = w_persist.shape
    if K != K2:
        raise ValueError(f"K mismatch: x_fp8 has {K}, the plane has {K2}")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=x_fp8.device)
    st = library().dps_linear_fp8act(int(enc), _dev(x_fp8, torch.uint8, "x_fp8"), _dev(scale, torch.float32, "scale"),
                                     _dev(w_persist, torch.uint8, "w_persist"), _dev(y, torch.float16, "y"), M, N, K,
                                     _stream(stream))
    _check(st, "dps_linear_fp8act")
    return y


def _host_bytes(t: torch.Tensor, what: str) -> int:
    if t.is_cuda or t.dtype != torch.uint8 or not t.is_contiguous():
        raise ValueError(f"{what} must be a contiguous uint8 host tensor (pinned, for the copies to be asynchronous)")
    return t.data_ptr()


def dps_backup_residual(w_resid: torch.Tensor, backup_host: Optional[torch.Tensor] = None, chunk_bytes: int = 0,
                        stream=None) -> torch.Tensor:
    """Copy a residual plane to (pinned) host memory in chunks; returns the host tensor."""
    if backup_host is None:
        backup_host = torch.empty(w_resid.shape, dtype=torch.uint8, pin_memory=True)
    if backup_host.numel() != w_resid.numel():
        raise ValueError("backup_host has the wrong size")
    st = library().dps_backup_residual(_dev(w_resid, torch.uint8, "w_resid"), _host_bytes(backup_host, "backup_host"),
                                       w_resid.numel(), int(chunk_bytes), _stream(stream))
    _check(st, "dps_backup_residual")
    return backup_host


def dps_restore_residual(w_resid: torch.Tensor, backup_host: torch.Tensor, chunk_bytes: int = 0, stream=None) -> None:
    """Copy a residual plane back from its host copy in chunks, on `stream`, without synchronising."""
    if backup_host.numel() != w_resid.numel():
        raise ValueError("backup_host has the wrong size")
    st = library().dps_restore_residual(_dev(w_resid, torch.uint8, "w_resid"), _host_bytes(backup_host, "backup_host"),
                                        w_resid.numel(), int(chunk_bytes), _stream(stream))
    _check(st, "dps_restore_residual")


def dps_stream_status(stream=None) -> int:
    """Synchronise the stream; return and clear the device status word."""
    return int(library().dps_stream_status(_stream(stream)))


def dps_debug_wait_timeout(limit_ns: int, stream=None) -> None:
    """Launches the self-test of the bounded device-side wait: one warp waits `limit_ns` nanoseconds for a
    barrier nobody signals, then sets the status word (dps_stream_status reports DPS_ERR_CUDA once)."""
    _check(library().dps_debug_wait_timeout(int(limit_ns), _stream(stream)), "dps_debug_wait_timeout")


def dps_launch_count() -> int:
    return int(library().dps_launch_count())


def dps_version() -> int:
    return int(library().dps_version())
