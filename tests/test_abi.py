"""CPU-side checks of the C-ABI library: it loads, exports everything the header declares,
and rejects bad arguments before touching a device."""
import ctypes
import re
from pathlib import Path

import pytest

from paper_2609_34380_b200 import binding

ROOT = Path(__file__).resolve().parents[1]
HEADER = ROOT / "include" / "dps.h"


def declared_functions():
    text = HEADER.read_text()
    return sorted(set(re.findall(r"DPS_API\s+[\w\s\*]+?\b(dps_\w+)\s*\(", text)))


def test_header_functions_are_exported_and_bound():
    names = declared_functions()
    assert len(names) >= 9
    lib = binding.library()
    for name in names:
        assert hasattr(lib, name), f"{name} not exported by libdps.so"
        assert name in binding.ABI, f"{name} has no ctypes signature in the binding"
    assert sorted(binding.ABI) == names


def test_version_and_status_strings():
    assert binding.dps_version() >= 1
    seen = {binding.status_string(s) for s in range(0, 10)}
    assert len(seen) == 10 and "unknown status" not in seen
    assert binding.status_string(99) == "unknown status"


def test_workspace_size_function():
    assert binding.dps_moe_workspace_bytes(512, 8, 4096) >= 4 * (512 + 2 * 8 + 1) + 512 * 4096 * 2
    assert binding.dps_moe_workspace_bytes(0, 8, 64) > 0
    assert binding.dps_moe_workspace_bytes(-1, 8, 64) == 0
    assert binding.dps_moe_workspace_bytes(16, 0, 64) == 0
    assert binding.dps_moe_workspace_bytes(16, 2000, 64) == 0
    assert binding.dps_moe_workspace_bytes(16, 8, 0) == 0
    assert binding.dps_moe_workspace_bytes(1 << 20, 64, 1024) % 256 == 0


def test_host_validation_needs_no_device():
    lib = binding.library()
    enc = ctypes.c_int32(binding.DPS_ENC_AUTO)
    fake = ctypes.c_void_p(0x1000)       # aligned, never dereferenced: every call below fails validation first
    odd = ctypes.c_void_p(0x1004)
    # split
    assert lib.dps_split_weights(fake, fake, fake, 4, 16, None, None) == binding.DPS_ERR_NULL
    enc.value = 7
    assert lib.dps_split_weights(fake, fake, fake, 4, 16, ctypes.byref(enc), None) == binding.DPS_ERR_ENCODING
    enc.value = binding.DPS_ENC_E5M2
    assert lib.dps_split_weights(fake, fake, fake, 4, 24, ctypes.byref(enc), None) == binding.DPS_ERR_SHAPE
    assert lib.dps_split_weights(fake, fake, fake, -1, 16, ctypes.byref(enc), None) == binding.DPS_ERR_SHAPE
    assert lib.dps_split_weights(None, fake, fake, 4, 16, ctypes.byref(enc), None) == binding.DPS_ERR_NULL
    assert lib.dps_split_weights(odd, fake, fake, 4, 16, ctypes.byref(enc), None) == binding.DPS_ERR_ALIGN
    enc.value = binding.DPS_ENC_AUTO
    assert lib.dps_split_weights(None, None, None, 0, 16, ctypes.byref(enc), None) == binding.DPS_OK
    assert enc.value == binding.DPS_ENC_E4M3
    # reconstruct
    assert lib.dps_reconstruct(fake, fake, fake, 4, 16, 0, None) == binding.DPS_ERR_ENCODING
    assert lib.dps_reconstruct(fake, fake, fake, 4, 8, 2, None) == binding.DPS_ERR_SHAPE
    assert lib.dps_reconstruct(None, fake, fake, 4, 16, 2, None) == binding.DPS_ERR_NULL
    assert lib.dps_reconstruct(fake, odd, fake, 4, 16, 2, None) == binding.DPS_ERR_ALIGN
    assert lib.dps_reconstruct(None, None, None, 0, 16, 2, None) == binding.DPS_OK
    # linear
    assert lib.dps_linear(2, 1, fake, fake, fake, fake, 1, 8, 16, None) == binding.DPS_ERR_MODE
    assert lib.dps_linear(0, 0, fake, fake, fake, fake, 1, 8, 16, None) == binding.DPS_ERR_ENCODING
    assert lib.dps_linear(0, 1, fake, fake, fake, fake, 1, 8, 24, None) == binding.DPS_ERR_SHAPE
    assert lib.dps_linear(0, 1, fake, fake, fake, fake, 1, 12, 16, None) == binding.DPS_ERR_SHAPE
    assert lib.dps_linear(0, 1, fake, fake, fake, fake, -1, 8, 16, None) == binding.DPS_ERR_SHAPE
    assert lib.dps_linear(0, 1, fake, fake, None, fake, 0, 8, 16, None) == binding.DPS_OK      # M == 0
    assert lib.dps_linear(1, 1, fake, fake, None, fake, 1, 8, 16, None) == binding.DPS_ERR_NULL  # full needs R
    assert lib.dps_linear(0, 1, None, fake, None, fake, 1, 8, 16, None) == binding.DPS_ERR_NULL
    assert lib.dps_linear(0, 1, fake, odd, None, fake, 1, 8, 16, None) == binding.DPS_ERR_ALIGN
    # moe
    encs = (ctypes.c_int32 * 2)(1, 2)
    bad = (ctypes.c_int32 * 2)(1, 0)
    args = dict(A=4, T=4, N=8, K=16, E=2)
    def moe(mode=0, enc=encs, x=fake, tor=None, eor=fake, p=fake, r=None, y=fake, ws=fake, wsb=1 << 24, **kw):
        a = {**args, **kw}
        return lib.dps_moe_linear(mode, enc, x, tor, eor, p, r, y, a["A"], a["T"], a["N"], a["K"], a["E"], ws, wsb, None)
    assert moe(mode=5) == binding.DPS_ERR_MODE
    assert moe(enc=bad) == binding.DPS_ERR_ENCODING
    assert moe(enc=None) == binding.DPS_ERR_NULL
    assert moe(K=20) == binding.DPS_ERR_SHAPE
    assert moe(E=0) == binding.DPS_ERR_SHAPE
    assert moe(A=0) == binding.DPS_OK
    assert moe(eor=None) == binding.DPS_ERR_NULL
    assert moe(mode=1) == binding.DPS_ERR_NULL
    assert moe(ws=None) == binding.DPS_ERR_WORKSPACE
    assert moe(wsb=8) == binding.DPS_ERR_WORKSPACE
    assert moe(ws=odd) == binding.DPS_ERR_WORKSPACE
    assert moe(x=odd) == binding.DPS_ERR_ALIGN
    # sizes the 32-bit row coordinates of the kernels cannot hold
    big = 1 << 31
    assert lib.dps_linear(0, 1, fake, fake, fake, fake, 1, big, 16, None) == binding.DPS_ERR_SHAPE
    assert lib.dps_linear(0, 1, fake, fake, fake, fake, 1, 8, big, None) == binding.DPS_ERR_SHAPE
    assert lib.dps_linear(0, 1, fake, fake, fake, fake, big, 8, 16, None) == binding.DPS_ERR_SHAPE
    assert lib.dps_linear_fp8act(1, fake, fake, fake, fake, 1, big, 16, None) == binding.DPS_ERR_SHAPE
    many = (ctypes.c_int32 * 1024)(*([1] * 1024))
    assert moe(enc=many, E=1024, N=1 << 21) == binding.DPS_ERR_SHAPE          # E * N = 2^31
    assert moe(enc=many, E=1024, N=(1 << 21) - 8, ws=None) == binding.DPS_ERR_WORKSPACE   # just below: accepted so far
    assert moe(N=big) == binding.DPS_ERR_SHAPE
    # the allocation-free variant validates the same way (and before it looks for a device)
    def moe_static(mode=0, enc=encs, x=fake, tor=None, eor=fake, p=fake, r=None, y=fake, **kw):
        a = {**args, **kw}
        return lib.dps_moe_linear_static(mode, enc, x, tor, eor, p, r, y, a["A"], a["T"], a["N"], a["K"], a["E"], None)
    assert moe_static(mode=5) == binding.DPS_ERR_MODE
    assert moe_static(enc=bad) == binding.DPS_ERR_ENCODING
    assert moe_static(enc=None) == binding.DPS_ERR_NULL
    assert moe_static(K=20) == binding.DPS_ERR_SHAPE
    assert moe_static(E=0) == binding.DPS_ERR_SHAPE
    assert moe_static(A=0) == binding.DPS_OK
    assert moe_static(eor=None) == binding.DPS_ERR_NULL
    assert moe_static(mode=1) == binding.DPS_ERR_NULL
    assert moe_static(x=odd) == binding.DPS_ERR_ALIGN
    assert moe_static(enc=many, E=1024, N=1 << 21) == binding.DPS_ERR_SHAPE
    assert moe_static(A=1 << 20, K=4096) == binding.DPS_ERR_WORKSPACE         # 8 GiB of regrouped activations
    # diagnostics
    assert lib.dps_debug_wait_timeout(0, None) == binding.DPS_ERR_SHAPE
    assert lib.dps_debug_wait_timeout(2_000_000_000, None) == binding.DPS_ERR_SHAPE


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", tmp_path / "libdps.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.library()
