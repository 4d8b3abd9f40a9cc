"""Host-side checks of the C ABI: the library loads without a GPU, exports every function the
header declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2603_13420_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "pskv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pskv_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_paths_entry_points():
    names = declared_functions()
    for required in ("pskv_attn_fwd", "pskv_attn_bwd", "pskv_attn_fwd_workspace_bytes",
                     "pskv_attn_bwd_workspace_bytes", "pskv_poll_device_status"):
        assert required in names


def test_library_exports_every_declared_symbol():
    lib = binding.lib()
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_binding_has_the_same_names():
    for name in declared_functions():
        assert hasattr(binding, name), name


def test_version_and_status_strings():
    assert binding.pskv_version() >= 100
    assert binding.pskv_status_string(0) == "PSKV_OK"
    assert binding.pskv_status_string(6) == "PSKV_ERR_DEVICE_TIMEOUT"
    assert "UNKNOWN" in binding.pskv_status_string(99)


def _fwd(lib, ptrs, scale, dims, ws=None, ws_bytes=0):
    vp = ctypes.c_void_p
    return lib.pskv_attn_fwd(*[vp(p) for p in ptrs[:5]], scale, vp(ptrs[5]), vp(ptrs[6]), *dims,
                             vp(ws) if ws else None, ws_bytes, None)


GOOD = [0x1000, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000]  # never dereferenced on the host


@pytest.mark.parametrize("dims,code", [
    ((0, 4, 4, 8, 32, 64), binding.PSKV_ERR_INVALID_ARG),
    ((8, 4, 3, 8, 32, 64), binding.PSKV_ERR_INVALID_ARG),     # Hq % Hkv != 0
    ((8, 4, 4, 0, 32, 64), binding.PSKV_ERR_INVALID_ARG),
    ((8, 4, 4, 8, -1, 64), binding.PSKV_ERR_INVALID_ARG),
    ((8, 4, 4, 8, 32, 96), binding.PSKV_ERR_UNSUPPORTED_SHAPE),
    ((8, 4, 4, 8, 32, 256), binding.PSKV_ERR_UNSUPPORTED_SHAPE),
])
def test_bad_sizes_are_rejected_on_the_host(dims, code):
    assert _fwd(binding.lib(), GOOD, 0.125, dims) == code
    assert binding.pskv_kernel_family(0, *dims) == -code


def test_null_and_misaligned_pointers_are_rejected_on_the_host():
    lib = binding.lib()
    dims = (8, 4, 4, 8, 32, 64)
    for k in range(7):
        ptrs = list(GOOD)
        ptrs[k] = 0
        assert _fwd(lib, ptrs, 0.125, dims) == binding.PSKV_ERR_INVALID_ARG
        ptrs[k] = GOOD[k] + 8
        assert _fwd(lib, ptrs, 0.125, dims) == binding.PSKV_ERR_INVALID_ARG
    assert _fwd(lib, GOOD, float("nan"), dims) == binding.PSKV_ERR_INVALID_ARG
    assert _fwd(lib, GOOD, -1.0, dims) == binding.PSKV_ERR_INVALID_ARG


def test_backward_requires_workspace():
    lib = binding.lib()
    vp = ctypes.c_void_p
    dims = (8, 4, 4, 8, 32, 64)
    need = binding.pskv_attn_bwd_workspace_bytes(*dims)
    assert need >= 8 * 4 * 8 * 4
    ptrs = [vp(0x1000 * (k + 1)) for k in range(8)]
    outs = [vp(0x1000 * (k + 9)) for k in range(3)]
    rc = lib.pskv_attn_bwd(*ptrs, 0.125, *outs, *dims, None, 0, None)
    assert rc == binding.PSKV_ERR_WORKSPACE
    rc = lib.pskv_attn_bwd(*ptrs, 0.125, *outs, *dims, vp(0x100000), need - 1, None)
    assert rc == binding.PSKV_ERR_WORKSPACE


def test_workspace_queries_and_family_are_pure_host_logic():
    for dims in [(8, 4, 4, 8, 32, 64), (512, 32, 8, 48, 256, 128), (2, 7, 1, 3, 5, 64)]:
        assert binding.pskv_attn_fwd_workspace_bytes(*dims) % 256 == 0
        assert binding.pskv_attn_bwd_workspace_bytes(*dims) % 256 == 0
        assert binding.pskv_kernel_family(0, *dims) in (0, 1, 2)
        assert binding.pskv_kernel_family(1, *dims) in (0, 1)


def test_no_device_means_error_not_fallback():
    """Without a usable sm_100 device a well-formed call must fail loudly, never compute on the CPU."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    dims = (8, 4, 4, 8, 32, 64)
    need = binding.pskv_attn_fwd_workspace_bytes(*dims)
    assert _fwd(binding.lib(), GOOD, 0.125, dims) == (binding.PSKV_ERR_WORKSPACE if need else rc_no_device())
    rc = _fwd(binding.lib(), GOOD, 0.125, dims, ws=0x100000, ws_bytes=max(need, 256))
    assert rc in (binding.PSKV_ERR_CUDA, binding.PSKV_ERR_UNSUPPORTED_ARCH)


def rc_no_device():
    return binding.PSKV_ERR_CUDA


def test_kernel_timing_interface_without_a_device():
    assert binding.pskv_kernel_timing_count() >= 5
    names = [binding.pskv_kernel_timing_name(i) for i in range(binding.pskv_kernel_timing_count())]
    assert "tc_fwd_kernel" in names and "tc_bwd_dq_kernel" in names
    binding.pskv_kernel_timing_enable(True)
    assert binding.pskv_kernel_timing_read(0) == (0.0, 0)
    binding.pskv_kernel_timing_enable(False)
