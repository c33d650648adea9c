"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, sizes are right, and host-detectable errors come back before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_2504_12285_b200 import binding

HEADER = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "bitlinear.h")


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bitlinear_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.lib()
    names = declared_symbols()
    assert "bitlinear_pack_weights" in names and "bitlinear_quant_act" in names and "bitlinear_forward" in names
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in bitlinear.h but not exported"
        assert name in binding._SIGNATURES, f"{name} has no Python binding signature"
    for name in binding._SIGNATURES:
        assert name in names, f"{name} is bound but not declared in bitlinear.h"


def test_binding_has_a_function_per_compute_entry_point():
    for name in declared_symbols():
        if name in ("bitlinear_status_string", "bitlinear_version"):
            continue
        assert callable(getattr(binding, name)), name


def test_size_queries():
    assert binding.bitlinear_packed_bytes(2560, 2560) == 2560 * 2560 // 4  # four ternary values per byte
    assert binding.bitlinear_packed_bytes(6912, 2560) == 4423680
    assert binding.bitlinear_packed_bytes(2560, 2500) == 0  # K not a multiple of 256
    assert binding.bitlinear_packed_bytes(100, 2560) == 0  # N not a multiple of 16
    assert binding.bitlinear_packed_bytes(16, 32768) == 0  # K above the supported maximum
    assert binding.bitlinear_pack_workspace_bytes(2560, 2560) >= 8
    small = binding.bitlinear_workspace_bytes(1, 2560, 2560)
    assert small >= 2560 + 8
    assert binding.bitlinear_workspace_bytes(16, 2560, 2560) >= 16 * 2560
    # above 16 tokens the tensor-core path may run and needs the unpacked codes
    assert binding.bitlinear_workspace_bytes(64, 2560, 2560) >= 64 * 2560 + 2560 * 2560
    assert binding.bitlinear_matmul_workspace_bytes(1, 2560, 2560, binding.PATH_AUTO) == 0
    assert binding.bitlinear_matmul_workspace_bytes(1, 2560, 2560, binding.PATH_GEMM) >= 2560 * 2560
    assert binding.bitlinear_workspace_bytes(-1, 2560, 2560) == 0


def test_status_strings():
    assert binding.status_string(0) == "ok"
    seen = {binding.status_string(i) for i in range(9)}
    assert len(seen) == 9
    assert binding.status_string(99) == "unknown status"


def test_host_detectable_errors_need_no_gpu():
    lib = binding.lib()
    buf = (ctypes.c_char * 4096)()
    addr = (ctypes.addressof(buf) + 255) // 256 * 256  # an aligned, non-NULL stand-in; never dereferenced
    NULL = None
    # NULL pointers
    assert lib.bitlinear_pack_weights(NULL, 0, 16, 256, 1e-5, addr, addr, addr, 4096, NULL) == 1
    assert lib.bitlinear_quant_act(NULL, NULL, 1e-5, 1, 256, addr, addr, addr, NULL) == 1
    assert lib.bitlinear_forward(addr, NULL, 1e-5, NULL, addr, 1, 16, 256, addr, 0, addr, 4096, NULL) == 1
    assert lib.bitlinear_matmul_q(addr, addr, NULL, addr, addr, 1, 16, 256, addr, 0, NULL, 0, NULL, 0, NULL) == 1
    # shapes
    assert lib.bitlinear_pack_weights(addr, 0, 15, 256, 1e-5, addr, addr, addr, 4096, NULL) == 2
    assert lib.bitlinear_pack_weights(addr, 0, 16, 128, 1e-5, addr, addr, addr, 4096, NULL) == 2
    assert lib.bitlinear_quant_act(addr, NULL, 1e-5, 1, 100, addr, addr, addr, NULL) == 2
    assert lib.bitlinear_quant_act(addr, NULL, 1e-5, -1, 256, addr, addr, addr, NULL) == 2
    assert lib.bitlinear_forward(addr, NULL, 1e-5, addr, addr, 1, 16, 300, addr, 0, addr, 4096, NULL) == 2
    # dtype codes
    assert lib.bitlinear_pack_weights(addr, 7, 16, 256, 1e-5, addr, addr, addr, 4096, NULL) == 5
    assert lib.bitlinear_forward(addr, NULL, 1e-5, addr, addr, 1, 16, 256, addr, 3, addr, 4096, NULL) == 5
    # alignment
    assert lib.bitlinear_pack_weights(addr + 4, 0, 16, 256, 1e-5, addr, addr, addr, 4096, NULL) == 3
    assert lib.bitlinear_quant_act(addr, NULL, 1e-5, 1, 256, addr + 8, addr, addr, NULL) == 3
    # workspace
    assert lib.bitlinear_pack_weights(addr, 0, 16, 256, 1e-5, addr, addr, NULL, 0, NULL) == 4
    assert lib.bitlinear_forward(addr, NULL, 1e-5, addr, addr, 1, 16, 256, addr, 0, addr, 8, NULL) == 4
    assert lib.bitlinear_forward_host(addr, NULL, 1e-5, addr, addr, 1, 16, 256, addr, 0, addr, 8, NULL) == 4
    # tensor-core path needs N % 128 == 0
    assert lib.bitlinear_matmul_q(addr, addr, addr, addr, addr, 64, 16, 256, addr, 0, NULL, 2, addr, 1 << 20, NULL) == 2
    # M == 0 is a successful no-op, decided on the host
    assert lib.bitlinear_quant_act(addr, NULL, 1e-5, 0, 256, addr, addr, addr, NULL) == 0
    assert lib.bitlinear_forward(addr, NULL, 1e-5, addr, addr, 0, 16, 256, addr, 0, addr, 4096, NULL) == 0


def test_batch_entry_point_host_checks():
    lib = binding.lib()
    buf = (ctypes.c_char * 4096)()
    addr = (ctypes.addressof(buf) + 255) // 256 * 256
    arr = (binding.Problem * 2)()
    arr[0] = binding.Problem(addr, None, addr, addr, addr, 1, 16, 256, 0, 1e-5, 0)
    arr[1] = binding.Problem(addr, None, addr, addr, addr, 4, 32, 512, 1, 1e-5, 0)
    need = lib.bitlinear_batch_workspace_bytes(ctypes.addressof(arr), 2)
    assert need >= 256 + 4 * 512
    assert lib.bitlinear_forward_batch(ctypes.addressof(arr), 2, 0, None, 0, None) == 4       # no workspace
    assert lib.bitlinear_forward_batch(ctypes.addressof(arr), 2, 0, addr, need - 1, None) == 4
    assert lib.bitlinear_forward_batch(None, 2, 0, addr, need, None) == 1
    assert lib.bitlinear_forward_batch(ctypes.addressof(arr), 0, 0, None, 0, None) == 0       # empty batch
    assert lib.bitlinear_forward_batch(ctypes.addressof(arr), 2, 8, addr, need, None) == 5    # unknown flag
    arr[1].M = 16                      # several tokens: every problem of the call gets 16-row token images of 16 * K bytes
    assert lib.bitlinear_batch_workspace_bytes(ctypes.addressof(arr), 2) >= 16 * (256 + 512)
    arr[1].M = 17                      # 17 to 96 tokens are cut into 16-token problems: two 16-row images for this one
    assert lib.bitlinear_batch_workspace_bytes(ctypes.addressof(arr), 2) >= 16 * 256 + 32 * 512
    arr[1].w_format = 1                                                                         # dense layout: decode sizes only
    assert lib.bitlinear_forward_batch(ctypes.addressof(arr), 2, 0, addr, 1 << 20, None) == 2
    assert lib.bitlinear_batch_workspace_bytes(ctypes.addressof(arr), 2) == 0
    arr[1].w_format = 0
    arr[1].M = 4
    arr[1].packed = None
    assert lib.bitlinear_forward_batch(ctypes.addressof(arr), 2, 0, addr, 1 << 20, None) == 1
    arr[1].packed = addr + 4
    assert lib.bitlinear_forward_batch(ctypes.addressof(arr), 2, 0, addr, 1 << 20, None) == 3


def test_binding_raises_instead_of_falling_back():
    import torch

    x = torch.zeros(1, 256, dtype=torch.bfloat16)
    with pytest.raises(TypeError):
        binding.bitlinear_quant_act(x, None)  # CPU tensors are refused: there is no CPU path
