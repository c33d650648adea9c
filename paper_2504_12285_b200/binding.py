"""Thin ctypes binding of libbitlinear.so: argument marshalling only.

Every function here has the name of the C entry point it calls (see
include/bitlinear.h) and does nothing but check tensor dtypes/devices, take
data pointers and the current CUDA stream, call into the library and raise on a
non-zero status.  PyTorch is used for device memory and streams only.  There is
no fallback: if the shared library is missing or a call fails, it raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

from . import build as _build

F32, BF16 = 0, 1
PATH_AUTO, PATH_GEMV, PATH_GEMM = 0, 1, 2

_lib = None
_c_void_p, _c_int, _c_size_t, _c_float = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t, ctypes.c_float

_SIGNATURES = {
    "bitlinear_status_string": (ctypes.c_char_p, [_c_int]),
    "bitlinear_version": (_c_int, []),
    "bitlinear_packed_bytes": (_c_size_t, [_c_int, _c_int]),
    "bitlinear_pack_workspace_bytes": (_c_size_t, [_c_int, _c_int]),
    "bitlinear_workspace_bytes": (_c_size_t, [_c_int, _c_int, _c_int]),
    "bitlinear_matmul_workspace_bytes": (_c_size_t, [_c_int, _c_int, _c_int, _c_int]),
    "bitlinear_host_staging_bytes": (_c_size_t, [_c_int, _c_int, _c_int, _c_int]),
    "bitlinear_pack_weights": (_c_int, [_c_void_p, _c_int, _c_int, _c_int, _c_float, _c_void_p, _c_void_p,
                                        _c_void_p, _c_size_t, _c_void_p]),
    "bitlinear_unpack_weights": (_c_int, [_c_void_p, _c_int, _c_int, _c_void_p, _c_void_p]),
    "bitlinear_packed5_bytes": (_c_size_t, [_c_int, _c_int]),
    "bitlinear_pack_weights5": (_c_int, [_c_void_p, _c_int, _c_int, _c_int, _c_float, _c_void_p, _c_void_p,
                                         _c_void_p, _c_size_t, _c_void_p]),
    "bitlinear_unpack_weights5": (_c_int, [_c_void_p, _c_int, _c_int, _c_void_p, _c_void_p]),
    "bitlinear_forward_batch_acc": (_c_int, [_c_void_p, _c_int, _c_int, _c_void_p, _c_void_p, _c_size_t, _c_void_p]),
    "bitlinear_quant_act": (_c_int, [_c_void_p, _c_void_p, _c_float, _c_int, _c_int, _c_void_p, _c_void_p,
                                     _c_void_p, _c_void_p]),
    "bitlinear_quant_act_relu2": (_c_int, [_c_void_p, _c_void_p, _c_void_p, _c_float, _c_int, _c_int, _c_void_p, _c_void_p,
                                           _c_void_p, _c_void_p, _c_void_p]),
    "bitlinear_matmul_q": (_c_int, [_c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int,
                                    _c_void_p, _c_int, _c_void_p, _c_int, _c_void_p, _c_size_t, _c_void_p]),
    "bitlinear_forward": (_c_int, [_c_void_p, _c_void_p, _c_float, _c_void_p, _c_void_p, _c_int, _c_int, _c_int,
                                   _c_void_p, _c_int, _c_void_p, _c_size_t, _c_void_p]),
    "bitlinear_forward_host": (_c_int, [_c_void_p, _c_void_p, _c_float, _c_void_p, _c_void_p, _c_int, _c_int,
                                        _c_int, _c_void_p, _c_int, _c_void_p, _c_size_t, _c_void_p]),
    "bitlinear_forward_master_workspace_bytes": (_c_size_t, [_c_int, _c_int, _c_int]),
    "bitlinear_forward_master": (_c_int, [_c_void_p, _c_void_p, _c_float, _c_void_p, _c_int, _c_float, _c_int, _c_int, _c_int,
                                          _c_void_p, _c_int, _c_void_p, _c_void_p, _c_void_p, _c_size_t, _c_void_p]),
    "bitlinear_rope_kv": (_c_int, [_c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_int, _c_float,
                                   _c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_void_p]),
    "bitlinear_attention_workspace_bytes": (_c_size_t, [_c_int, _c_int, _c_int, _c_int, _c_int]),
    "bitlinear_attention_decode": (_c_int, [_c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_int,
                                            _c_int, _c_int, _c_void_p, _c_void_p, _c_size_t, _c_void_p]),
    "bitlinear_rope_table": (_c_int, [_c_float, _c_int, _c_int, _c_void_p, _c_void_p]),
    "bitlinear_attention_decode_append": (_c_int, [_c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p,
                                                   _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_void_p, _c_void_p, _c_size_t,
                                                   _c_void_p]),
    "bitlinear_lm_head": (_c_int, [_c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_void_p, _c_void_p]),
    "bitlinear_embed": (_c_int, [_c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_void_p, _c_void_p]),
    "bitlinear_poll_status": (_c_int, [_c_void_p]),
    "bitlinear_probe_int8_mma_rate": (_c_int, [_c_int, ctypes.POINTER(ctypes.c_double), _c_void_p]),
    "bitlinear_selftest_wait_timeout": (_c_int, [ctypes.c_uint, _c_void_p]),
    "bitlinear_glue_relu2_mul": (_c_int, [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_void_p]),
    "bitlinear_glue_residual_add": (_c_int, [_c_void_p, _c_void_p, _c_int, _c_int, _c_void_p]),
    "bitlinear_glue_attn_standin": (_c_int, [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_int, _c_void_p]),
    "bitlinear_decode_chain_workspace_bytes": (_c_size_t, [_c_int, _c_int, _c_int, _c_int, _c_int, _c_int]),
    "bitlinear_decode_chain": (_c_int, [_c_void_p, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_float, _c_void_p,
                                        _c_void_p, _c_int, _c_void_p, _c_size_t, _c_void_p]),
    "bitlinear_static_scratch_bytes": (_c_size_t, []),
    "bitlinear_forward_static": (_c_int, [_c_void_p, _c_void_p, _c_float, _c_void_p, _c_void_p, _c_int, _c_int, _c_int,
                                          _c_void_p, _c_int, _c_void_p]),
    "bitlinear_batch_workspace_bytes": (_c_size_t, [_c_void_p, _c_int]),
    "bitlinear_forward_batch": (_c_int, [_c_void_p, _c_int, _c_int, _c_void_p, _c_size_t, _c_void_p]),
    "bitlinear_forward_batch_host": (_c_int, [_c_void_p, _c_int, _c_int, _c_void_p, _c_void_p, _c_size_t, _c_void_p,
                                              _c_void_p, _c_size_t, _c_void_p, _c_size_t, _c_void_p]),
}

WEIGHTS_2BIT, WEIGHTS_DENSE5 = 0, 1
X_PLAIN, X_RELU2, X_RESIDUAL, X_ATTN_STANDIN = 0, 1, 2, 3
BATCH_REUSE_PLAN = 1
BATCH_REUSE_ACT = 2
BATCH_REUSE_WEIGHTS = 4


class Problem(ctypes.Structure):
    """Mirror of the C struct bitlinear_problem."""
    _fields_ = [("x", _c_void_p), ("gain", _c_void_p), ("packed", _c_void_p), ("s_w", _c_void_p), ("y", _c_void_p),
                ("M", _c_int), ("N", _c_int), ("K", _c_int), ("y_dtype", _c_int), ("rms_eps", _c_float),
                ("w_format", _c_int), ("x_op", _c_int), ("x_arg0", _c_int), ("x_arg1", _c_int), ("reserved", _c_int),
                ("x2", _c_void_p), ("x_out", _c_void_p)]


class BitLinearError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where} failed: status {status} ({status_string(status)})")


def library_path() -> Path:
    return _build.LIB


def lib() -> ctypes.CDLL:
    """Load libbitlinear.so (building it with nvcc if absent); raises if that is impossible."""
    global _lib
    if _lib is None:
        path = _build.build()
        loaded = ctypes.CDLL(str(path))
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(loaded, name)  # AttributeError if an entry point is missing
            fn.restype = res
            fn.argtypes = args
        _lib = loaded
    return _lib


def status_string(status: int) -> str:
    return lib().bitlinear_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise BitLinearError(status, where)


def _ptr(t: torch.Tensor | None) -> int | None:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous CUDA tensor of {dtype}")
    return t


def _ydt(dtype) -> int:
    if dtype == torch.float32:
        return F32
    if dtype == torch.bfloat16:
        return BF16
    raise TypeError("output dtype must be float32 or bfloat16")


def bitlinear_packed_bytes(N: int, K: int) -> int:
    return int(lib().bitlinear_packed_bytes(N, K))


def bitlinear_pack_workspace_bytes(N: int, K: int) -> int:
    return int(lib().bitlinear_pack_workspace_bytes(N, K))


def bitlinear_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(lib().bitlinear_workspace_bytes(M, N, K))


def bitlinear_matmul_workspace_bytes(M: int, N: int, K: int, path: int = PATH_AUTO) -> int:
    return int(lib().bitlinear_matmul_workspace_bytes(M, N, K, path))


def bitlinear_host_staging_bytes(M: int, N: int, K: int, y_dtype=torch.float32) -> int:
    return int(lib().bitlinear_host_staging_bytes(M, N, K, _ydt(y_dtype)))


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device=device)


def bitlinear_pack_weights(W: torch.Tensor, eps_w: float = 1e-5):
    """W [N, K] fp32 or bf16 on the GPU -> (packed uint8 [N*K/4], s_w fp32 [1]), both on the GPU."""
    if W.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("W must be float32 or bfloat16")
    _dev(W, W.dtype, "W")
    N, K = W.shape
    nbytes = bitlinear_packed_bytes(N, K)
    if nbytes == 0:
        raise BitLinearError(2, "bitlinear_pack_weights")
    packed = torch.empty(nbytes, dtype=torch.uint8, device=W.device)
    s_w = torch.empty(1, dtype=torch.float32, device=W.device)
    ws = _workspace(bitlinear_pack_workspace_bytes(N, K), W.device)
    rc = lib().bitlinear_pack_weights(_ptr(W), F32 if W.dtype == torch.float32 else BF16, N, K, eps_w, _ptr(packed),
                                      _ptr(s_w), _ptr(ws), ws.numel(), _stream())
    _check(rc, "bitlinear_pack_weights")
    return packed, s_w


def bitlinear_packed5_bytes(N: int, K: int) -> int:
    return int(lib().bitlinear_packed5_bytes(N, K))


def bitlinear_pack_weights5(W: torch.Tensor, eps_w: float = 1e-5):
    """W [N, K] fp32 or bf16 on the GPU -> (dense packed uint8, five values per byte, s_w fp32 [1])."""
    if W.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("W must be float32 or bfloat16")
    _dev(W, W.dtype, "W")
    N, K = W.shape
    nbytes = bitlinear_packed5_bytes(N, K)
    if nbytes == 0:
        raise BitLinearError(2, "bitlinear_pack_weights5")
    packed = torch.empty(nbytes, dtype=torch.uint8, device=W.device)
    s_w = torch.empty(1, dtype=torch.float32, device=W.device)
    ws = _workspace(bitlinear_pack_workspace_bytes(N, K), W.device)
    rc = lib().bitlinear_pack_weights5(_ptr(W), F32 if W.dtype == torch.float32 else BF16, N, K, eps_w, _ptr(packed),
                                       _ptr(s_w), _ptr(ws), ws.numel(), _stream())
    _check(rc, "bitlinear_pack_weights5")
    return packed, s_w


def bitlinear_unpack_weights5(packed: torch.Tensor, N: int, K: int) -> torch.Tensor:
    _dev(packed, torch.uint8, "packed")
    wq = torch.empty(N, K, dtype=torch.int8, device=packed.device)
    _check(lib().bitlinear_unpack_weights5(_ptr(packed), N, K, _ptr(wq), _stream()), "bitlinear_unpack_weights5")
    return wq


def bitlinear_unpack_weights(packed: torch.Tensor, N: int, K: int) -> torch.Tensor:
    _dev(packed, torch.uint8, "packed")
    wq = torch.empty(N, K, dtype=torch.int8, device=packed.device)
    _check(lib().bitlinear_unpack_weights(_ptr(packed), N, K, _ptr(wq), _stream()), "bitlinear_unpack_weights")
    return wq


def bitlinear_quant_act(x: torch.Tensor, gain: torch.Tensor | None, rms_eps: float = 1e-5):
    """x [M, K] bf16 -> (xq int8 [M, K], d fp32 [M], xsum int32 [M])."""
    _dev(x, torch.bfloat16, "x")
    if gain is not None:
        _dev(gain, torch.bfloat16, "gain")
    M, K = x.shape
    xq = torch.empty(M, K, dtype=torch.int8, device=x.device)
    d = torch.empty(max(M, 1), dtype=torch.float32, device=x.device)[:M]
    xsum = torch.empty(max(M, 1), dtype=torch.int32, device=x.device)[:M]
    rc = lib().bitlinear_quant_act(_ptr(x), _ptr(gain), rms_eps, M, K, _ptr(xq), _ptr(d), _ptr(xsum), _stream())
    _check(rc, "bitlinear_quant_act")
    return xq, d, xsum


def bitlinear_quant_act_relu2(gate: torch.Tensor, up: torch.Tensor, gain: torch.Tensor | None, rms_eps: float = 1e-5,
                              want_x: bool = False):
    """gate, up [M, F] fp32 -> (xq int8 [M, F], d fp32 [M], xsum int32 [M][, f bf16 [M, F]]): squared-ReLU gate fused
    with the down projection's RMSNorm + int8 quantiser."""
    _dev(gate, torch.float32, "gate"), _dev(up, torch.float32, "up")
    if gain is not None:
        _dev(gain, torch.bfloat16, "gain")
    M, F = gate.shape
    xq = torch.empty(M, F, dtype=torch.int8, device=gate.device)
    d = torch.empty(max(M, 1), dtype=torch.float32, device=gate.device)[:M]
    xsum = torch.empty(max(M, 1), dtype=torch.int32, device=gate.device)[:M]
    f = torch.empty(M, F, dtype=torch.bfloat16, device=gate.device) if want_x else None
    rc = lib().bitlinear_quant_act_relu2(_ptr(gate), _ptr(up), _ptr(gain), rms_eps, M, F, _ptr(f), _ptr(xq), _ptr(d),
                                         _ptr(xsum), _stream())
    _check(rc, "bitlinear_quant_act_relu2")
    return (xq, d, xsum, f) if want_x else (xq, d, xsum)


def bitlinear_matmul_q(xq, d, xsum, packed, s_w, N: int, y_dtype=torch.float32, want_acc: bool = False,
                       path: int = PATH_AUTO, ws: torch.Tensor | None = None):
    """Contraction + epilogue on quantised activations -> y [M, N] (and the int32 accumulators)."""
    _dev(xq, torch.int8, "xq")
    _dev(d, torch.float32, "d")
    _dev(xsum, torch.int32, "xsum")
    _dev(packed, torch.uint8, "packed")
    _dev(s_w, torch.float32, "s_w")
    M, K = xq.shape
    y = torch.empty(M, N, dtype=y_dtype, device=xq.device)
    acc = torch.empty(M, N, dtype=torch.int32, device=xq.device) if want_acc else None
    if ws is None:
        ws = _workspace(bitlinear_matmul_workspace_bytes(M, N, K, path), xq.device)
    rc = lib().bitlinear_matmul_q(_ptr(xq), _ptr(d), _ptr(xsum), _ptr(packed), _ptr(s_w), M, N, K, _ptr(y),
                                  _ydt(y_dtype), _ptr(acc), path, _ptr(ws), ws.numel(), _stream())
    _check(rc, "bitlinear_matmul_q")
    return (y, acc) if want_acc else y


def bitlinear_forward(x, gain, packed, s_w, N: int, rms_eps: float = 1e-5, y_dtype=torch.float32,
                      ws: torch.Tensor | None = None, out: torch.Tensor | None = None) -> torch.Tensor:
    """The whole BitLinear forward on device tensors -> y [M, N]."""
    _dev(x, torch.bfloat16, "x")
    if gain is not None:
        _dev(gain, torch.bfloat16, "gain")
    _dev(packed, torch.uint8, "packed")
    _dev(s_w, torch.float32, "s_w")
    M, K = x.shape
    y = out if out is not None else torch.empty(M, N, dtype=y_dtype, device=x.device)
    if ws is None:
        ws = _workspace(bitlinear_workspace_bytes(M, N, K), x.device)
    rc = lib().bitlinear_forward(_ptr(x), _ptr(gain), rms_eps, _ptr(packed), _ptr(s_w), M, N, K, _ptr(y),
                                 _ydt(y.dtype), _ptr(ws), ws.numel(), _stream())
    _check(rc, "bitlinear_forward")
    return y


def bitlinear_forward_host(x_host, gain, packed, s_w, N: int, y_host, rms_eps: float = 1e-5,
                           ws: torch.Tensor | None = None) -> torch.Tensor:
    """Forward with HOST activations in and HOST result out (copies inside; synchronises)."""
    if x_host.is_cuda or y_host.is_cuda or x_host.dtype != torch.bfloat16:
        raise TypeError("x_host / y_host must be CPU tensors (x bf16)")
    M, K = x_host.shape
    if ws is None:
        ws = _workspace(bitlinear_workspace_bytes(M, N, K) + bitlinear_host_staging_bytes(M, N, K, y_host.dtype),
                        packed.device)
    rc = lib().bitlinear_forward_host(_ptr(x_host), _ptr(gain), rms_eps, _ptr(packed), _ptr(s_w), M, N, K,
                                      _ptr(y_host), _ydt(y_host.dtype), _ptr(ws), ws.numel(), _stream())
    _check(rc, "bitlinear_forward_host")
    return y_host


def bitlinear_glue_relu2_mul(gate: torch.Tensor, up: torch.Tensor, u: torch.Tensor) -> torch.Tensor:
    """u (bf16) = relu(gate)^2 * up, gate / up fp32 [M, F]."""
    _dev(gate, torch.float32, "gate"), _dev(up, torch.float32, "up"), _dev(u, torch.bfloat16, "u")
    M, F = gate.shape
    _check(lib().bitlinear_glue_relu2_mul(_ptr(gate), _ptr(up), _ptr(u), M, F, _stream()), "bitlinear_glue_relu2_mul")
    return u


def bitlinear_glue_residual_add(h: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
    """h (bf16, in place) = h + y, y fp32 [M, N]."""
    _dev(h, torch.bfloat16, "h"), _dev(y, torch.float32, "y")
    M, N = h.shape
    _check(lib().bitlinear_glue_residual_add(_ptr(h), _ptr(y), M, N, _stream()), "bitlinear_glue_residual_add")
    return h


def bitlinear_glue_attn_standin(q: torch.Tensor, v: torch.Tensor, o_in: torch.Tensor, n_q_heads: int, n_kv_heads: int,
                                head_dim: int) -> torch.Tensor:
    """o_in (bf16) = q + v of the matching KV head: a stand-in for attention that keeps a layer's data dependence."""
    _dev(q, torch.float32, "q"), _dev(v, torch.float32, "v"), _dev(o_in, torch.bfloat16, "o_in")
    rc = lib().bitlinear_glue_attn_standin(_ptr(q), _ptr(v), _ptr(o_in), q.shape[0], n_q_heads, n_kv_heads, head_dim,
                                           _stream())
    _check(rc, "bitlinear_glue_attn_standin")
    return o_in


class ChainLayer(ctypes.Structure):
    """Mirror of the C struct bitlinear_chain_layer."""
    _fields_ = [("packed", _c_void_p * 7), ("s_w", _c_void_p * 7), ("gain", _c_void_p * 4)]


CHAIN_MATRICES = ("q", "k", "v", "o", "gate", "up", "down")


class ChainLayers:
    """Host array of bitlinear_chain_layer plus the tensors it points to (kept alive).

    layers: list of dicts with keys q,k,v,o,gate,up,down -> (packed uint8, s_w fp32 [1]) and "gains" -> four bf16 [K]
    tensors or None (inputs of {q,k,v}, o, {gate,up}, down)."""

    def __init__(self, layers):
        self.keep = layers
        self.count = len(layers)
        self.array = (ChainLayer * max(self.count, 1))()
        for i, layer in enumerate(layers):
            for j, name in enumerate(CHAIN_MATRICES):
                packed, s_w = layer[name]
                _dev(packed, torch.uint8, name), _dev(s_w, torch.float32, name + ".s_w")
                self.array[i].packed[j] = packed.data_ptr()
                self.array[i].s_w[j] = s_w.data_ptr()
            for j, gain in enumerate(layer["gains"]):
                if gain is not None:
                    _dev(gain, torch.bfloat16, "gain")
                self.array[i].gain[j] = None if gain is None else gain.data_ptr()


def bitlinear_decode_chain_workspace_bytes(n_layers: int, hidden: int, ffn: int, n_q_heads: int, n_kv_heads: int,
                                           head_dim: int) -> int:
    return int(lib().bitlinear_decode_chain_workspace_bytes(n_layers, hidden, ffn, n_q_heads, n_kv_heads, head_dim))


def bitlinear_decode_chain(layers: ChainLayers, hidden: int, ffn: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                           h: torch.Tensor, ws: torch.Tensor, rms_eps: float = 1e-5, k_out: torch.Tensor | None = None,
                           reuse_plan: bool = False) -> torch.Tensor:
    """One token through the whole stack in one persistent kernel; h (bf16 [1, hidden] or [hidden]) is updated in place."""
    _dev(h, torch.bfloat16, "h"), _dev(ws, torch.uint8, "ws")
    if k_out is not None:
        _dev(k_out, torch.float32, "k_out")
    rc = lib().bitlinear_decode_chain(ctypes.addressof(layers.array), layers.count, hidden, ffn, n_q_heads, n_kv_heads,
                                      head_dim, rms_eps, _ptr(h), _ptr(k_out), BATCH_REUSE_PLAN if reuse_plan else 0,
                                      _ptr(ws), ws.numel(), _stream())
    _check(rc, "bitlinear_decode_chain")
    return h


def bitlinear_static_scratch_bytes() -> int:
    return int(lib().bitlinear_static_scratch_bytes())


def bitlinear_forward_master_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(lib().bitlinear_forward_master_workspace_bytes(M, N, K))


def bitlinear_forward_master(x, gain, W, N: int | None = None, rms_eps: float = 1e-5, eps_w: float = 1e-5, y_dtype=torch.float32,
                             want_packed: bool = False):
    """The training-time forward: master weights W [N, K] (fp32 or bf16) are quantised on the fly.  Returns y, or
    (y, packed, s_w) with want_packed."""
    _dev(x, torch.bfloat16, "x")
    if gain is not None:
        _dev(gain, torch.bfloat16, "gain")
    if W.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("W must be float32 or bfloat16")
    _dev(W, W.dtype, "W")
    M, K = x.shape
    if W.shape[1] != K or (N is not None and W.shape[0] != N):
        raise ValueError("W must be [N, K]")
    N = W.shape[0]
    y = torch.empty(M, N, dtype=y_dtype, device=x.device)
    ws = _workspace(bitlinear_forward_master_workspace_bytes(M, N, K), x.device)
    packed = torch.empty(bitlinear_packed_bytes(N, K), dtype=torch.uint8, device=x.device) if want_packed else None
    s_w = torch.empty(1, dtype=torch.float32, device=x.device) if want_packed else None
    rc = lib().bitlinear_forward_master(_ptr(x), _ptr(gain), rms_eps, _ptr(W), BF16 if W.dtype == torch.bfloat16 else F32, eps_w,
                                        M, N, K, _ptr(y), _ydt(y_dtype), _ptr(packed), _ptr(s_w), _ptr(ws), ws.numel(), _stream())
    _check(rc, "bitlinear_forward_master")
    return (y, packed, s_w) if want_packed else y


def bitlinear_forward_static(x, gain, packed, s_w, N: int, rms_eps: float = 1e-5, y_dtype=torch.float32,
                             out: torch.Tensor | None = None) -> torch.Tensor:
    """Decode-sized forward (M <= 16) that takes no workspace: for callers that cannot allocate device
    memory, the scratch is a fixed array inside the library.  Calls on one device must not overlap."""
    _dev(x, torch.bfloat16, "x")
    if gain is not None:
        _dev(gain, torch.bfloat16, "gain")
    _dev(packed, torch.uint8, "packed")
    _dev(s_w, torch.float32, "s_w")
    M, K = x.shape
    if out is not None:
        if not out.is_cuda or not out.is_contiguous() or out.dtype not in (torch.float32, torch.bfloat16):
            raise TypeError("out must be a contiguous CUDA tensor of float32 or bfloat16")
        if tuple(out.shape) != (M, N):
            raise ValueError(f"out must have shape ({M}, {N})")
    y = out if out is not None else torch.empty(M, N, dtype=y_dtype, device=x.device)
    rc = lib().bitlinear_forward_static(_ptr(x), _ptr(gain), rms_eps, _ptr(packed), _ptr(s_w), M, N, K, _ptr(y),
                                        _ydt(y.dtype), _stream())
    _check(rc, "bitlinear_forward_static")
    return y


class ProblemBatch:
    """A host array of bitlinear_problem descriptors plus the tensors they point to (kept alive)."""

    def __init__(self, items, rms_eps: float = 1e-5, w_format: int = WEIGHTS_2BIT):
        """items: iterable of (x [M,K] bf16, gain [K] bf16 or None, packed uint8, s_w fp32 [1], y [M,N]) with an
        optional sixth entry (x_op, x2, x_out, x_arg0, x_arg1): the element-wise step fused into the quantiser (X_RELU2:
        x = gate fp32, x2 = up fp32; X_RESIDUAL: x = h bf16, x2 = y fp32; X_ATTN_STANDIN: x = q fp32, x2 = v fp32,
        x_arg0 = head_dim, x_arg1 = query heads per KV head; x_out = bf16 [M,K] or None);
        w_format: the layout of every packed matrix of the batch (WEIGHTS_2BIT or WEIGHTS_DENSE5)."""
        self.tensors = [tuple(it[:5]) for it in items]
        self.steps = [it[5] if len(it) > 5 else None for it in items]  # kept alive with the batch
        self.array = (Problem * max(len(self.tensors), 1))()
        for i, (x, gain, packed, s_w, y) in enumerate(self.tensors):
            step = self.steps[i]
            _dev(x, torch.bfloat16 if step is None or step[0] == X_RESIDUAL else torch.float32, "x")
            if gain is not None:
                _dev(gain, torch.bfloat16, "gain")
            _dev(packed, torch.uint8, "packed")
            _dev(s_w, torch.float32, "s_w")
            if not y.is_cuda or not y.is_contiguous():
                raise TypeError("y must be a contiguous CUDA tensor")
            M, K = x.shape
            if y.shape[0] != M:
                raise ValueError("x and y disagree on M")
            op, x2, x_out, arg0, arg1 = (X_PLAIN, None, None, 0, 0) if step is None else step
            if x2 is not None:
                _dev(x2, torch.float32, "x2")
            if x_out is not None:
                _dev(x_out, torch.bfloat16, "x_out")
            self.array[i] = Problem(_ptr(x), _ptr(gain), _ptr(packed), _ptr(s_w), _ptr(y), M, y.shape[1], K,
                                    _ydt(y.dtype), rms_eps, w_format, op, arg0, arg1, 0, _ptr(x2), _ptr(x_out))
        self.count = len(self.tensors)

    def workspace_bytes(self) -> int:
        return int(lib().bitlinear_batch_workspace_bytes(ctypes.addressof(self.array), self.count))


def bitlinear_batch_workspace_bytes(batch: ProblemBatch) -> int:
    return batch.workspace_bytes()


def bitlinear_forward_batch(batch: ProblemBatch, ws: torch.Tensor, reuse_plan: bool = False,
                            reuse_act: bool = False, reuse_weights: bool = False) -> None:
    """Run every forward of the batch (decode sizes, M <= 16) in two launches; results land in the y tensors."""
    _dev(ws, torch.uint8, "ws")
    flags = ((BATCH_REUSE_PLAN if reuse_plan else 0) | (BATCH_REUSE_ACT if reuse_act else 0) |
             (BATCH_REUSE_WEIGHTS if reuse_weights else 0))
    rc = lib().bitlinear_forward_batch(ctypes.addressof(batch.array), batch.count, flags, _ptr(ws), ws.numel(),
                                       _stream())
    _check(rc, "bitlinear_forward_batch")


def bitlinear_forward_batch_acc(batch: ProblemBatch, accs, ws: torch.Tensor, reuse_plan: bool = False) -> None:
    """bitlinear_forward_batch that also stores the int32 accumulators: accs[i] is None or an int32 [M, N] CUDA tensor."""
    _dev(ws, torch.uint8, "ws")
    arr = (_c_void_p * max(batch.count, 1))()
    for i, a in enumerate(accs):
        if a is not None:
            _dev(a, torch.int32, "acc")
            arr[i] = a.data_ptr()
    rc = lib().bitlinear_forward_batch_acc(ctypes.addressof(batch.array), batch.count, BATCH_REUSE_PLAN if reuse_plan else 0,
                                           ctypes.addressof(arr), _ptr(ws), ws.numel(), _stream())
    _check(rc, "bitlinear_forward_batch_acc")


def bitlinear_forward_batch_host(batch: ProblemBatch, x_host: torch.Tensor, x_dev: torch.Tensor, y_dev: torch.Tensor,
                                 y_host: torch.Tensor, ws: torch.Tensor, reuse_plan: bool = False) -> None:
    """Batch forward with HOST activations in and HOST results out: x_host -> x_dev arena, run, y_dev arena -> y_host."""
    if x_host.is_cuda or y_host.is_cuda or not x_dev.is_cuda or not y_dev.is_cuda:
        raise TypeError("x_host / y_host must be CPU tensors and x_dev / y_dev CUDA tensors")
    xb, yb = x_host.numel() * x_host.element_size(), y_host.numel() * y_host.element_size()
    if xb > x_dev.numel() * x_dev.element_size() or yb > y_dev.numel() * y_dev.element_size():
        raise ValueError("device arenas are smaller than the host buffers")
    rc = lib().bitlinear_forward_batch_host(ctypes.addressof(batch.array), batch.count,
                                            BATCH_REUSE_PLAN if reuse_plan else 0, _ptr(x_host), _ptr(x_dev), xb,
                                            _ptr(y_dev), _ptr(y_host), yb, _ptr(ws), ws.numel(), _stream())
    _check(rc, "bitlinear_forward_batch_host")


def _cache_dims(k_cache, v_cache, n_kv_heads: int, head_dim: int):
    """(n_seq, t_max) of a key/value cache pair [n_seq, n_kv, t_max, D] or [n_kv, t_max, D]."""
    if k_cache.shape != v_cache.shape or k_cache.dim() not in (3, 4) or tuple(k_cache.shape[-3::2]) != (n_kv_heads, head_dim):
        raise ValueError(f"caches must both be [n_seq, {n_kv_heads}, t_max, {head_dim}] or [{n_kv_heads}, t_max, {head_dim}]")
    return (k_cache.shape[0] if k_cache.dim() == 4 else 1), k_cache.shape[-2]


def bitlinear_rope_kv(q, k, v, positions, k_cache, v_cache, n_q_heads: int, n_kv_heads: int, head_dim: int,
                      rope_base: float = 500000.0, seq_ids=None, q_out=None):
    """Rotate q, k (fp32 [M, heads * D]) at `positions` (int32 [M]); q -> bf16 (returned), k / v appended to the bf16
    caches [n_seq, n_kv, t_max, D] (contiguous) at those positions."""
    _dev(q, torch.float32, "q"), _dev(k, torch.float32, "k"), _dev(v, torch.float32, "v")
    _dev(positions, torch.int32, "positions"), _dev(k_cache, torch.bfloat16, "k_cache"), _dev(v_cache, torch.bfloat16, "v_cache")
    if seq_ids is not None:
        _dev(seq_ids, torch.int32, "seq_ids")
    M = q.shape[0]
    n_seq, t_max = _cache_dims(k_cache, v_cache, n_kv_heads, head_dim)
    if q_out is None:
        q_out = torch.empty(M, n_q_heads * head_dim, dtype=torch.bfloat16, device=q.device)
    rc = lib().bitlinear_rope_kv(_ptr(q), _ptr(k), _ptr(v), _ptr(positions), _ptr(seq_ids), M, n_q_heads, n_kv_heads, head_dim,
                                 rope_base, _ptr(q_out), _ptr(k_cache), _ptr(v_cache), n_seq, t_max, _stream())
    _check(rc, "bitlinear_rope_kv")
    return q_out


def bitlinear_attention_workspace_bytes(M: int, n_q_heads: int, n_kv_heads: int, head_dim: int, t_max: int) -> int:
    return int(lib().bitlinear_attention_workspace_bytes(M, n_q_heads, n_kv_heads, head_dim, t_max))


def bitlinear_attention_decode(q, k_cache, v_cache, lengths, n_q_heads: int, n_kv_heads: int, head_dim: int, seq_ids=None,
                               out=None, ws=None):
    """q bf16 [M, n_q * D] against the first lengths[m] rows of its sequence's bf16 cache -> bf16 [M, n_q * D]."""
    _dev(q, torch.bfloat16, "q"), _dev(k_cache, torch.bfloat16, "k_cache"), _dev(v_cache, torch.bfloat16, "v_cache")
    _dev(lengths, torch.int32, "lengths")
    if seq_ids is not None:
        _dev(seq_ids, torch.int32, "seq_ids")
    M = q.shape[0]
    n_seq, t_max = _cache_dims(k_cache, v_cache, n_kv_heads, head_dim)
    if out is None:
        out = torch.empty(M, n_q_heads * head_dim, dtype=torch.bfloat16, device=q.device)
    if ws is None:
        ws = _workspace(bitlinear_attention_workspace_bytes(M, n_q_heads, n_kv_heads, head_dim, t_max), q.device)
    rc = lib().bitlinear_attention_decode(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(lengths), _ptr(seq_ids), M, n_q_heads,
                                          n_kv_heads, head_dim, n_seq, t_max, _ptr(out), _ptr(ws), ws.numel(), _stream())
    _check(rc, "bitlinear_attention_decode")
    return out


def bitlinear_rope_table(head_dim: int, t_max: int, rope_base: float = 500000.0, device="cuda:0"):
    """(cos, sin) of every (position, pair) -> fp32 [t_max, D / 2, 2], for bitlinear_attention_decode_append."""
    table = torch.empty(t_max, head_dim // 2, 2, dtype=torch.float32, device=device)
    with torch.cuda.device(table.device):
        _check(lib().bitlinear_rope_table(rope_base, head_dim, t_max, _ptr(table), _stream()), "bitlinear_rope_table")
    return table


def bitlinear_attention_decode_append(q, k, v, rope_table, k_cache, v_cache, lengths, n_q_heads: int, n_kv_heads: int, head_dim: int,
                                      seq_ids=None, out=None, ws=None):
    """Rotary embedding, cache append at row lengths[m] - 1 and attention over rows 0 .. lengths[m] - 1 in the attention
    launches: q, k, v fp32 projections of one token per (distinct) sequence -> bf16 [M, n_q * D]."""
    _dev(q, torch.float32, "q"), _dev(k, torch.float32, "k"), _dev(v, torch.float32, "v"), _dev(rope_table, torch.float32, "rope_table")
    _dev(k_cache, torch.bfloat16, "k_cache"), _dev(v_cache, torch.bfloat16, "v_cache"), _dev(lengths, torch.int32, "lengths")
    if seq_ids is not None:
        _dev(seq_ids, torch.int32, "seq_ids")
    M = q.shape[0]
    n_seq, t_max = _cache_dims(k_cache, v_cache, n_kv_heads, head_dim)
    if rope_table.dim() != 3 or rope_table.shape[0] < t_max or tuple(rope_table.shape[1:]) != (head_dim // 2, 2):
        raise ValueError(f"rope_table must be [>= {t_max}, {head_dim // 2}, 2]")
    if out is None:
        out = torch.empty(M, n_q_heads * head_dim, dtype=torch.bfloat16, device=q.device)
    if ws is None:
        ws = _workspace(bitlinear_attention_workspace_bytes(M, n_q_heads, n_kv_heads, head_dim, t_max), q.device)
    rc = lib().bitlinear_attention_decode_append(_ptr(q), _ptr(k), _ptr(v), _ptr(rope_table), _ptr(k_cache), _ptr(v_cache),
                                                 _ptr(lengths), _ptr(seq_ids), M, n_q_heads, n_kv_heads, head_dim, n_seq, t_max,
                                                 _ptr(out), _ptr(ws), ws.numel(), _stream())
    _check(rc, "bitlinear_attention_decode_append")
    return out


def bitlinear_lm_head(x, table, out=None):
    """x bf16 [M, K] (M <= 16), table bf16 [V, K] -> logits fp32 [M, V]."""
    _dev(x, torch.bfloat16, "x"), _dev(table, torch.bfloat16, "table")
    M, K = x.shape
    V = table.shape[0]
    if out is None:
        out = torch.empty(M, V, dtype=torch.float32, device=x.device)
    _check(lib().bitlinear_lm_head(_ptr(x), _ptr(table), M, V, K, _ptr(out), _stream()), "bitlinear_lm_head")
    return out


def bitlinear_embed(ids, table, out=None):
    """ids int32 [M], table bf16 [V, K] -> bf16 [M, K]."""
    _dev(ids, torch.int32, "ids"), _dev(table, torch.bfloat16, "table")
    M, (V, K) = ids.shape[0], table.shape
    if out is None:
        out = torch.empty(M, K, dtype=torch.bfloat16, device=table.device)
    _check(lib().bitlinear_embed(_ptr(ids), _ptr(table), M, V, K, _ptr(out), _stream()), "bitlinear_embed")
    return out


def bitlinear_selftest_wait_timeout(limit_us: int = 1000) -> None:
    """Launch the bounded-wait self-test: a tiny kernel whose wait runs out after limit_us microseconds."""
    _check(lib().bitlinear_selftest_wait_timeout(int(limit_us), _stream()), "bitlinear_selftest_wait_timeout")


def bitlinear_probe_int8_mma_rate(n_mma_per_sm: int) -> float:
    """Launch the int8 tensor-core rate probe on the current stream; returns the integer operations of the launch."""
    ops = ctypes.c_double(0.0)
    _check(lib().bitlinear_probe_int8_mma_rate(int(n_mma_per_sm), ctypes.byref(ops), _stream()), "bitlinear_probe_int8_mma_rate")
    return ops.value


def bitlinear_poll_status() -> int:
    return int(lib().bitlinear_poll_status(_stream()))
