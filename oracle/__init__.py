"""NumPy front end of the CPU oracle (oracle/bitlinear_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package imports nothing of theirs.

The C file is compiled on first use with gcc (-O2 -ffp-contract=off -fopenmp)
into oracle/liboracle.so; arrays are passed as plain pointers.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "bitlinear_oracle.c"
_LIB = _HERE / "liboracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle if the shared object is missing or older than its source."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC",
               "-shared", "-Wall", "-Wextra", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        lib.oracle_pack.restype = ctypes.c_int
        lib.oracle_unpack.restype = ctypes.c_int
        lib.oracle_pack5.restype = ctypes.c_int
        lib.oracle_unpack5.restype = ctypes.c_int
        lib.oracle_packed5_bytes.restype = ctypes.c_long
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even."""
    x = _c(x, np.float32)
    out = np.empty(x.shape, np.uint16)
    _load().oracle_f32_to_bf16(_p(x), ctypes.c_long(x.size), _p(out))
    return out


def bf16_to_f32(x: np.ndarray) -> np.ndarray:
    x = _c(x, np.uint16)
    out = np.empty(x.shape, np.float32)
    _load().oracle_bf16_to_f32(_p(x), ctypes.c_long(x.size), _p(out))
    return out


def absmax_quant(y: np.ndarray):
    """Steps 3-4 alone on fp32 rows [M, K] -> (q int8 [M,K], d fp32 [M], xsum int32 [M])."""
    y = _c(y, np.float32)
    M, K = y.shape
    q = np.empty((M, K), np.int8)
    d = np.empty(M, np.float32)
    xsum = np.empty(M, np.int32)
    _load().oracle_absmax_quant(_p(y), M, K, _p(q), _p(d), _p(xsum))
    return q, d, xsum


def rmsnorm_quant(x_bf16: np.ndarray, gain_bf16: np.ndarray | None, eps: float, want_norm: bool = False):
    """Steps 1-4 on bf16 bit patterns [M, K].

    Returns dict(q, d, xsum, fragile[, y_norm]).
    """
    x = _c(x_bf16, np.uint16)
    M, K = x.shape
    g = None if gain_bf16 is None else _c(gain_bf16, np.uint16)
    if g is not None:
        assert g.shape == (K,)
    q = np.empty((M, K), np.int8)
    d = np.empty(M, np.float32)
    xsum = np.empty(M, np.int32)
    fragile = np.zeros(M, np.int32)
    yn = np.empty((M, K), np.float32) if want_norm else None
    _load().oracle_rmsnorm_quant(_p(x), _p(g), ctypes.c_float(eps), M, K, _p(q), _p(d), _p(xsum), _p(yn),
                                 _p(fragile))
    out = dict(q=q, d=d, xsum=xsum, fragile=fragile)
    if want_norm:
        out["y_norm"] = yn
    return out


def weight_scale(W: np.ndarray, eps_w: float):
    """Step 5 -> (s_w as np.float32, fragile flag)."""
    W = _c(W, np.float32)
    s = ctypes.c_float(0.0)
    frag = ctypes.c_int(0)
    _load().oracle_weight_scale(_p(W), ctypes.c_long(W.size), ctypes.c_float(eps_w), ctypes.byref(s),
                                ctypes.byref(frag))
    return np.float32(s.value), bool(frag.value)


def weight_quant(W: np.ndarray, s_w) -> np.ndarray:
    """Step 6 -> int8 array of W's shape with values in {-1, 0, 1}."""
    W = _c(W, np.float32)
    wq = np.empty(W.shape, np.int8)
    _load().oracle_weight_quant(_p(W), ctypes.c_long(W.size), ctypes.c_float(float(s_w)), _p(wq))
    return wq


def pack(wq: np.ndarray) -> np.ndarray:
    """Step 7 -> uint8 [N*K/4] in the tiled 2-bit layout."""
    wq = _c(wq, np.int8)
    N, K = wq.shape
    out = np.empty(N * K // 4, np.uint8)
    rc = _load().oracle_pack(_p(wq), N, K, _p(out))
    if rc != 0:
        raise ValueError(f"oracle_pack failed with {rc}")
    return out


def unpack(packed: np.ndarray, N: int, K: int) -> np.ndarray:
    packed = _c(packed, np.uint8)
    assert packed.size == N * K // 4
    wq = np.empty((N, K), np.int8)
    rc = _load().oracle_unpack(_p(packed), N, K, _p(wq))
    if rc != 0:
        raise ValueError(f"oracle_unpack failed with {rc}")
    return wq


def packed5_bytes(N: int, K: int) -> int:
    """Bytes of the five-per-byte form of an [N, K] ternary matrix (K padded to a multiple of 320 columns)."""
    return int(_load().oracle_packed5_bytes(N, K))


def pack5(wq: np.ndarray) -> np.ndarray:
    """Step 7b -> uint8 [N * Kp / 5] in the tiled five-per-byte layout."""
    wq = _c(wq, np.int8)
    N, K = wq.shape
    nbytes = packed5_bytes(N, K)
    if nbytes == 0:
        raise ValueError("oracle_pack5: unsupported shape")
    out = np.empty(nbytes, np.uint8)
    rc = _load().oracle_pack5(_p(wq), N, K, _p(out))
    if rc != 0:
        raise ValueError(f"oracle_pack5 failed with {rc}")
    return out


def unpack5(packed: np.ndarray, N: int, K: int) -> np.ndarray:
    packed = _c(packed, np.uint8)
    assert packed.size == packed5_bytes(N, K)
    wq = np.empty((N, K), np.int8)
    rc = _load().oracle_unpack5(_p(packed), N, K, _p(wq))
    if rc != 0:
        raise ValueError(f"oracle_unpack5 failed with {rc}")
    return wq


def matmul_i32(q: np.ndarray, wq: np.ndarray) -> np.ndarray:
    """Step 8: q int8 [M,K], wq int8 [N,K] -> int32 [M,N]."""
    q = _c(q, np.int8)
    wq = _c(wq, np.int8)
    M, K = q.shape
    N, K2 = wq.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    _load().oracle_matmul_i32(_p(q), _p(wq), M, N, K, _p(acc))
    return acc


def matmul_i32_sampled(q: np.ndarray, wq: np.ndarray, m_idx: np.ndarray, n_idx: np.ndarray) -> np.ndarray:
    """Step 8 for selected (m, n) pairs only."""
    q = _c(q, np.int8)
    wq = _c(wq, np.int8)
    m_idx = _c(m_idx, np.int32)
    n_idx = _c(n_idx, np.int32)
    K = q.shape[1]
    assert wq.shape[1] == K and m_idx.shape == n_idx.shape
    acc = np.empty(m_idx.size, np.int32)
    _load().oracle_matmul_i32_sampled(_p(q), _p(wq), K, _p(m_idx), _p(n_idx), ctypes.c_long(m_idx.size), _p(acc))
    return acc


def dequant(acc: np.ndarray, s_w, d: np.ndarray) -> np.ndarray:
    """Step 9: int32 [M,N] -> fp32 [M,N]."""
    acc = _c(acc, np.int32)
    d = _c(d, np.float32)
    M, N = acc.shape
    y = np.empty((M, N), np.float32)
    _load().oracle_dequant(_p(acc), ctypes.c_float(float(s_w)), _p(d), M, N, _p(y))
    return y


def quantize_weights(W: np.ndarray, eps_w: float):
    """Steps 5-7 -> dict(s_w, wq, packed, fragile)."""
    s_w, frag = weight_scale(W, eps_w)
    wq = weight_quant(W, s_w)
    return dict(s_w=s_w, wq=wq, packed=pack(wq), fragile=frag)


def bitlinear_forward(x_bf16: np.ndarray, gain_bf16, rms_eps: float, wq: np.ndarray, s_w):
    """Steps 1-4 and 8-9 chained -> dict(q, d, xsum, acc, y, fragile)."""
    a = rmsnorm_quant(x_bf16, gain_bf16, rms_eps)
    acc = matmul_i32(a["q"], wq)
    y = dequant(acc, s_w, a["d"])
    return dict(q=a["q"], d=a["d"], xsum=a["xsum"], fragile=a["fragile"], acc=acc, y=y)


# ---- glue between the BitLinear matmuls of a decoder layer (paper Section 2: squared ReLU in the feed-forward block,
# ---- residual connections), each followed by the next BitLinear's own RMSNorm + quantiser.  One fp32 operation per
# ---- arithmetic step, then one round-to-nearest-even cast to bf16: the next BitLinear reads bf16.


def glue_relu2(gate: np.ndarray, up: np.ndarray) -> np.ndarray:
    """f = bf16( fl32( fl32(r * r) * up ) ), r = max(gate, 0)  ->  bf16 bit patterns."""
    gate, up = _c(gate, np.float32), _c(up, np.float32)
    r = np.maximum(gate, np.float32(0.0))
    return f32_to_bf16(((r * r).astype(np.float32) * up).astype(np.float32))


def glue_residual(h_bits: np.ndarray, y: np.ndarray) -> np.ndarray:
    """h' = bf16( fl32( float(h) + y ) )  ->  bf16 bit patterns."""
    return f32_to_bf16((bf16_to_f32(h_bits) + _c(y, np.float32)).astype(np.float32))


def glue_attn_standin(q: np.ndarray, v: np.ndarray, n_q_heads: int, n_kv_heads: int, head_dim: int) -> np.ndarray:
    """Stand-in for attention (which is not a BitLinear): a[m, h*D + j] = bf16( fl32( q[m, h*D + j] + v[m, kv(h)*D + j] ) ),
    kv(h) = h // (n_q_heads // n_kv_heads)."""
    q, v = _c(q, np.float32), _c(v, np.float32)
    group = n_q_heads // n_kv_heads
    a = np.empty_like(q)
    for head in range(n_q_heads):
        kv = head // group
        a[:, head * head_dim:(head + 1) * head_dim] = (q[:, head * head_dim:(head + 1) * head_dim] +
                                                       v[:, kv * head_dim:(kv + 1) * head_dim]).astype(np.float32)
    return f32_to_bf16(a)


def relu2_rmsnorm_quant(gate, up, gain_bf16, eps: float):
    """Squared-ReLU gate fused with the down projection's sub-LN + int8 quantiser: rmsnorm_quant(glue_relu2(gate, up)).
    Returns the dict of rmsnorm_quant plus x = the bf16 bit patterns that were quantised."""
    x = glue_relu2(gate, up)
    out = rmsnorm_quant(x, gain_bf16, eps)
    out["x"] = x
    return out


def residual_rmsnorm_quant(h_bits, y, gain_bf16, eps: float):
    """Residual add fused with the next BitLinear's RMSNorm + quantiser; x = the new hidden state (bf16 bits)."""
    x = glue_residual(h_bits, y)
    out = rmsnorm_quant(x, gain_bf16, eps)
    out["x"] = x
    return out


def attn_standin_rmsnorm_quant(q, v, n_q_heads: int, n_kv_heads: int, head_dim: int, gain_bf16, eps: float):
    x = glue_attn_standin(q, v, n_q_heads, n_kv_heads, head_dim)
    out = rmsnorm_quant(x, gain_bf16, eps)
    out["x"] = x
    return out
