"""ctypes front end of the CPU oracle (``bitrl_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's CPU-baseline
leg.  The CUDA library and its Python binding never import this package, and this package never imports
them.  Arrays are numpy; bf16 tensors travel as ``uint16`` bit patterns.

Each wrapper only marshals arguments; the arithmetic lives in the C++ file, where every function names
the passage of the paper it follows (Sec. III-A Eq. 2 for the ternary quantizer, the last paragraph of
Sec. III-A and the edge-deployment paragraph of Sec. V for the integer contraction).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

from .rl_math import gae, log_softmax, mlp_head, ppo_loss  # noqa: F401  (heads, GAE and PPO objective, numpy fp64)

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "bitrl_oracle.cpp"
_LIB = _HERE / "liboracle.so"

_i64 = ctypes.c_int64
_f32 = ctypes.c_float
_int = ctypes.c_int
_vp = ctypes.c_void_p


def build(force: bool = False) -> Path:
    """Compile the oracle with g++ (no fast-math, no FMA contraction)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.check_call(
            ["g++", "-O3", "-std=c++17", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
             "-pthread", str(_SRC), "-o", str(tmp)])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _lib.oracle_absmean.restype = _f32
        _lib.oracle_absmean.argtypes = [_vp, _i64]
        _lib.oracle_ternarize.argtypes = [_vp, _i64, _f32, _vp]
        _lib.oracle_w8_quantize.argtypes = [_vp, _i64, _vp, _vp]
        _lib.oracle_w8_quantize.restype = None
        _lib.oracle_w4_quantize.argtypes = [_vp, _i64, _vp, _vp]
        _lib.oracle_w4_quantize.restype = None
        _lib.oracle_w4_pack.argtypes = [_vp, _i64, _i64, _vp]
        _lib.oracle_w4_pack.restype = None
        _lib.oracle_pack.argtypes = [_vp, _i64, _i64, _vp]
        _lib.oracle_unpack.argtypes = [_vp, _i64, _i64, _vp]
        _lib.oracle_pack5.argtypes = [_vp, _i64, _i64, _vp]
        _lib.oracle_pack5.restype = None
        _lib.oracle_unpack5.argtypes = [_vp, _i64, _i64, _vp]
        _lib.oracle_unpack5.restype = None
        _lib.oracle_quant_act.argtypes = [_vp, _i64, _i64, _vp, _vp]
        _lib.oracle_contract.argtypes = [_vp, _vp, _i64, _i64, _i64, _vp, _int]
        _lib.oracle_contract_pairs.argtypes = [_vp, _vp, _i64, _vp, _vp, _i64, _vp]
        _lib.oracle_rescale.argtypes = [_vp, _i64, _i64, _f32, _vp, _vp, _vp, _vp]
        _lib.oracle_rmsnorm_f32.argtypes = [_vp, _i64, _i64, _vp]
        _lib.oracle_rmsnorm_bf16.argtypes = [_vp, _i64, _i64, _vp]
        _lib.oracle_relu2_gate.argtypes = [_vp, _i64, _i64, _vp]
        _lib.oracle_identity_attention.argtypes = [_vp, _i64, _i64, _i64, _i64, _vp]
        _lib.oracle_residual_add.argtypes = [_vp, _vp, _i64]
        _lib.oracle_attention.argtypes = [_vp, _vp, _i64, _i64, _i64, _i64, ctypes.c_double, _vp]
        _lib.oracle_attention.restype = None
        _lib.oracle_encoder_block.argtypes = [_vp, _i64, _i64, _i64, _i64, _i64,
                                              _vp, _f32, _vp, _f32, _vp, _f32, _vp, _f32, _int]
        _lib.oracle_encoder_block_states.argtypes = [_vp, _i64, _i64, _i64, _i64, _i64,
                                                     _vp, _f32, _vp, _f32, _vp, _f32, _vp, _f32,
                                                     _vp, _i64, ctypes.c_double, _int]
        _lib.oracle_encoder_block_states.restype = None
        for name in ("oracle_ternarize", "oracle_pack", "oracle_unpack", "oracle_quant_act",
                     "oracle_contract", "oracle_contract_pairs", "oracle_rescale", "oracle_rmsnorm_f32",
                     "oracle_rmsnorm_bf16", "oracle_relu2_gate", "oracle_identity_attention",
                     "oracle_residual_add", "oracle_encoder_block"):
            getattr(_lib, name).restype = None
    return _lib


def default_threads() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


def _c(a: np.ndarray, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _p(a: np.ndarray):
    return a.ctypes.data_as(_vp)


def absmean(W: np.ndarray) -> np.float32:
    """gamma = mean|W| (fp64 serial sum, one rounding to fp32)."""
    W = _c(W, np.float32)
    return np.float32(_L().oracle_absmean(_p(W), W.size))


def ternarize(W: np.ndarray, gamma=None):
    """Eq. 2 with tau=(gamma+1e-5)/2 as RoundClip.  Returns (W_q int8 [N,K], gamma fp32)."""
    W = _c(W, np.float32)
    g = absmean(W) if gamma is None else np.float32(gamma)
    Wq = np.empty(W.shape, np.int8)
    _L().oracle_ternarize(_p(W), W.size, _f32(float(g)), _p(Wq))
    return Wq, g


def w8_quantize(W: np.ndarray):
    """Symmetric absmax int8 quantization of a weight matrix (one scale per matrix).  Returns (W_q int8, scale fp32);
    ``bitlinear(x, W_q, scale)`` is then the W8A8 layer of the higher-precision critic."""
    W = _c(W, np.float32)
    Wq = np.empty(W.shape, np.int8)
    scale = np.zeros((1,), np.float32)
    _L().oracle_w8_quantize(_p(W), W.size, _p(Wq), _p(scale))
    return Wq, np.float32(scale[0])


def w4_quantize(W: np.ndarray):
    """Symmetric absmax int4 quantization (one scale per matrix).  Returns (W_q int8 with values in [-8, 7], scale)."""
    W = _c(W, np.float32)
    Wq = np.empty(W.shape, np.int8)
    scale = np.zeros((1,), np.float32)
    _L().oracle_w4_quantize(_p(W), W.size, _p(Wq), _p(scale))
    return Wq, np.float32(scale[0])


def w4_pack(Wq: np.ndarray) -> np.ndarray:
    """Two biased codes (q + 8) per byte, even k in the low nibble."""
    Wq = _c(Wq, np.int8)
    N, K = Wq.shape
    assert K % 2 == 0
    out = np.empty((N, K // 2), np.uint8)
    _L().oracle_w4_pack(_p(Wq), N, K, _p(out))
    return out


def pack(Wq: np.ndarray) -> np.ndarray:
    Wq = _c(Wq, np.int8)
    N, K = Wq.shape
    assert K % 4 == 0
    out = np.empty((N, K // 4), np.uint8)
    _L().oracle_pack(_p(Wq), N, K, _p(out))
    return out


def unpack(packed: np.ndarray, K: int) -> np.ndarray:
    packed = _c(packed, np.uint8)
    N = packed.shape[0]
    assert packed.shape[1] * 4 == K
    out = np.empty((N, K), np.int8)
    _L().oracle_unpack(_p(packed), N, K, _p(out))
    return out


def pack5(Wq: np.ndarray) -> np.ndarray:
    """Five weights per byte, base 3: uint8 [N, ceil(K/5)]; missing positions of a row's last byte count as zero weights."""
    Wq = _c(Wq, np.int8)
    N, K = Wq.shape
    out = np.empty((N, (K + 4) // 5), np.uint8)
    _L().oracle_pack5(_p(Wq), N, K, _p(out))
    return out


def unpack5(packed: np.ndarray, K: int) -> np.ndarray:
    packed = _c(packed, np.uint8)
    N = packed.shape[0]
    assert packed.shape[1] == (K + 4) // 5
    Wq = np.empty((N, K), np.int8)
    _L().oracle_unpack5(_p(packed), N, K, _p(Wq))
    return Wq


def quant_act(x_bf16: np.ndarray):
    """x_bf16: uint16 bit patterns [M,K].  Returns (x_q int8 [M,K], absmax fp32 [M])."""
    x = _c(x_bf16, np.uint16)
    M, K = x.shape
    xq = np.empty((M, K), np.int8)
    a = np.empty((M,), np.float32)
    _L().oracle_quant_act(_p(x), M, K, _p(xq), _p(a))
    return xq, a


def contract(xq: np.ndarray, Wq: np.ndarray, threads: int | None = None) -> np.ndarray:
    xq = _c(xq, np.int8)
    Wq = _c(Wq, np.int8)
    M, K = xq.shape
    N, K2 = Wq.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    _L().oracle_contract(_p(xq), _p(Wq), M, N, K, _p(acc), threads or default_threads())
    return acc


def contract_pairs(xq: np.ndarray, Wq: np.ndarray, ms: np.ndarray, ns: np.ndarray) -> np.ndarray:
    xq = _c(xq, np.int8)
    Wq = _c(Wq, np.int8)
    ms = _c(ms, np.int64)
    ns = _c(ns, np.int64)
    K = xq.shape[1]
    assert Wq.shape[1] == K and ms.shape == ns.shape
    acc = np.empty(ms.shape, np.int32)
    _L().oracle_contract_pairs(_p(xq), _p(Wq), K, _p(ms), _p(ns), ms.size, _p(acc))
    return acc


def rescale(acc: np.ndarray, gamma, absmax: np.ndarray):
    """Returns (y fp32, y bf16 bit patterns, y64 reference)."""
    acc = _c(acc, np.int32)
    a = _c(absmax, np.float32)
    M, N = acc.shape
    y32 = np.empty((M, N), np.float32)
    yb = np.empty((M, N), np.uint16)
    y64 = np.empty((M, N), np.float64)
    _L().oracle_rescale(_p(acc), M, N, _f32(float(gamma)), _p(a), _p(y32), _p(yb), _p(y64))
    return y32, yb, y64


def bitlinear(x_bf16: np.ndarray, Wq: np.ndarray, gamma, threads: int | None = None) -> dict:
    """quant -> contract -> rescale, with every intermediate returned."""
    xq, a = quant_act(x_bf16)
    acc = contract(xq, Wq, threads)
    y32, yb, y64 = rescale(acc, gamma, a)
    return {"xq": xq, "absmax": a, "acc": acc, "y32": y32, "ybf16": yb, "y64": y64}


def rmsnorm_bf16(x_bf16: np.ndarray) -> np.ndarray:
    x = _c(x_bf16, np.uint16)
    T, K = x.shape
    u = np.empty((T, K), np.uint16)
    _L().oracle_rmsnorm_bf16(_p(x), T, K, _p(u))
    return u


def rmsnorm_f32(x: np.ndarray) -> np.ndarray:
    x = _c(x, np.float32)
    T, K = x.shape
    u = np.empty((T, K), np.uint16)
    _L().oracle_rmsnorm_f32(_p(x), T, K, _p(u))
    return u


def relu2_gate(gu_bf16: np.ndarray) -> np.ndarray:
    gu = _c(gu_bf16, np.uint16)
    T, F2 = gu.shape
    assert F2 % 2 == 0
    f = np.empty((T, F2 // 2), np.float32)
    _L().oracle_relu2_gate(_p(gu), T, F2 // 2, _p(f))
    return f


def identity_attention(qkv_bf16: np.ndarray, n_heads: int, n_kv_heads: int, head_dim: int) -> np.ndarray:
    qkv = _c(qkv_bf16, np.uint16)
    T = qkv.shape[0]
    assert qkv.shape[1] == (n_heads + 2 * n_kv_heads) * head_dim
    att = np.empty((T, n_heads * head_dim), np.uint16)
    _L().oracle_identity_attention(_p(qkv), T, n_heads, n_kv_heads, head_dim, _p(att))
    return att


def attention(qkv_bf16: np.ndarray, states, n_heads: int, n_kv_heads: int, head_dim: int, theta: float) -> np.ndarray:
    """Causal GQA attention with rotary embedding inside each state; returns bf16 bits [T, n_heads*hd].
    `states` is either one length S shared by all states or the offsets [n_states+1] of ragged states."""
    qkv = _c(qkv_bf16, np.uint16)
    T = qkv.shape[0]
    off = _state_offsets(states, T)
    assert qkv.shape[1] == (n_heads + 2 * n_kv_heads) * head_dim and head_dim % 2 == 0
    att = np.empty((T, n_heads * head_dim), np.uint16)
    _L().oracle_attention(_p(qkv), _p(off), len(off) - 1, n_heads, n_kv_heads, head_dim, ctypes.c_double(theta), _p(att))
    return att


def residual_add(h_bf16: np.ndarray, y_bf16: np.ndarray) -> np.ndarray:
    h = np.array(h_bf16, dtype=np.uint16, order="C", copy=True)
    y = _c(y_bf16, np.uint16)
    assert h.shape == y.shape
    _L().oracle_residual_add(_p(h), _p(y), h.size)
    return h


def _state_offsets(states, T):
    if np.ndim(states) == 0:
        assert T % int(states) == 0
        return np.arange(0, T + 1, int(states), dtype=np.int64)
    off = _c(np.asarray(states), np.int64)
    assert off[0] == 0 and off[-1] == T and np.all(np.diff(off) >= 1)
    return off


def encoder_block(h_bf16: np.ndarray, d_ff: int, n_heads: int, n_kv_heads: int, layer, threads=None,
                  states=None, theta: float = 500000.0):
    """layer = ((Wq_qkv, g), (Wq_out, g), (Wq_gateup, g), (Wq_down, g)).  Returns the new h (bf16 bits).
    states=None: identity attention; else a common state length or the offsets of ragged states (real attention)."""
    h = np.array(h_bf16, dtype=np.uint16, order="C", copy=True)
    T, d = h.shape
    mats = [(_c(w, np.int8), float(g)) for (w, g) in layer]
    off = None if states is None else _state_offsets(states, T)
    _L().oracle_encoder_block_states(_p(h), T, d, d_ff, n_heads, n_kv_heads,
                                     _p(mats[0][0]), _f32(mats[0][1]), _p(mats[1][0]), _f32(mats[1][1]),
                                     _p(mats[2][0]), _f32(mats[2][1]), _p(mats[3][0]), _f32(mats[3][1]),
                                     None if off is None else _p(off), 0 if off is None else len(off) - 1,
                                     ctypes.c_double(theta), threads or default_threads())
    return h


def encoder_forward(h_bf16: np.ndarray, d_ff: int, n_heads: int, n_kv_heads: int, layers, threads=None,
                    states=None, theta: float = 500000.0):
    h = h_bf16
    for layer in layers:
        h = encoder_block(h, d_ff, n_heads, n_kv_heads, layer, threads, states, theta)
    return h
