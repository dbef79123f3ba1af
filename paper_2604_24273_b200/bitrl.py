"""Thin ctypes binding of ``libbitrl.so`` (declared in ``include/bitrl.h``).

Argument marshalling only: every step of the layer runs in the library's CUDA kernels.  PyTorch is used for
device memory and streams.  There is no CPU fallback: if the library is missing or a call fails, an
exception is raised.

The functions mirror the C names without the ``bitrl_`` prefix:
``pack_ternary``, ``Linear`` (create/destroy), ``quant_act``, ``bitlinear_forward``, ``bitlinear_forward_debug``,
``bitlinear_forward_q``, ``rmsnorm_quant``, ``vrepeat_rmsnorm_quant``, ``relu2gate_rmsnorm_quant``, ``attention``,
``pool_last_token``, ``Encoder`` (``forward``, ``forward_states``), ``heads_forward``, ``gae``, ``ppo_loss``,
``w8_quantize``, ``w8a8_forward``, ``w4_quantize``, ``w4a8_forward``,
``poll_status``.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_HERE = Path(__file__).resolve().parent
LIB_PATH = _HERE / "libbitrl.so"

OK = 0
ERR_NULL, ERR_SHAPE, ERR_ALIGN, ERR_ARCH, ERR_CUDA, ERR_TIMEOUT, ERR_WORKSPACE, ERR_DTYPE, ERR_LIMIT = range(-1, -10, -1)
PACK_STATIC_MAX_WEIGHTS = 1 << 28
OUT_F32, OUT_BF16 = 0, 1
GEMV_MAX_M = 16

_vp = ctypes.c_void_p
_i32 = ctypes.c_int32
_sz = ctypes.c_size_t

class W8Matrix(ctypes.Structure):
    """Mirror of ``bitrl_w8_matrix_t``."""
    _fields_ = [("wq", ctypes.c_void_p), ("scale", ctypes.c_void_p), ("N", ctypes.c_int32), ("K", ctypes.c_int32)]


class HeadDesc(ctypes.Structure):
    """Mirror of ``bitrl_head_t``."""
    _fields_ = [("W1t", ctypes.c_void_p), ("b1", ctypes.c_void_p), ("W2t", ctypes.c_void_p), ("b2", ctypes.c_void_p),
                ("W3t", ctypes.c_void_p), ("b3", ctypes.c_void_p), ("n_out", ctypes.c_int32)]


_f32 = ctypes.c_float

EXPORTS = {
    "bitrl_pack_workspace_bytes": (_sz, [_i32, _i32]),
    "bitrl_pack_ternary": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp, _sz, _vp]),
    "bitrl_pack_ternary_static": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp]),
    "bitrl_linear_create": (_i32, [_vp, _vp, _i32, _i32, ctypes.POINTER(_vp), _vp]),
    "bitrl_linear_destroy": (_i32, [_vp]),
    "bitrl_quant_act": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp, _vp]),
    "bitrl_workspace_bytes": (_sz, [_i32, _i32, _i32]),
    "bitrl_bitlinear_forward": (_i32, [_vp, _vp, _i32, _i32, _i32, _vp, _i32, _vp, _sz, _vp]),
    "bitrl_bitlinear_forward_multi": (_i32, [_i32, ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp), _i32,
                                             _i32, _vp]),
    "bitrl_bitlinear_forward_debug": (_i32, [_vp, _vp, _i32, _i32, _i32, _vp, _i32, _vp, _sz, _vp, _vp, _vp, _vp]),
    "bitrl_bitlinear_forward_q": (_i32, [_vp, _vp, _vp, _vp, _i32, _vp, _i32, _vp, _vp, _vp]),
    "bitrl_rmsnorm_quant": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp]),
    "bitrl_vrepeat_rmsnorm_quant": (_i32, [_vp, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp]),
    "bitrl_relu2gate_rmsnorm_quant": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp]),
    "bitrl_encoder_create": (_i32, [ctypes.POINTER(_vp), _i32, _i32, _i32, _i32, _i32, ctypes.POINTER(_vp)]),
    "bitrl_encoder_destroy": (_i32, [_vp]),
    "bitrl_encoder_workspace_bytes": (_sz, [_vp, _i32]),
    "bitrl_encoder_forward": (_i32, [_vp, _vp, _i32, _vp, _vp, _sz, _vp]),
    "bitrl_attention_workspace_bytes": (_sz, [_i32, _i32]),
    "bitrl_attention": (_i32, [_vp, _i32, _vp, _i32, _i32, _i32, _i32, _i32, ctypes.c_double, _vp, _vp, _sz, _vp]),
    "bitrl_pool_last_token": (_i32, [_vp, _i32, _vp, _i32, _i32, _i32, _vp, _vp]),
    "bitrl_encoder_states_workspace_bytes": (_sz, [_vp, _i32, _i32]),
    "bitrl_encoder_forward_states": (_i32, [_vp, _vp, _i32, _vp, _i32, _i32, ctypes.c_double, _vp, _vp, _vp, _sz, _vp]),
    "bitrl_heads_forward": (_i32, [_vp, _i32, _i32, _i32, _i32, ctypes.POINTER(HeadDesc), _i32, ctypes.POINTER(_vp), _vp]),
    "bitrl_gae": (_i32, [_vp, _vp, _vp, _i32, _i32, _f32, _f32, _vp, _vp, _vp]),
    "bitrl_ppo_loss": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _f32, _f32, _vp, _vp, _vp, _vp, _vp]),
    "bitrl_w8_quantize": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp]),
    "bitrl_w8a8_workspace_bytes": (_sz, [_i32, _i32]),
    "bitrl_w8a8_forward": (_i32, [_vp, _vp, _vp, _i32, _i32, _i32, _vp, _i32, _vp, _sz, _vp]),
    "bitrl_w8a8_forward_debug": (_i32, [_vp, _vp, _vp, _i32, _i32, _i32, _vp, _i32, _vp, _sz, _vp, _vp, _vp, _vp]),
    "bitrl_w8a8_forward_multi": (_i32, [_i32, ctypes.POINTER(W8Matrix), ctypes.POINTER(_vp), ctypes.POINTER(_vp), _i32, _i32, _vp]),
    "bitrl_w4a8_forward_multi": (_i32, [_i32, ctypes.POINTER(W8Matrix), ctypes.POINTER(_vp), ctypes.POINTER(_vp), _i32, _i32, _vp]),
    "bitrl_w4_quantize": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp]),
    "bitrl_w4a8_workspace_bytes": (_sz, [_i32, _i32, _i32]),
    "bitrl_w4a8_forward": (_i32, [_vp, _vp, _vp, _i32, _i32, _i32, _vp, _i32, _vp, _sz, _vp]),
    "bitrl_w4a8_forward_debug": (_i32, [_vp, _vp, _vp, _i32, _i32, _i32, _vp, _i32, _vp, _sz, _vp, _vp, _vp, _vp]),
    "bitrl_pack5": (_i32, [_vp, _i32, _i32, _vp, _vp]),
    "bitrl_linear5_create": (_i32, [_vp, _vp, _i32, _i32, ctypes.POINTER(_vp), _vp]),
    "bitrl_linear5_destroy": (_i32, [_vp]),
    "bitrl_linear5_bytes": (_sz, [_vp]),
    "bitrl_bitlinear5_forward_multi": (_i32, [_i32, ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp), _i32,
                                              _i32, _vp]),
    "bitrl_selftest_wait_timeout": (_i32, [ctypes.c_int64, _vp]),
    "bitrl_poll_status": (_i32, [_vp]),
    "bitrl_last_timeout_stage": (_i32, []),
    "bitrl_last_cuda_error": (_i32, []),
    "bitrl_status_string": (ctypes.c_char_p, [_i32]),
    "bitrl_launch_count": (ctypes.c_uint64, []),
    "bitrl_gemm_plan": (_i32, [_i32, _i32, _i32, _i32, ctypes.POINTER(_i32), ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
}


class BitrlError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().bitrl_status_string(status).decode()
        extra = f" (cuda error {lib().bitrl_last_cuda_error()})" if status == ERR_CUDA else ""
        super().__init__(f"{where}: {msg}{extra} [{status}]")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the library; fails loudly when it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2604_24273_b200.build` "
                              "(or __graft_entry__.build()); there is no CPU fallback")
        L = ctypes.CDLL(str(LIB_PATH))
        for name, (res, args) in EXPORTS.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != OK:
        raise BitrlError(status, where)


def _ptr(t):
    return None if t is None else _vp(t.data_ptr())


def _stream():
    return _vp(torch.cuda.current_stream().cuda_stream)


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of dtype {dtype}")
    return t


def launch_count() -> int:
    return int(lib().bitrl_launch_count())


GEMM_SINGLE, GEMM_SPLIT_SCRATCH, GEMM_SPLIT_CLUSTER, GEMM_PAIRED = 0, 1, 2, 3


def gemm_plan(M: int, K: int, N: int, with_workspace: bool = True):
    """(tokens per tile, k ranges per tile, kind) the launcher takes for this product on the current device."""
    tok, splits, kind = _i32(), _i32(), _i32()
    _check(lib().bitrl_gemm_plan(M, K, N, int(with_workspace), ctypes.byref(tok), ctypes.byref(splits),
                                 ctypes.byref(kind)), "bitrl_gemm_plan")
    return tok.value, splits.value, kind.value


def poll_status() -> None:
    """Synchronizes the current stream and raises if a device-side wait expired."""
    _check(lib().bitrl_poll_status(_stream()), "bitrl_poll_status")


def pack_ternary(W: torch.Tensor):
    """W: CUDA fp32 [N,K].  Returns (packed uint8 [N,K/4] canonical, gamma fp32 [1])."""
    _dev(W, torch.float32, "W")
    N, K = W.shape
    packed = torch.empty((N, K // 4), dtype=torch.uint8, device=W.device)
    gamma = torch.empty((1,), dtype=torch.float32, device=W.device)
    nbytes = lib().bitrl_pack_workspace_bytes(N, K)
    ws = torch.empty((nbytes,), dtype=torch.uint8, device=W.device)
    _check(lib().bitrl_pack_ternary(_ptr(W), N, K, _ptr(packed), _ptr(gamma), _ptr(ws), nbytes, _stream()),
           "bitrl_pack_ternary")
    return packed, gamma


def pack_ternary_static(W: torch.Tensor, packed: torch.Tensor, gamma: torch.Tensor) -> None:
    """``bitrl_pack_ternary_static``: packs into caller-provided ``packed`` / ``gamma`` and allocates nothing, for
    callers that may not touch the device allocator.  At most ``PACK_STATIC_MAX_WEIGHTS`` weights; calls must not
    overlap on the GPU (they share one fixed scratch array inside the library)."""
    _dev(W, torch.float32, "W")
    _dev(packed, torch.uint8, "packed")
    _dev(gamma, torch.float32, "gamma")
    N, K = W.shape
    if packed.numel() != N * K // 4 or gamma.numel() < 1:
        raise ValueError("packed must hold N*K/4 bytes and gamma one float")
    _check(lib().bitrl_pack_ternary_static(_ptr(W), N, K, _ptr(packed), _ptr(gamma), _stream()),
           "bitrl_pack_ternary_static")


class Linear:
    """Owns a ``bitrl_linear_t`` (kernel-layout ternary weights + gamma)."""

    def __init__(self, packed: torch.Tensor, gamma: torch.Tensor, N: int, K: int):
        _dev(packed, torch.uint8, "packed")
        _dev(gamma, torch.float32, "gamma")
        self.N, self.K = int(N), int(K)
        self.device = packed.device
        h = _vp()
        _check(lib().bitrl_linear_create(_ptr(packed), _ptr(gamma), self.N, self.K, ctypes.byref(h), _stream()),
               "bitrl_linear_create")
        self.handle = h

    @classmethod
    def from_master(cls, W: torch.Tensor) -> "Linear":
        packed, gamma = pack_ternary(W)
        return cls(packed, gamma, W.shape[0], W.shape[1])

    def close(self):
        if getattr(self, "handle", None):
            lib().bitrl_linear_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def quant_act(x: torch.Tensor, want_rowsum: bool = True):
    """x: CUDA bf16 [M,K] -> (x_q int8 [M,K], absmax fp32 [M], rowsum int32 [M] or None)."""
    _dev(x, torch.bfloat16, "x")
    M, K = x.shape
    xq = torch.empty((M, K), dtype=torch.int8, device=x.device)
    a = torch.empty((M,), dtype=torch.float32, device=x.device)
    rs = torch.empty((M,), dtype=torch.int32, device=x.device) if want_rowsum else None
    _check(lib().bitrl_quant_act(_ptr(x), M, K, _ptr(xq), _ptr(a), _ptr(rs), _stream()), "bitrl_quant_act")
    return xq, a, rs


def workspace_bytes(M: int, K: int, N: int) -> int:
    return int(lib().bitrl_workspace_bytes(M, K, N))


def _out(M, N, out_dtype, device):
    return torch.empty((M, N), dtype=torch.float32 if out_dtype == OUT_F32 else torch.bfloat16, device=device)


def bitlinear_forward(w: Linear, x: torch.Tensor, out_dtype: int = OUT_BF16, y: torch.Tensor | None = None,
                      workspace: torch.Tensor | None = None, streaming: bool = False) -> torch.Tensor:
    """y = BitLinear(x): x CUDA bf16 [M,K] -> y [M,N].  ``streaming`` (M <= GEMV_MAX_M): pass no workspace, so that
    the streaming kernel serves the call whatever M is."""
    _dev(x, torch.bfloat16, "x")
    M, K = x.shape
    if y is None:
        y = _out(M, w.N, out_dtype, x.device)
    need = 0 if streaming else workspace_bytes(M, K, w.N)
    if workspace is None and need:
        workspace = torch.empty((need,), dtype=torch.uint8, device=x.device)
    nbytes = 0 if workspace is None else workspace.numel()
    _check(lib().bitrl_bitlinear_forward(w.handle, _ptr(x), M, K, w.N, _ptr(y), out_dtype, _ptr(workspace), nbytes,
                                         _stream()), "bitrl_bitlinear_forward")
    return y


class MultiCall:
    """Argument block of ``bitrl_bitlinear_forward_multi``: ``count`` independent layers, one launch.

    The three host pointer arrays are built once; ``run()`` only makes the C call (cheap enough to sit in a
    CUDA-graph capture or a hot loop)."""

    def __init__(self, ws, xs, ys, out_dtype: int = OUT_BF16):
        assert len(ws) == len(xs) == len(ys) >= 1
        self.M = xs[0].shape[0]
        for w, x, y in zip(ws, xs, ys):
            _dev(x, torch.bfloat16, "x")
            assert x.shape == (self.M, w.K) and tuple(y.shape) == (self.M, w.N) and y.is_cuda and y.is_contiguous()
            assert y.dtype == (torch.float32 if out_dtype == OUT_F32 else torch.bfloat16)
        self.keep = (list(ws), list(xs), list(ys))
        n = len(ws)
        self.count, self.out_dtype = n, out_dtype
        self.w = (_vp * n)(*[w.handle for w in ws])
        self.x = (_vp * n)(*[x.data_ptr() for x in xs])
        self.y = (_vp * n)(*[y.data_ptr() for y in ys])

    def run(self):
        _check(lib().bitrl_bitlinear_forward_multi(self.count, self.w, self.x, self.y, self.M, self.out_dtype,
                                                   _stream()), "bitrl_bitlinear_forward_multi")
        return self.keep[2]


LINEAR5_MAX_M = 2


def pack5(packed: torch.Tensor, N: int, K: int) -> torch.Tensor:
    """Canonical 2-bit codes [N,K/4] -> five weights per byte [N, ceil(K/5)] (base 3)."""
    _dev(packed, torch.uint8, "packed")
    out = torch.empty((N, (K + 4) // 5), dtype=torch.uint8, device=packed.device)
    _check(lib().bitrl_pack5(_ptr(packed), N, K, _ptr(out), _stream()), "bitrl_pack5")
    return out


class Linear5:
    """Owns a ``bitrl_linear5_t``: the weights in the five-per-byte kernel layout + gamma."""

    def __init__(self, packed5: torch.Tensor, gamma: torch.Tensor, N: int, K: int):
        _dev(packed5, torch.uint8, "packed5")
        _dev(gamma, torch.float32, "gamma")
        self.N, self.K = int(N), int(K)
        h = _vp()
        _check(lib().bitrl_linear5_create(_ptr(packed5), _ptr(gamma), self.N, self.K, ctypes.byref(h), _stream()),
               "bitrl_linear5_create")
        self.handle = h
        self.nbytes = int(lib().bitrl_linear5_bytes(h))

    @classmethod
    def from_master(cls, W: torch.Tensor) -> "Linear5":
        packed, gamma = pack_ternary(W)
        return cls(pack5(packed, W.shape[0], W.shape[1]), gamma, W.shape[0], W.shape[1])

    def close(self):
        if getattr(self, "handle", None):
            lib().bitrl_linear5_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class MultiCall5(MultiCall):
    """Argument block of ``bitrl_bitlinear5_forward_multi`` (M <= 2)."""

    def run(self):
        _check(lib().bitrl_bitlinear5_forward_multi(self.count, self.w, self.x, self.y, self.M, self.out_dtype,
                                                    _stream()), "bitrl_bitlinear5_forward_multi")
        return self.keep[2]


def bitlinear_forward_debug(w: Linear, x: torch.Tensor, out_dtype: int = OUT_BF16, streaming: bool = False):
    """Returns (y, x_q int8 [M,K], absmax fp32 [M], acc int32 [M,N]).  ``streaming``: as in bitlinear_forward."""
    _dev(x, torch.bfloat16, "x")
    M, K = x.shape
    y = _out(M, w.N, out_dtype, x.device)
    xq = torch.empty((M, K), dtype=torch.int8, device=x.device)
    a = torch.empty((M,), dtype=torch.float32, device=x.device)
    acc = torch.empty((M, w.N), dtype=torch.int32, device=x.device)
    need = 0 if streaming else workspace_bytes(M, K, w.N)
    ws = torch.empty((max(need, 16),), dtype=torch.uint8, device=x.device)
    _check(lib().bitrl_bitlinear_forward_debug(w.handle, _ptr(x), M, K, w.N, _ptr(y), out_dtype, _ptr(ws), ws.numel(),
                                               _ptr(xq), _ptr(a), _ptr(acc), _stream()),
           "bitrl_bitlinear_forward_debug")
    return y, xq, a, acc


def bitlinear_forward_q(w: Linear, xq: torch.Tensor, absmax: torch.Tensor, rowsum: torch.Tensor,
                        out_dtype: int = OUT_BF16, residual: torch.Tensor | None = None, y: torch.Tensor | None = None,
                        want_acc: bool = False):
    _dev(xq, torch.int8, "xq")
    _dev(absmax, torch.float32, "absmax")
    _dev(rowsum, torch.int32, "rowsum")
    M = xq.shape[0]
    if y is None:
        y = _out(M, w.N, out_dtype, xq.device)
    acc = torch.empty((M, w.N), dtype=torch.int32, device=xq.device) if want_acc else None
    if residual is not None:
        _dev(residual, torch.bfloat16, "residual")
    _check(lib().bitrl_bitlinear_forward_q(w.handle, _ptr(xq), _ptr(absmax), _ptr(rowsum), M, _ptr(y), out_dtype,
                                           _ptr(residual), _ptr(acc), _stream()), "bitrl_bitlinear_forward_q")
    return (y, acc) if want_acc else y


def _producer_out(T, K, device, want_u):
    xq = torch.empty((T, K), dtype=torch.int8, device=device)
    a = torch.empty((T,), dtype=torch.float32, device=device)
    rs = torch.empty((T,), dtype=torch.int32, device=device)
    u = torch.empty((T, K), dtype=torch.bfloat16, device=device) if want_u else None
    return xq, a, rs, u


def rmsnorm_quant(h: torch.Tensor, want_u: bool = False):
    _dev(h, torch.bfloat16, "h")
    T, K = h.shape
    xq, a, rs, u = _producer_out(T, K, h.device, want_u)
    _check(lib().bitrl_rmsnorm_quant(_ptr(h), T, K, _ptr(xq), _ptr(a), _ptr(rs), _ptr(u), _stream()),
           "bitrl_rmsnorm_quant")
    return xq, a, rs, u


def vrepeat_rmsnorm_quant(qkv: torch.Tensor, n_heads: int, n_kv_heads: int, head_dim: int, want_u: bool = False):
    _dev(qkv, torch.bfloat16, "qkv")
    T = qkv.shape[0]
    assert qkv.shape[1] == (n_heads + 2 * n_kv_heads) * head_dim
    xq, a, rs, u = _producer_out(T, n_heads * head_dim, qkv.device, want_u)
    _check(lib().bitrl_vrepeat_rmsnorm_quant(_ptr(qkv), T, n_heads, n_kv_heads, head_dim, _ptr(xq), _ptr(a), _ptr(rs),
                                             _ptr(u), _stream()), "bitrl_vrepeat_rmsnorm_quant")
    return xq, a, rs, u


def relu2gate_rmsnorm_quant(gu: torch.Tensor, want_u: bool = False):
    _dev(gu, torch.bfloat16, "gu")
    T, F2 = gu.shape
    xq, a, rs, u = _producer_out(T, F2 // 2, gu.device, want_u)
    _check(lib().bitrl_relu2gate_rmsnorm_quant(_ptr(gu), T, F2 // 2, _ptr(xq), _ptr(a), _ptr(rs), _ptr(u), _stream()),
           "bitrl_relu2gate_rmsnorm_quant")
    return xq, a, rs, u


ATTN_MAX_STATE_TOKENS = 128
ROPE_THETA = 500000.0


def _states(states, T: int, device):
    """``states``: an int (every state has that many tokens) or a CUDA int32 tensor of offsets [n_states+1] together
    with the largest length, as a tuple ``(offsets, max_len)``.  Returns (offsets or None, n_states, max_len)."""
    if isinstance(states, int):
        if T % states != 0:
            raise ValueError("T is not a multiple of the common state length")
        return None, T // states, states
    off, max_len = states
    _dev(off, torch.int32, "state offsets")
    return off, off.numel() - 1, int(max_len)


def attention(qkv: torch.Tensor, states, n_heads: int, n_kv_heads: int, head_dim: int,
              theta: float = ROPE_THETA) -> torch.Tensor:
    """Causal GQA attention with rotary embedding inside each state: qkv bf16 [T, (nh+2nkv)*hd] -> att bf16 [T, nh*hd]."""
    _dev(qkv, torch.bfloat16, "qkv")
    T = qkv.shape[0]
    assert qkv.shape[1] == (n_heads + 2 * n_kv_heads) * head_dim
    off, n_states, max_len = _states(states, T, qkv.device)
    att = torch.empty((T, n_heads * head_dim), dtype=torch.bfloat16, device=qkv.device)
    nbytes = max(int(lib().bitrl_attention_workspace_bytes(max_len, head_dim)), 16)
    ws = torch.empty((nbytes,), dtype=torch.uint8, device=qkv.device)
    _check(lib().bitrl_attention(_ptr(qkv), T, _ptr(off), n_states, max_len, n_heads, n_kv_heads, head_dim,
                                 float(theta), _ptr(att), _ptr(ws), nbytes, _stream()), "bitrl_attention")
    return att


def pool_last_token(h: torch.Tensor, states) -> torch.Tensor:
    """h bf16 [T,d] -> bf16 [n_states,d]: the last token of every state."""
    _dev(h, torch.bfloat16, "h")
    T, d = h.shape
    off, n_states, max_len = _states(states, T, h.device)
    out = torch.empty((n_states, d), dtype=torch.bfloat16, device=h.device)
    _check(lib().bitrl_pool_last_token(_ptr(h), T, _ptr(off), n_states, max_len, d, _ptr(out), _stream()),
           "bitrl_pool_last_token")
    return out


def w8_quantize(W: torch.Tensor):
    """W CUDA fp32 [N,K] -> (W_q int8 [N,K], scale fp32 [2]; scale[0] is the scale)."""
    _dev(W, torch.float32, "W")
    N, K = W.shape
    wq = torch.empty((N, K), dtype=torch.int8, device=W.device)
    scale = torch.empty((2,), dtype=torch.float32, device=W.device)
    _check(lib().bitrl_w8_quantize(_ptr(W), N, K, _ptr(wq), _ptr(scale), _stream()), "bitrl_w8_quantize")
    return wq, scale


def w8a8_forward(wq: torch.Tensor, scale: torch.Tensor, x: torch.Tensor, out_dtype: int = OUT_BF16, debug: bool = False,
                 y: torch.Tensor | None = None, workspace: torch.Tensor | None = None, streaming: bool = False):
    """y = W8A8(x).  With debug=True returns (y, x_q, absmax, acc).  ``streaming`` (M <= GEMV_MAX_M): pass a workspace too
    small for the GEMM form, so that the streaming kernel serves the call whatever M is."""
    _dev(wq, torch.int8, "wq")
    _dev(scale, torch.float32, "scale")
    _dev(x, torch.bfloat16, "x")
    M, K = x.shape
    N = wq.shape[0]
    if y is None:
        y = _out(M, N, out_dtype, x.device)
    if workspace is None:
        need = 0 if streaming else int(lib().bitrl_w8a8_workspace_bytes(M, K))
        workspace = torch.empty((max(need, 16),), dtype=torch.uint8, device=x.device)
    if not debug:
        _check(lib().bitrl_w8a8_forward(_ptr(wq), _ptr(scale), _ptr(x), M, K, N, _ptr(y), out_dtype, _ptr(workspace),
                                        workspace.numel(), _stream()), "bitrl_w8a8_forward")
        return y
    xq = torch.empty((M, K), dtype=torch.int8, device=x.device)
    a = torch.empty((M,), dtype=torch.float32, device=x.device)
    acc = torch.empty((M, N), dtype=torch.int32, device=x.device)
    _check(lib().bitrl_w8a8_forward_debug(_ptr(wq), _ptr(scale), _ptr(x), M, K, N, _ptr(y), out_dtype, _ptr(workspace),
                                          workspace.numel(), _ptr(xq), _ptr(a), _ptr(acc), _stream()),
           "bitrl_w8a8_forward_debug")
    return y, xq, a, acc


W8_MULTI_MAX_M = 2


class W8MultiCall:
    """Argument block of ``bitrl_w8a8_forward_multi``: ``count`` independent W8A8 layers (M <= 2), one launch.
    ``mats`` = list of (W_q int8 [N,K], scale fp32) pairs as returned by ``w8_quantize``.
    With ``int4=True``: ``bitrl_w4a8_forward_multi`` on (packed uint8 [N,K/2], scale) pairs from ``w4_quantize``."""

    def __init__(self, mats, xs, ys, out_dtype: int = OUT_BF16, int4: bool = False):
        assert len(mats) == len(xs) == len(ys) >= 1
        self.M = xs[0].shape[0]
        self.int4 = int4
        kmul = 2 if int4 else 1
        for (wq, scale), x, y in zip(mats, xs, ys):
            _dev(wq, torch.uint8 if int4 else torch.int8, "wq")
            _dev(scale, torch.float32, "scale")
            _dev(x, torch.bfloat16, "x")
            assert x.shape == (self.M, wq.shape[1] * kmul) and tuple(y.shape) == (self.M, wq.shape[0]) and y.is_contiguous()
            assert y.dtype == (torch.float32 if out_dtype == OUT_F32 else torch.bfloat16)
        self.keep = (list(mats), list(xs), list(ys))
        n = len(mats)
        self.count, self.out_dtype = n, out_dtype
        self.mats = (W8Matrix * n)(*[W8Matrix(wq.data_ptr(), sc.data_ptr(), wq.shape[0], wq.shape[1] * kmul) for wq, sc in mats])
        self.x = (_vp * n)(*[x.data_ptr() for x in xs])
        self.y = (_vp * n)(*[y.data_ptr() for y in ys])

    def run(self):
        fn = lib().bitrl_w4a8_forward_multi if self.int4 else lib().bitrl_w8a8_forward_multi
        _check(fn(self.count, self.mats, self.x, self.y, self.M, self.out_dtype, _stream()),
               "bitrl_w4a8_forward_multi" if self.int4 else "bitrl_w8a8_forward_multi")
        return self.keep[2]


def w4_quantize(W: torch.Tensor):
    """W CUDA fp32 [N,K] -> (packed uint8 [N,K/2], scale fp32 [2]; scale[0] is the scale)."""
    _dev(W, torch.float32, "W")
    N, K = W.shape
    packed = torch.empty((N, K // 2), dtype=torch.uint8, device=W.device)
    scale = torch.empty((2,), dtype=torch.float32, device=W.device)
    _check(lib().bitrl_w4_quantize(_ptr(W), N, K, _ptr(packed), _ptr(scale), _stream()), "bitrl_w4_quantize")
    return packed, scale


def w4a8_forward(packed: torch.Tensor, scale: torch.Tensor, x: torch.Tensor, out_dtype: int = OUT_BF16,
                 debug: bool = False, y: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
                 streaming: bool = False):
    """y = W4A8(x).  With debug=True returns (y, x_q, absmax, acc).  ``streaming``: as in w8a8_forward."""
    _dev(packed, torch.uint8, "packed")
    _dev(scale, torch.float32, "scale")
    _dev(x, torch.bfloat16, "x")
    M, K = x.shape
    N = packed.shape[0]
    if y is None:
        y = _out(M, N, out_dtype, x.device)
    if workspace is None:
        need = 0 if streaming else int(lib().bitrl_w4a8_workspace_bytes(M, K, N))
        workspace = torch.empty((max(need, 16),), dtype=torch.uint8, device=x.device)
    if not debug:
        _check(lib().bitrl_w4a8_forward(_ptr(packed), _ptr(scale), _ptr(x), M, K, N, _ptr(y), out_dtype, _ptr(workspace),
                                        workspace.numel(), _stream()), "bitrl_w4a8_forward")
        return y
    xq = torch.empty((M, K), dtype=torch.int8, device=x.device)
    a = torch.empty((M,), dtype=torch.float32, device=x.device)
    acc = torch.empty((M, N), dtype=torch.int32, device=x.device)
    _check(lib().bitrl_w4a8_forward_debug(_ptr(packed), _ptr(scale), _ptr(x), M, K, N, _ptr(y), out_dtype, _ptr(workspace),
                                          workspace.numel(), _ptr(xq), _ptr(a), _ptr(acc), _stream()),
           "bitrl_w4a8_forward_debug")
    return y, xq, a, acc


def heads_forward(h: torch.Tensor, heads):
    """h bf16 [B,d]; heads = list of (W1t [d,H1], b1, W2t [H1,H2], b2, W3t [H2,O], b3) CUDA fp32 tensors.
    Returns one fp32 [B,O] tensor per head."""
    _dev(h, torch.bfloat16, "h")
    B, d = h.shape
    H1, H2 = heads[0][0].shape[1], heads[0][2].shape[1]
    descs = (HeadDesc * len(heads))()
    outs = []
    for i, (W1t, b1, W2t, b2, W3t, b3) in enumerate(heads):
        for t in (W1t, b1, W2t, b2, W3t, b3):
            _dev(t, torch.float32, "head weights")
        assert W1t.shape == (d, H1) and W2t.shape == (H1, H2) and W3t.shape[0] == H2
        descs[i] = HeadDesc(W1t.data_ptr(), b1.data_ptr(), W2t.data_ptr(), b2.data_ptr(), W3t.data_ptr(), b3.data_ptr(),
                            W3t.shape[1])
        outs.append(torch.empty((B, W3t.shape[1]), dtype=torch.float32, device=h.device))
    optr = (_vp * len(heads))(*[o.data_ptr() for o in outs])
    _check(lib().bitrl_heads_forward(_ptr(h), B, d, H1, H2, descs, len(heads), optr, _stream()), "bitrl_heads_forward")
    return outs


def gae(rewards: torch.Tensor, values: torch.Tensor, dones: torch.Tensor, gamma: float = 0.99, lam: float = 0.95):
    """rewards, dones fp32 [T,E]; values fp32 [T+1,E].  Returns (advantages, returns), both [T,E]."""
    for t in (rewards, values, dones):
        _dev(t, torch.float32, "gae input")
    T, E = rewards.shape
    assert values.shape == (T + 1, E) and dones.shape == (T, E)
    adv, ret = torch.empty_like(rewards), torch.empty_like(rewards)
    _check(lib().bitrl_gae(_ptr(rewards), _ptr(values), _ptr(dones), T, E, gamma, lam, _ptr(adv), _ptr(ret), _stream()),
           "bitrl_gae")
    return adv, ret


def ppo_loss(logits, actions, old_logp, adv, values, returns, eps: float = 0.1, beta: float = 0.05):
    """Returns dict(summary fp32 [4] = {L_clip, entropy, policy_loss, value_loss}, terms [B,4], dlogits [B,A], dvalues [B])."""
    _dev(logits, torch.float32, "logits")
    _dev(actions, torch.int32, "actions")
    for t in (old_logp, adv, values, returns):
        _dev(t, torch.float32, "ppo input")
    B, A = logits.shape
    terms = torch.empty((B, 4), dtype=torch.float32, device=logits.device)
    dlogits = torch.empty_like(logits)
    dvalues = torch.empty((B,), dtype=torch.float32, device=logits.device)
    summary = torch.empty((4,), dtype=torch.float32, device=logits.device)
    _check(lib().bitrl_ppo_loss(_ptr(logits), _ptr(actions), _ptr(old_logp), _ptr(adv), _ptr(values), _ptr(returns), B, A,
                                eps, beta, _ptr(terms), _ptr(dlogits), _ptr(dvalues), _ptr(summary), _stream()),
           "bitrl_ppo_loss")
    return {"summary": summary, "terms": terms, "dlogits": dlogits, "dvalues": dvalues}


class Encoder:
    """Owns a ``bitrl_encoder_t`` over ``layers`` = list of (qkv, out, gateup, down) ``Linear`` tuples."""

    def __init__(self, layers, d: int, d_ff: int, n_heads: int, n_kv_heads: int):
        self.layers = [tuple(l) for l in layers]  # keeps the handles alive
        flat = [w.handle for l in self.layers for w in l]
        arr = (_vp * len(flat))(*flat)
        h = _vp()
        _check(lib().bitrl_encoder_create(arr, len(self.layers), d, d_ff, n_heads, n_kv_heads, ctypes.byref(h)),
               "bitrl_encoder_create")
        self.handle = h
        self.d, self.d_ff, self.n_heads, self.n_kv_heads = d, d_ff, n_heads, n_kv_heads

    def workspace_bytes(self, T: int) -> int:
        return int(lib().bitrl_encoder_workspace_bytes(self.handle, T))

    def forward(self, h_in: torch.Tensor, h_out: torch.Tensor | None = None,
                workspace: torch.Tensor | None = None) -> torch.Tensor:
        _dev(h_in, torch.bfloat16, "h_in")
        T = h_in.shape[0]
        if h_out is None:
            h_out = torch.empty_like(h_in)
        if workspace is None:
            workspace = torch.empty((self.workspace_bytes(T),), dtype=torch.uint8, device=h_in.device)
        _check(lib().bitrl_encoder_forward(self.handle, _ptr(h_in), T, _ptr(h_out), _ptr(workspace), workspace.numel(),
                                           _stream()), "bitrl_encoder_forward")
        return h_out

    def states_workspace_bytes(self, T: int, max_state_len: int) -> int:
        return int(lib().bitrl_encoder_states_workspace_bytes(self.handle, T, max_state_len))

    def forward_states(self, h_in: torch.Tensor, states, theta: float = ROPE_THETA, h_out: torch.Tensor | None = None,
                       pooled: torch.Tensor | None = None, want_pooled: bool = False,
                       workspace: torch.Tensor | None = None):
        """The encoder with real attention inside each state; returns h_out, or (h_out, pooled) when pooling."""
        _dev(h_in, torch.bfloat16, "h_in")
        T = h_in.shape[0]
        off, n_states, max_len = _states(states, T, h_in.device)
        if h_out is None:
            h_out = torch.empty_like(h_in)
        if pooled is None and want_pooled:
            pooled = torch.empty((n_states, self.d), dtype=torch.bfloat16, device=h_in.device)
        if workspace is None:
            workspace = torch.empty((self.states_workspace_bytes(T, max_len),), dtype=torch.uint8, device=h_in.device)
        _check(lib().bitrl_encoder_forward_states(self.handle, _ptr(h_in), T, _ptr(off), n_states, max_len,
                                                  float(theta), _ptr(h_out), _ptr(pooled), _ptr(workspace),
                                                  workspace.numel(), _stream()), "bitrl_encoder_forward_states")
        return (h_out, pooled) if pooled is not None else h_out

    def close(self):
        if getattr(self, "handle", None):
            lib().bitrl_encoder_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
