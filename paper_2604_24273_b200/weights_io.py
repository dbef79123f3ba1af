"""Flat file for the packed ternary weights of one matrix: what ``bitrl_pack_ternary`` produces, so that a frozen
backbone is ternarized once and loaded without its fp32 master weights afterwards.

Layout (little endian): 8-byte magic ``b"BITRL2B1"``, int32 N, int32 K, float32 gamma, 4 reserved bytes (zero), then
the canonical packed bytes ``uint8 [N][K/4]`` (code of k in bits ``2 (k % 4)`` of byte ``k / 4``, code = W_q + 1).
Host-side only: the functions take and return numpy arrays / CPU tensors; copying to the device and
``Linear(packed, gamma, N, K)`` stay with the caller.
"""
from __future__ import annotations

import struct
from pathlib import Path

import numpy as np

MAGIC = b"BITRL2B1"
HEADER = struct.Struct("<8siif4x")


def save_packed(path, packed, gamma, N: int, K: int) -> None:
    """packed: uint8 array-like [N, K/4] (numpy or CPU torch tensor); gamma: float or 1-element array."""
    arr = np.ascontiguousarray(np.asarray(packed), dtype=np.uint8)
    if K % 4 != 0 or arr.shape != (N, K // 4):
        raise ValueError(f"packed has shape {arr.shape}, expected ({N}, {K // 4})")
    if any(np.any(((arr >> shift) & 0x03) == 3) for shift in (0, 2, 4, 6)):
        raise ValueError("packed contains the 2-bit code 3, which no ternary weight has")
    g = np.float32(np.asarray(gamma, dtype=np.float32).reshape(-1)[0])
    with open(Path(path), "wb") as f:
        f.write(HEADER.pack(MAGIC, int(N), int(K), float(g)))
        f.write(arr.tobytes())


def load_packed(path):
    """Returns (packed uint8 [N, K/4], gamma np.float32, N, K); raises ValueError on a foreign or truncated file."""
    data = Path(path).read_bytes()
    if len(data) < HEADER.size:
        raise ValueError("file shorter than the header")
    magic, N, K, gamma = HEADER.unpack_from(data, 0)
    if magic != MAGIC:
        raise ValueError("not a packed-weight file (magic mismatch)")
    if N < 1 or K < 4 or K % 4 != 0:
        raise ValueError(f"bad shape in header: N={N}, K={K}")
    want = N * (K // 4)
    if len(data) - HEADER.size != want:
        raise ValueError(f"payload is {len(data) - HEADER.size} bytes, header says {want}")
    packed = np.frombuffer(data, dtype=np.uint8, count=want, offset=HEADER.size).reshape(N, K // 4).copy()
    return packed, np.float32(gamma), int(N), int(K)
