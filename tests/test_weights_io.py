"""The flat file for packed ternary weights: round trip on the oracle's packed bytes, and the refusals."""
import numpy as np
import pytest

from paper_2604_24273_b200 import inputs, weights_io


def test_round_trip_of_oracle_packed_bytes(oracle_mod, tmp_path):
    N, K = 128, 384
    W = inputs.master_weights(N, K, 77).numpy()
    Wq, g = oracle_mod.ternarize(W)
    packed = oracle_mod.pack(Wq)
    f = tmp_path / "w.bitrl"
    weights_io.save_packed(f, packed, g, N, K)
    assert f.stat().st_size == 24 + N * K // 4
    p2, g2, n2, k2 = weights_io.load_packed(f)
    assert (n2, k2) == (N, K) and g2 == np.float32(g) and g2.dtype == np.float32
    assert np.array_equal(p2, packed)
    assert np.array_equal(oracle_mod.unpack(p2, K), Wq)


def test_refusals(tmp_path):
    f = tmp_path / "w.bitrl"
    good = np.full((4, 2), 0x55, np.uint8)  # all-zero weights
    with pytest.raises(ValueError):
        weights_io.save_packed(f, good, 0.5, 4, 12)          # shape does not match N x K/4
    with pytest.raises(ValueError):
        weights_io.save_packed(f, np.full((4, 2), 0xFF, np.uint8), 0.5, 4, 8)  # code 3
    weights_io.save_packed(f, good, 0.5, 4, 8)
    raw = f.read_bytes()
    (tmp_path / "short").write_bytes(raw[:-1])
    with pytest.raises(ValueError):
        weights_io.load_packed(tmp_path / "short")
    (tmp_path / "magic").write_bytes(b"X" + raw[1:])
    with pytest.raises(ValueError):
        weights_io.load_packed(tmp_path / "magic")
    (tmp_path / "tiny").write_bytes(raw[:10])
    with pytest.raises(ValueError):
        weights_io.load_packed(tmp_path / "tiny")
