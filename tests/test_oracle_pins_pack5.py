"""Pins of the oracle's five-weights-per-byte packing (`pack5` / `unpack5`), none of which goes through the oracle's
own code for the thing checked: hand-worked bytes, Python's own base-3 integer parser on every one of the 3^5 digit
strings, the byte-count rule, the padding rule, and the size ratio against the 2-bit format."""
import itertools
import json
from pathlib import Path

import numpy as np

GOLDEN = json.loads((Path(__file__).parent / "golden" / "pack5_worked_example.json").read_text())


def test_pack5_golden_bytes(oracle_mod):
    Wq = np.array(GOLDEN["W_q"], np.int8)
    assert oracle_mod.pack5(Wq).tolist() == GOLDEN["packed5"]
    sp = GOLDEN["special_bytes"]
    for value, key in ((0, "all_zero_weights"), (1, "all_plus_one"), (-1, "all_minus_one")):
        assert oracle_mod.pack5(np.full((1, 5), value, np.int8)).tolist() == [[sp[key]]]


def test_pack5_is_the_base3_number_of_every_digit_string(oracle_mod):
    """All 243 combinations of five weights: the byte equals int(<digits, most significant first>, 3) as parsed by
    Python, the bytes are exactly 0..242 once each, and unpack5 inverts them."""
    combos = np.array(list(itertools.product((-1, 0, 1), repeat=5)), np.int8)  # [243, 5]
    packed = oracle_mod.pack5(combos)
    assert packed.shape == (243, 1)
    want = [int("".join(str(int(w) + 1) for w in row[::-1]), 3) for row in combos]
    assert packed[:, 0].tolist() == want
    assert sorted(want) == list(range(243))
    assert np.array_equal(oracle_mod.unpack5(packed, 5), combos)


def test_pack5_byte_count_padding_and_roundtrip(oracle_mod):
    rng = np.random.default_rng(5)
    for K in (1, 4, 5, 6, 7, 128, 2560, 6912):
        Wq = rng.integers(-1, 2, (3, K)).astype(np.int8)
        p = oracle_mod.pack5(Wq)
        assert p.shape == (3, -(-K // 5))  # ceil(K/5) bytes per row
        assert np.array_equal(oracle_mod.unpack5(p, K), Wq)
        # missing positions of the last byte are zero weights: packing the row extended with zeros gives the same bytes
        Kp = 5 * p.shape[1]
        ext = np.zeros((3, Kp), np.int8)
        ext[:, :K] = Wq
        assert np.array_equal(oracle_mod.pack5(ext), p)
        assert p.max() <= 242
    # 2560 weights take 512 bytes: 0.8 of the 640 bytes of the 2-bit format, 1.6 bits per weight
    assert oracle_mod.pack5(np.zeros((1, 2560), np.int8)).shape[1] * 10 == oracle_mod.pack(np.zeros((1, 2560), np.int8)).shape[1] * 8


def test_pack5_digit_positions(oracle_mod):
    """One non-zero weight at position i of byte j moves exactly that byte by +-3^i from the all-zero byte 121."""
    K = 12
    for k in range(K):
        for w in (-1, 1):
            Wq = np.zeros((1, K), np.int8)
            Wq[0, k] = w
            p = oracle_mod.pack5(Wq)[0].astype(int)
            want = [121, 121, 121]
            want[k // 5] += w * 3 ** (k % 5)
            assert p.tolist() == want
