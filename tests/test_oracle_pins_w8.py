"""Pins of the oracle's eight-bit weight quantizer and the W8A8 layer built from it, against the definition evaluated
in fp64, error bounds, a special case that reduces to the ternary layer, and library integer / fp64 matmuls."""
import numpy as np
import torch

import oracle
from paper_2604_24273_b200 import inputs


def test_w8_codes_follow_the_definition_and_the_error_bound():
    """absmax element -> +-127; |W - q*scale| <= scale/2; codes equal rint(127 W / max|W|) evaluated in fp64 away from
    ties.  Catches a scale of max/128, truncation instead of rounding, a per-row scale."""
    W = inputs.master_weights(96, 160, 9100).numpy()
    Wq, scale = oracle.w8_quantize(W)
    a = np.abs(W).max()
    assert Wq.dtype == np.int8 and np.abs(Wq.astype(np.int32)).max() == 127
    i = np.unravel_index(np.abs(W).argmax(), W.shape)
    assert abs(int(Wq[i])) == 127 and np.sign(Wq[i]) == np.sign(W[i])
    assert scale == np.float32(a) / np.float32(127.0)
    t = W.astype(np.float64) * 127.0 / float(a)
    away = np.abs(t - np.floor(t) - 0.5) > 1e-4
    assert away.mean() > 0.99 and np.array_equal(Wq[away], np.rint(t[away]).astype(np.int8))
    assert np.all(np.abs(W.astype(np.float64) - Wq.astype(np.float64) * float(scale)) <= float(scale) * 0.5 * (1 + 1e-5))
    Wz, sz = oracle.w8_quantize(np.zeros((4, 8), np.float32))
    assert not Wz.any() and np.isfinite(sz)


def test_w8_on_a_scaled_ternary_matrix_is_127_times_the_ternary_layer():
    """W = c*T with T in {-1,0,1}: codes are 127*T, so the int32 sums are 127 times the ternary ones and the outputs
    agree with the ternary layer with gamma = c up to fp32 rounding of the scales."""
    rng = np.random.default_rng(1)
    T = rng.integers(-1, 2, size=(48, 128)).astype(np.int8)
    c = np.float32(0.0173)
    Wq, scale = oracle.w8_quantize(T.astype(np.float32) * c)
    assert np.array_equal(Wq.astype(np.int32), 127 * T.astype(np.int32))
    x = inputs.bf16_bits(inputs.activations(5, 128, 9101))
    r8, rt = oracle.bitlinear(x, Wq, scale), oracle.bitlinear(x, T, c)
    assert np.array_equal(r8["acc"], 127 * rt["acc"])
    np.testing.assert_allclose(r8["y64"], rt["y64"], rtol=1e-6)


def test_w8a8_layer_against_fp64_and_integer_library_matmuls():
    W = inputs.master_weights(64, 256, 9102).numpy()
    Wq, scale = oracle.w8_quantize(W)
    x = inputs.activations(7, 256, 9103)
    ref = oracle.bitlinear(inputs.bf16_bits(x), Wq, scale)
    xq, a = ref["xq"], ref["absmax"]
    acc_t = torch.from_numpy(xq.astype(np.int32)) @ torch.from_numpy(Wq.astype(np.int32)).T
    assert np.array_equal(ref["acc"], acc_t.numpy())
    dense = (xq.astype(np.float64) * (a.astype(np.float64)[:, None] / 127.0)) @ (Wq.astype(np.float64) * float(scale)).T
    np.testing.assert_allclose(ref["y64"], dense, rtol=1e-12, atol=1e-300)
    # the quantized layer approximates the fp64 layer on the unquantized operands (coarse sanity: both int8 grids)
    full = x.to(torch.float64).numpy() @ W.astype(np.float64).T
    assert np.linalg.norm(ref["y64"] - full) / np.linalg.norm(full) < 0.05
    # fp32 / bf16 outputs are roundings of the same product, also when |acc| exceeds 2^24
    big = np.full((1, 256), 127, np.int8)
    accb = oracle.contract(big, np.full((3, 256), 127, np.int8))
    assert accb[0, 0] == 127 * 127 * 256


def test_w4_codes_definition_error_bound_and_packing():
    """absmax element -> +-7, codes in [-8, 7] and equal to rint(7 W / max|W|) in fp64 away from ties, error at most
    half a step; the packed byte holds k even in the low nibble as q + 8 (checked against numpy bit operations)."""
    W = inputs.master_weights(64, 96, 9110).numpy()
    Wq, scale = oracle.w4_quantize(W)
    a = np.abs(W).max()
    assert Wq.min() >= -8 and Wq.max() <= 7 and np.abs(Wq.astype(np.int32)).max() == 7
    assert scale == np.float32(a) / np.float32(7.0)
    t = W.astype(np.float64) * 7.0 / float(a)
    away = np.abs(t - np.floor(t) - 0.5) > 1e-4
    assert away.mean() > 0.99 and np.array_equal(Wq[away], np.rint(t[away]).astype(np.int8))
    assert np.all(np.abs(W.astype(np.float64) - Wq.astype(np.float64) * float(scale)) <= float(scale) * 0.5 * (1 + 1e-5))
    packed = oracle.w4_pack(Wq)
    assert packed.shape == (64, 48)
    lo = (packed & 0x0F).astype(np.int32) - 8
    hi = (packed >> 4).astype(np.int32) - 8
    assert np.array_equal(lo, Wq[:, 0::2]) and np.array_equal(hi, Wq[:, 1::2])


def test_w4a8_layer_against_library_matmuls():
    W = inputs.master_weights(32, 128, 9111).numpy()
    Wq, scale = oracle.w4_quantize(W)
    x = inputs.activations(3, 128, 9112)
    ref = oracle.bitlinear(inputs.bf16_bits(x), Wq, scale)
    acc_t = torch.from_numpy(ref["xq"].astype(np.int32)) @ torch.from_numpy(Wq.astype(np.int32)).T
    assert np.array_equal(ref["acc"], acc_t.numpy())
    dense = (ref["xq"].astype(np.float64) * (ref["absmax"].astype(np.float64)[:, None] / 127.0)) @ (Wq.astype(np.float64) * float(scale)).T
    np.testing.assert_allclose(ref["y64"], dense, rtol=1e-12, atol=1e-300)
