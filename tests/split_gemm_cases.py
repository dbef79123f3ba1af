"""Shapes with few output tiles and a long K, where the GEMM launcher splits K, checked stage by stage against the
oracle.  Shared by the in-process test of the cluster form and the child process that runs the scratch form."""
import numpy as np

from paper_2604_24273_b200 import inputs

# (M, K, N, out_dtype): one and several token tiles, ragged tails, fewer 8-token units than k ranges (M = 17),
# k-block counts that leave uneven ranges (K = 640, 6912), many token tiles of one weight tile (M = 1000, 2000),
# both output types
CASES = [(17, 6912, 256, 1), (33, 2560, 128, 0), (40, 1024, 128, 1), (64, 1024, 256, 1), (64, 6912, 2560, 1),
         (64, 2560, 6912, 1), (100, 640, 128, 0), (128, 6912, 384, 1), (200, 2560, 256, 1), (256, 6912, 2560, 1),
         (257, 3840, 128, 0), (300, 6912, 128, 1), (32, 6912, 2560, 1), (32, 2560, 3840, 1), (2000, 2560, 128, 1),
         (1000, 640, 256, 0)]


def check_case(O, B, M, K, N, out_dtype, wseed=8100):
    """Whole layer with debug taps, the plain call, and the pre-quantized call with a residual: int8 codes, absmax and
    int32 sums bit-exact, outputs bit-identical to the oracle's three fp32 operations (+ RNE to bf16, + residual)."""
    W = inputs.master_weights(N, K, wseed + N + K)
    Wq, g = O.ternarize(W.numpy())
    packed, gamma = B.pack_ternary(W.cuda())
    lin = B.Linear(packed, gamma, N, K)
    x = inputs.activations(M, K, 8200 + M)
    ref = O.bitlinear(inputs.bf16_bits(x), Wq, g)
    y, xq, a, acc = B.bitlinear_forward_debug(lin, x.cuda(), out_dtype)
    y2 = B.bitlinear_forward(lin, x.cuda(), out_dtype)
    B.poll_status()
    assert np.array_equal(xq.cpu().numpy(), ref["xq"]), (M, K, N)
    assert np.array_equal(a.cpu().numpy(), ref["absmax"]), (M, K, N)
    assert np.array_equal(acc.cpu().numpy(), ref["acc"]), (M, K, N)
    if out_dtype == B.OUT_F32:
        assert np.array_equal(y.cpu().numpy(), ref["y32"]), (M, K, N)
        assert np.array_equal(y2.cpu().numpy(), ref["y32"]), (M, K, N)
        return
    assert np.array_equal(inputs.bf16_bits(y.cpu()), ref["ybf16"]), (M, K, N)
    assert np.array_equal(inputs.bf16_bits(y2.cpu()), ref["ybf16"]), (M, K, N)
    res = inputs.activations(M, N, 8300 + M, outliers=False)
    xq_g, a_g, rs_g = B.quant_act(x.cuda())
    yr = res.cuda()
    B.bitlinear_forward_q(lin, xq_g, a_g, rs_g, B.OUT_BF16, residual=yr, y=yr)  # in place, as the encoder calls it
    B.poll_status()
    assert np.array_equal(inputs.bf16_bits(yr.cpu()), O.residual_add(inputs.bf16_bits(res), ref["ybf16"])), (M, K, N)
