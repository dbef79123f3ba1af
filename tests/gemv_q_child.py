"""Child process of test_forward_q_streaming_kernel_forced: with BITRL_GEMV_Q_MAX_M=16 in the environment every
pre-quantized call with M <= 16 takes the streaming kernel (by default only M <= 4 does).  Integer sums and the
residual epilogue must equal the oracle's."""
import sys

import numpy as np
import torch

import oracle as O
from paper_2604_24273_b200 import bitrl as B, inputs

O.build()
B.lib()
torch.cuda.set_device(0)
for M, K, N in [(5, 256, 384), (8, 2560, 3840), (13, 6912, 2560), (16, 2560, 2560)]:
    W = inputs.master_weights(N, K, 8500 + M)
    Wq, g = O.ternarize(W.numpy())
    lin = B.Linear.from_master(W.cuda())
    x = inputs.activations(M, K, 8600 + M)
    res = inputs.activations(M, N, 8700 + M, outliers=False)
    ref = O.bitlinear(inputs.bf16_bits(x), Wq, g)
    xq, a, rs = B.quant_act(x.cuda())
    n0 = B.launch_count()
    y, acc = B.bitlinear_forward_q(lin, xq, a, rs, B.OUT_BF16, residual=res.cuda(), want_acc=True)
    assert B.launch_count() - n0 == 1
    B.poll_status()
    assert np.array_equal(acc.cpu().numpy(), ref["acc"]), (M, K, N)
    assert np.array_equal(inputs.bf16_bits(y.cpu()), O.residual_add(inputs.bf16_bits(res), ref["ybf16"])), (M, K, N)
print("streaming forward_q parity ok")
sys.exit(0)
