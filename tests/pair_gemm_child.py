"""Child process of test_gemm_paired_ctas_forced: with BITRL_GEMM_PAIR=1 in the environment every GEMM launch whose
shape allows it (M >= 1024, an even number of 128-row tiles) takes the paired-CTA kernel (tcgen05 cta_group::2).  Ragged
token counts, one and several k blocks, both output types; every stage must equal the oracle's."""
import sys

import numpy as np
import torch

import oracle as O
from paper_2604_24273_b200 import bitrl as B, inputs

O.build()
B.lib()
torch.cuda.set_device(0)
for M, K, N, out_dtype in [(1024, 128, 256, 1), (1061, 512, 512, 0), (1500, 640, 768, 1), (2048, 2560, 256, 1)]:
    W = inputs.master_weights(N, K, 77)
    Wq, g = O.ternarize(W.numpy())
    packed, gamma = B.pack_ternary(W.cuda())
    lin = B.Linear(packed, gamma, N, K)
    x = inputs.activations(M, K, 2600 + M)
    ref = O.bitlinear(inputs.bf16_bits(x), Wq, g)
    y, xq, a, acc = B.bitlinear_forward_debug(lin, x.cuda(), out_dtype)
    y2 = B.bitlinear_forward(lin, x.cuda(), out_dtype)
    torch.cuda.synchronize()
    B.poll_status()
    assert np.array_equal(xq.cpu().numpy(), ref["xq"]), (M, K, N)
    assert np.array_equal(acc.cpu().numpy(), ref["acc"]), (M, K, N)
    if out_dtype == B.OUT_F32:
        assert np.array_equal(y.cpu().numpy(), ref["y32"]), (M, K, N)
        assert np.array_equal(y2.cpu().numpy(), ref["y32"]), (M, K, N)
    else:
        assert np.array_equal(inputs.bf16_bits(y.cpu()), ref["ybf16"]), (M, K, N)
        assert np.array_equal(inputs.bf16_bits(y2.cpu()), ref["ybf16"]), (M, K, N)
print("paired-CTA GEMM parity ok")
sys.exit(0)
