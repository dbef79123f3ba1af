"""Child process of test_scratch_split_form_still_exact: with BITRL_GEMM_CLSK=0 in the environment (the knob is read once
per process) split launches go through the int32 scratch and the finishing kernel instead of a cluster."""
import sys

import torch

import oracle as O
from paper_2604_24273_b200 import bitrl as B
from split_gemm_cases import CASES, check_case

O.build()
B.lib()
torch.cuda.set_device(0)
kinds = set()
for M, K, N, out_dtype in CASES:
    kinds.add(B.gemm_plan(M, K, N)[2])
    check_case(O, B, M, K, N, out_dtype)
assert B.GEMM_SPLIT_CLUSTER not in kinds and B.GEMM_SPLIT_SCRATCH in kinds, kinds
print("scratch split-K parity ok")
sys.exit(0)
