"""Split-K of the tensor-core GEMM inside a thread-block cluster (partial sums exchanged through distributed shared
memory) against the oracle, and the older scratch form kept behind its knob."""
import os
import subprocess
import sys
from pathlib import Path

import pytest
import torch

from split_gemm_cases import CASES, check_case

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_24273_b200 import bitrl

    bitrl.lib()
    torch.cuda.set_device(0)
    return bitrl


@pytest.mark.parametrize("M,K,N,out_dtype", CASES)
def test_cluster_split_case(oracle_mod, B, M, K, N, out_dtype):
    check_case(oracle_mod, B, M, K, N, out_dtype)


def test_cases_cover_the_cluster_form(B):
    """The launcher really takes the cluster form on these shapes, with several cluster sizes and both tile widths."""
    plans = {(M, K, N): B.gemm_plan(M, K, N) for M, K, N, _ in CASES}
    cluster = {k: p for k, p in plans.items() if p[2] == B.GEMM_SPLIT_CLUSTER}
    assert len(cluster) >= 10, plans
    assert len({p[1] for p in cluster.values()}) >= 4, plans       # distinct cluster sizes
    assert {p[0] for p in cluster.values()} == {64, 128}, plans    # both token-tile widths
    for tok, splits, _ in cluster.values():
        assert 2 <= splits <= 8
    # the batched-state layers of the block: one launch, no scratch, no finishing kernel
    for M, K, N in ((64, 6912, 2560), (64, 2560, 6912), (32, 6912, 2560)):
        assert plans[(M, K, N)][2] == B.GEMM_SPLIT_CLUSTER, plans[(M, K, N)]
    # large launches are untouched
    assert B.gemm_plan(4096, 2560, 6912)[2] == B.GEMM_PAIRED
    assert B.gemm_plan(2048, 2560, 6912)[1] == 1


def test_cluster_split_is_one_launch(B):
    from paper_2604_24273_b200 import inputs

    M, K, N = 64, 6912, 2560
    lin = B.Linear.from_master(inputs.master_weights(N, K, 8400).cuda())
    xq, a, rs = B.quant_act(inputs.activations(M, K, 8401).cuda())
    n0 = B.launch_count()
    B.bitlinear_forward_q(lin, xq, a, rs, B.OUT_BF16)
    assert B.launch_count() - n0 == 1
    B.poll_status()


def test_scratch_split_form_still_exact(B):
    root = Path(__file__).resolve().parent.parent
    env = dict(os.environ, BITRL_GEMM_CLSK="0", PYTHONPATH=str(root))
    r = subprocess.run([sys.executable, str(root / "tests" / "scratch_split_child.py")], env=env, cwd=str(root),
                       capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    assert "scratch split-K parity ok" in r.stdout


def test_random_shapes_sampled_rows(oracle_mod, B):
    """40 seeded random (M, K, N) over the range where the launcher switches between the unsplit, cluster and scratch
    forms: int32 sums of 12 sampled token rows per case against the oracle, and two runs bit-identical (the exchange
    inside a cluster must not depend on which CTA finishes first)."""
    import random

    import numpy as np

    from paper_2604_24273_b200 import inputs

    rnd = random.Random(20240607)
    layers, kinds = {}, set()
    for case in range(40):
        K = rnd.choice([640, 1024, 2560, 3840, 6912])
        N = rnd.choice([128, 256, 384, 2560])
        M = rnd.choice([5, 9, 17, 31, 33, 40, 63, 65, 100, 127, 129, 200, 256, 300, 511, 700, 1000])
        if (N, K) not in layers:
            W = inputs.master_weights(N, K, 8800 + N + K)
            layers[(N, K)] = (oracle_mod.ternarize(W.numpy())[0], B.Linear.from_master(W.cuda()))
        Wq, lin = layers[(N, K)]
        x = inputs.activations(M, K, 8900 + case)
        res = inputs.activations(M, N, 9000 + case, outliers=False).cuda()
        xq, a, rs = B.quant_act(x.cuda())
        y1, acc1 = B.bitlinear_forward_q(lin, xq, a, rs, B.OUT_BF16, residual=res, want_acc=True)
        y2, acc2 = B.bitlinear_forward_q(lin, xq, a, rs, B.OUT_BF16, residual=res, want_acc=True)
        B.poll_status()
        assert torch.equal(acc1, acc2) and torch.equal(y1, y2), (M, K, N)
        rows = np.unique(np.concatenate([[0, M - 1], np.random.default_rng(case).integers(0, M, 10)]))
        assert np.array_equal(acc1.cpu().numpy()[rows], oracle_mod.contract(xq.cpu().numpy()[rows], Wq)), (M, K, N)
        kinds.add(B.gemm_plan(M, K, N)[2])
    assert B.GEMM_SPLIT_CLUSTER in kinds and B.GEMM_SINGLE in kinds
