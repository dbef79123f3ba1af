"""GPU parity of the W8A8 layer (int8 weights with one absmax scale per matrix, the higher-precision critic of the
paper's ablations) through the C ABI against the CPU oracle: codes, int8 activations and int32 sums bit-exact, rescaled
outputs within 1e-3 (fp32) / 8e-3 (bf16) of the fp64 reference - and in fact equal bit for bit, both sides doing the
same int32 -> fp32 conversion and the same three fp32 operations."""
import numpy as np
import pytest
import torch

from paper_2604_24273_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_24273_b200 import bitrl

    bitrl.lib()
    torch.cuda.set_device(0)
    return bitrl


def bits_to_f64(bits):
    return (np.asarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rel_err(y, y64):
    denom = np.where(y64 == 0, 1.0, np.abs(y64))
    return float((np.abs(np.asarray(y, np.float64) - y64) / denom).max())


_cache = {}


def weights(oracle_mod, B, N, K, seed):
    if (N, K, seed) not in _cache:
        W = inputs.master_weights(N, K, seed)
        Wq, scale = oracle_mod.w8_quantize(W.numpy())
        wq_gpu, scale_gpu = B.w8_quantize(W.cuda())
        B.poll_status()
        assert np.array_equal(wq_gpu.cpu().numpy(), Wq), "int8 weight codes differ from the oracle"
        assert np.float32(scale_gpu.cpu().numpy()[0]) == scale
        _cache[(N, K, seed)] = (Wq, scale, wq_gpu, scale_gpu)
    return _cache[(N, K, seed)]


@pytest.mark.parametrize("M", [1, 2, 3, 8, 13, 16, 17, 64, 300, 513])
@pytest.mark.parametrize("K,N,seed,out_dtype", [(256, 384, 9200, 1), (640, 128, 9201, 0), (2560, 2560, 9202, 1)])
@pytest.mark.parametrize("streaming", [False, True])
def test_w8a8_full(oracle_mod, B, M, K, N, seed, out_dtype, streaming):
    """streaming: without a workspace, so that the streaming kernel also serves 5 <= M <= 16 (with one, those take the
    quantizer + tensor-core GEMM)."""
    if streaming and not 4 < M <= 16:
        pytest.skip("same path as without the flag")
    Wq, scale, wq_gpu, scale_gpu = weights(oracle_mod, B, N, K, seed)
    x = inputs.activations(M, K, 9300 + M)
    ref = oracle_mod.bitlinear(inputs.bf16_bits(x), Wq, scale)
    n0 = B.launch_count()
    y, xq, a, acc = B.w8a8_forward(wq_gpu, scale_gpu, x.cuda(), out_dtype, debug=True, streaming=streaming)
    assert (B.launch_count() - n0 == 1) == (M <= 4 or streaming)
    y2 = B.w8a8_forward(wq_gpu, scale_gpu, x.cuda(), out_dtype, streaming=streaming)
    B.poll_status()
    assert np.array_equal(xq.cpu().numpy(), ref["xq"])
    assert np.array_equal(a.cpu().numpy(), ref["absmax"])
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    if out_dtype == B.OUT_F32:
        assert rel_err(y.cpu().numpy(), ref["y64"]) <= 1e-3
        assert np.array_equal(y.cpu().numpy(), ref["y32"]) and torch.equal(y, y2)
    else:
        yb = inputs.bf16_bits(y.cpu())
        assert rel_err(bits_to_f64(yb), ref["y64"]) <= 8e-3
        assert np.array_equal(yb, ref["ybf16"]) and torch.equal(y, y2)


@pytest.mark.parametrize("M,K,N,seed,out_dtype", [(2048, 128, 256, 9210, 1), (2085, 640, 512, 9211, 0),
                                                   (2300, 2560, 768, 9212, 1)])
def test_w8a8_paired_cta_shapes_full(oracle_mod, B, M, K, N, seed, out_dtype):
    """M >= 2048 with an even number of 128-row tiles: the paired-CTA kernel (tcgen05 cta_group::2); ragged token counts,
    one and several k blocks, every stage against the oracle."""
    test_w8a8_full(oracle_mod, B, M, K, N, seed, out_dtype, False)


@pytest.mark.parametrize("M,K,N,seed,out_dtype", [(17, 6912, 256, 9220, 1), (64, 6912, 2560, 9221, 1), (100, 640, 128, 9222, 0),
                                                   (200, 2560, 256, 9223, 1), (256, 6912, 2560, 9221, 0)])
def test_w8a8_cluster_split_shapes_full(oracle_mod, B, M, K, N, seed, out_dtype):
    """Few tiles and a long K: the k ranges of a tile go to the CTAs of a cluster (partial sums exchanged through
    distributed shared memory); one launch after the quantizer, every stage against the oracle."""
    x = inputs.activations(M, K, 9300 + M).cuda()
    Wq, scale, wq_gpu, scale_gpu = weights(oracle_mod, B, N, K, seed)
    n0 = B.launch_count()
    B.w8a8_forward(wq_gpu, scale_gpu, x, out_dtype)
    assert B.launch_count() - n0 == 2
    test_w8a8_full(oracle_mod, B, M, K, N, seed, out_dtype, False)


@pytest.mark.parametrize("M", [1, 2, 4])
def test_w8a8_long_rows_both_forms(oracle_mod, B, M):
    """K = 6912 > 4096: with a workspace even M <= 4 takes quantizer + GEMM (cluster split-K); without one the streaming
    kernel (one, two or four rows per warp).  Same bits, both equal to the oracle."""
    K, N = 6912, 2560
    Wq, scale, wq_gpu, scale_gpu = weights(oracle_mod, B, N, K, 9221)
    x = inputs.activations(M, K, 9350 + M)
    ref = oracle_mod.bitlinear(inputs.bf16_bits(x), Wq, scale)
    for streaming in (False, True):
        n0 = B.launch_count()
        y, xq, a, acc = B.w8a8_forward(wq_gpu, scale_gpu, x.cuda(), B.OUT_BF16, debug=True, streaming=streaming)
        assert B.launch_count() - n0 == (1 if streaming else 2)
        B.poll_status()
        assert np.array_equal(xq.cpu().numpy(), ref["xq"]) and np.array_equal(acc.cpu().numpy(), ref["acc"])
        assert np.array_equal(inputs.bf16_bits(y.cpu()), ref["ybf16"])


def test_w8a8_m4096_sampled(oracle_mod, B):
    """The batched-state shape at full size (M = 4096, 2560 -> 6912): sampled outputs one by one."""
    K, N, M = 2560, 6912, 4096
    Wq, scale, wq_gpu, scale_gpu = weights(oracle_mod, B, N, K, 9203)
    x = inputs.activations(M, K, 9400)
    y, xq, a, acc = B.w8a8_forward(wq_gpu, scale_gpu, x.cuda(), B.OUT_BF16, debug=True)
    B.poll_status()
    xq_o, a_o = oracle_mod.quant_act(inputs.bf16_bits(x))
    assert np.array_equal(xq.cpu().numpy(), xq_o) and np.array_equal(a.cpu().numpy(), a_o)
    rng = np.random.default_rng(5)
    ms = np.concatenate([[0, 255, 256, 4095], rng.integers(0, M, 500)])
    ns = np.concatenate([[0, 127, 128, 6911], rng.integers(0, N, 500)])
    want = oracle_mod.contract_pairs(xq_o, Wq, ms, ns)
    assert np.array_equal(acc.cpu().numpy()[ms, ns], want)
    y64 = want.astype(np.float64) * float(scale) * a_o[ms].astype(np.float64) / 127.0
    assert rel_err(bits_to_f64(inputs.bf16_bits(y.cpu())[ms, ns]), y64) <= 8e-3


@pytest.mark.parametrize("M,out_dtype", [(1, 1), (2, 0), (2, 1)])
def test_w8a8_forward_multi_matches_oracle_and_single_calls(oracle_mod, B, M, out_dtype):
    """Several independent W8A8 layers in one launch (rows per ring slot: 12 at K = 2560, 4 at 6912, 25 at 1280, a ragged
    last slot everywhere): bit-identical to the oracle and to separate calls."""
    specs = [(384, 256, 9200), (2560, 2560, 9202), (2560, 6912, 9204), (128, 640, 9201), (6912, 2560, 9203), (640, 1280, 9205)]
    xs_cpu = {K: inputs.activations(M, K, 9800 + K + M) for K in {k for _, k, _ in specs}}
    xs_gpu = {K: v.cuda() for K, v in xs_cpu.items()}
    mats, xs, ys, refs = [], [], [], []
    dt = torch.float32 if out_dtype == 0 else torch.bfloat16
    for N, K, seed in specs:
        Wq, scale, wq_gpu, scale_gpu = weights(oracle_mod, B, N, K, seed)
        mats.append((wq_gpu, scale_gpu))
        xs.append(xs_gpu[K])
        ys.append(torch.full((M, N), 7.0, dtype=dt, device="cuda"))
        refs.append(oracle_mod.bitlinear(inputs.bf16_bits(xs_cpu[K]), Wq, scale))
    call = B.W8MultiCall(mats, xs, ys, out_dtype)
    call.run()
    call.run()
    B.poll_status()
    for (wq_gpu, scale_gpu), x, y, ref in zip(mats, xs, ys, refs):
        assert torch.equal(B.w8a8_forward(wq_gpu, scale_gpu, x, out_dtype), y)
        if out_dtype == 0:
            assert np.array_equal(y.cpu().numpy(), ref["y32"])
        else:
            yb = inputs.bf16_bits(y.cpu())
            assert np.array_equal(yb, ref["ybf16"])
            assert rel_err(bits_to_f64(yb), ref["y64"]) <= 8e-3
    L = B.lib()
    assert L.bitrl_w8a8_forward_multi(1, call.mats, call.x, call.y, 3, out_dtype, None) == B.ERR_SHAPE
    assert L.bitrl_w8a8_forward_multi(0, call.mats, call.x, call.y, M, out_dtype, None) == B.ERR_SHAPE


def test_w8a8_argument_errors(oracle_mod, B):
    L = B.lib()
    Wq, scale, wq_gpu, scale_gpu = weights(oracle_mod, B, 384, 256, 9200)
    x = inputs.activations(20, 256, 1).cuda()
    y = torch.empty((20, 384), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty((L.bitrl_w8a8_workspace_bytes(20, 256),), dtype=torch.uint8, device="cuda")
    assert L.bitrl_w8a8_workspace_bytes(4, 256) == 0  # the streaming kernel needs none
    call = lambda M, K, N, wsb: L.bitrl_w8a8_forward(wq_gpu.data_ptr(), scale_gpu.data_ptr(), x.data_ptr(), M, K, N,
                                                     y.data_ptr(), 1, ws.data_ptr(), wsb, None)
    assert call(0, 256, 384, ws.numel()) == B.ERR_SHAPE
    assert call(20, 200, 384, ws.numel()) == B.ERR_SHAPE
    assert call(20, 256, 384, 16) == B.ERR_WORKSPACE
    assert call(20, 256, 384, ws.numel()) == B.OK
    assert call(4, 256, 384, 0) == B.OK
    B.poll_status()
