"""GPU parity of the W4A8 layer (int4 weights, one absmax scale per matrix: the INT4 critic of the paper's ablations)
through the C ABI against the CPU oracle: packed codes, int8 activations and int32 sums bit-exact, rescaled outputs
within 1e-3 (fp32) / 8e-3 (bf16) of the fp64 reference and equal bit for bit to the oracle's fp32 / bf16 results."""
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
        Wq, scale = oracle_mod.w4_quantize(W.numpy())
        packed_gpu, scale_gpu = B.w4_quantize(W.cuda())
        B.poll_status()
        assert np.array_equal(packed_gpu.cpu().numpy(), oracle_mod.w4_pack(Wq)), "packed int4 codes differ from the oracle"
        assert np.float32(scale_gpu.cpu().numpy()[0]) == scale
        _cache[(N, K, seed)] = (Wq, scale, packed_gpu, scale_gpu)
    return _cache[(N, K, seed)]


@pytest.mark.parametrize("M", [1, 2, 3, 8, 13, 16, 17, 64, 300])
@pytest.mark.parametrize("K,N,seed,out_dtype", [(256, 384, 9500, 1), (640, 128, 9501, 0), (2560, 2560, 9502, 1)])
@pytest.mark.parametrize("streaming", [False, True])
def test_w4a8_full(oracle_mod, B, M, K, N, seed, out_dtype, streaming):
    """streaming: without a workspace, so that the streaming kernel also serves 5 <= M <= 16 (with one, those take the
    quantizer + expansion + tensor-core GEMM)."""
    if streaming and not 4 < M <= 16:
        pytest.skip("same path as without the flag")
    Wq, scale, packed_gpu, scale_gpu = weights(oracle_mod, B, N, K, seed)
    x = inputs.activations(M, K, 9600 + M)
    ref = oracle_mod.bitlinear(inputs.bf16_bits(x), Wq, scale)
    n0 = B.launch_count()
    y, xq, a, acc = B.w4a8_forward(packed_gpu, scale_gpu, x.cuda(), out_dtype, debug=True, streaming=streaming)
    assert (B.launch_count() - n0 == 1) == (M <= 4 or streaming)
    y2 = B.w4a8_forward(packed_gpu, scale_gpu, x.cuda(), out_dtype, streaming=streaming)
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


@pytest.mark.parametrize("M", [1, 2, 4])
def test_w4a8_long_rows_both_forms(oracle_mod, B, M):
    """K = 6912 with few rows: the streaming kernel with one (M = 1) or four rows per warp, with and without a workspace."""
    K, N = 6912, 256
    Wq, scale, packed_gpu, scale_gpu = weights(oracle_mod, B, N, K, 9520)
    x = inputs.activations(M, K, 9650 + M)
    ref = oracle_mod.bitlinear(inputs.bf16_bits(x), Wq, scale)
    for streaming in (False, True):
        n0 = B.launch_count()
        y, xq, a, acc = B.w4a8_forward(packed_gpu, scale_gpu, x.cuda(), B.OUT_BF16, debug=True, streaming=streaming)
        assert B.launch_count() - n0 == 1
        B.poll_status()
        assert np.array_equal(xq.cpu().numpy(), ref["xq"]) and np.array_equal(acc.cpu().numpy(), ref["acc"])
        assert np.array_equal(inputs.bf16_bits(y.cpu()), ref["ybf16"])


@pytest.mark.parametrize("M,out_dtype", [(1, 1), (2, 0), (2, 1)])
def test_w4a8_forward_multi_matches_oracle_and_single_calls(oracle_mod, B, M, out_dtype):
    """Several independent W4A8 layers in one launch: bit-identical to the oracle and to separate calls."""
    specs = [(384, 256, 9500), (128, 640, 9501), (2560, 2560, 9502), (384, 256, 9500), (2560, 6912, 9504)]
    xs_cpu = {K: inputs.activations(M, K, 9900 + K + M) for K in {k for _, k, _ in specs}}
    xs_gpu = {K: v.cuda() for K, v in xs_cpu.items()}
    mats, xs, ys, refs = [], [], [], []
    dt = torch.float32 if out_dtype == 0 else torch.bfloat16
    for N, K, seed in specs:
        Wq, scale, packed_gpu, scale_gpu = weights(oracle_mod, B, N, K, seed)
        mats.append((packed_gpu, scale_gpu))
        xs.append(xs_gpu[K])
        ys.append(torch.full((M, N), 7.0, dtype=dt, device="cuda"))
        refs.append(oracle_mod.bitlinear(inputs.bf16_bits(xs_cpu[K]), Wq, scale))
    call = B.W8MultiCall(mats, xs, ys, out_dtype, int4=True)
    call.run()
    call.run()
    B.poll_status()
    for (packed_gpu, scale_gpu), x, y, ref in zip(mats, xs, ys, refs):
        assert torch.equal(B.w4a8_forward(packed_gpu, scale_gpu, x, out_dtype), y)
        if out_dtype == 0:
            assert np.array_equal(y.cpu().numpy(), ref["y32"])
        else:
            yb = inputs.bf16_bits(y.cpu())
            assert np.array_equal(yb, ref["ybf16"])
            assert rel_err(bits_to_f64(yb), ref["y64"]) <= 8e-3


def test_w4a8_argument_errors(oracle_mod, B):
    L = B.lib()
    Wq, scale, packed_gpu, scale_gpu = weights(oracle_mod, B, 384, 256, 9500)
    x = inputs.activations(20, 256, 1).cuda()
    y = torch.empty((20, 384), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty((L.bitrl_w4a8_workspace_bytes(20, 256, 384),), dtype=torch.uint8, device="cuda")
    assert L.bitrl_w4a8_workspace_bytes(4, 256, 384) == 0
    call = lambda M, K, N, wsb: L.bitrl_w4a8_forward(packed_gpu.data_ptr(), scale_gpu.data_ptr(), x.data_ptr(), M, K, N,
                                                     y.data_ptr(), 1, ws.data_ptr(), wsb, None)
    assert call(0, 256, 384, ws.numel()) == B.ERR_SHAPE
    assert call(20, 256, 300, ws.numel()) == B.ERR_SHAPE
    assert call(20, 256, 384, 16) == B.ERR_WORKSPACE
    assert call(20, 256, 384, ws.numel()) == B.OK
    assert call(4, 256, 384, 0) == B.OK
    B.poll_status()
