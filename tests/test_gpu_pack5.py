"""GPU parity of the five-weights-per-byte path (1.6 bits per weight, decoded through a lookup table): packed bytes
equal to the oracle's base-3 packing byte for byte, and the grouped streaming kernel on that format bit-identical to the
oracle's outputs and to the 2-bit kernel's, at M = 1 and 2."""
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


_cache = {}


def layer5(oracle_mod, B, N, K, seed):
    if (N, K, seed) not in _cache:
        W = inputs.master_weights(N, K, seed)
        Wq, g = oracle_mod.ternarize(W.numpy())
        packed, gamma = B.pack_ternary(W.cuda())
        p5 = B.pack5(packed, N, K)
        B.poll_status()
        assert np.array_equal(p5.cpu().numpy(), oracle_mod.pack5(Wq)), "base-3 bytes differ from the oracle"
        _cache[(N, K, seed)] = (Wq, g, B.Linear5(p5, gamma, N, K), B.Linear(packed, gamma, N, K))
    return _cache[(N, K, seed)]


@pytest.mark.parametrize("N,K,seed", [(128, 128, 6), (384, 256, 7), (256, 640, 8), (2560, 6912, 5003), (3840, 2560, 5000)])
def test_pack5_bytes_match_oracle(oracle_mod, B, N, K, seed):
    _, _, lin5, _ = layer5(oracle_mod, B, N, K, seed)
    pieces = -(-K // 160)
    assert lin5.nbytes == (N // 128) * pieces * 4096  # what a forward call streams: 1.6 bits per weight (+ padding to 160)


@pytest.mark.parametrize("M,out_dtype", [(1, 1), (2, 0), (2, 1)])
def test_forward_multi5_matches_oracle_and_two_bit_path(oracle_mod, B, M, out_dtype):
    specs = [(3840, 2560, 5000), (384, 256, 7), (2560, 6912, 5003), (128, 128, 6), (2560, 2560, 5001), (256, 640, 8),
             (13824, 2560, 5002)]
    xs_cpu = {K: inputs.activations(M, K, 3700 + K + M) for K in {k for _, k, _ in specs}}
    xs_gpu = {K: v.cuda() for K, v in xs_cpu.items()}
    ws5, ws2, xs, ys5, ys2, refs = [], [], [], [], [], []
    dt = torch.float32 if out_dtype == 0 else torch.bfloat16
    for N, K, seed in specs:
        Wq, g, lin5, lin2 = layer5(oracle_mod, B, N, K, seed)
        ws5.append(lin5)
        ws2.append(lin2)
        xs.append(xs_gpu[K])
        ys5.append(torch.full((M, N), 7.0, dtype=dt, device="cuda"))
        ys2.append(torch.full((M, N), 9.0, dtype=dt, device="cuda"))
        refs.append(oracle_mod.bitlinear(inputs.bf16_bits(xs_cpu[K]), Wq, g))
    call5 = B.MultiCall5(ws5, xs, ys5, out_dtype)
    call5.run()
    call5.run()
    B.MultiCall(ws2, xs, ys2, out_dtype).run()
    B.poll_status()
    for y5, y2, ref in zip(ys5, ys2, refs):
        assert torch.equal(y5, y2)
        if out_dtype == 0:
            assert np.array_equal(y5.cpu().numpy(), ref["y32"])
        else:
            yb = inputs.bf16_bits(y5.cpu())
            assert np.array_equal(yb, ref["ybf16"])
            y64 = ref["y64"]
            err = np.abs(bits_to_f64(yb) - y64) / np.where(y64 == 0, 1.0, np.abs(y64))
            assert err.max() <= 8e-3


def test_forward_multi5_argument_errors(oracle_mod, B):
    import ctypes
    L = B.lib()
    _, _, lin5, _ = layer5(oracle_mod, B, 384, 256, 7)
    x = inputs.activations(2, 256, 1).cuda()
    y = torch.empty(2, 384, dtype=torch.bfloat16, device="cuda")
    vp = ctypes.c_void_p
    w1, x1, y1 = (vp * 1)(lin5.handle), (vp * 1)(x.data_ptr()), (vp * 1)(y.data_ptr())
    assert L.bitrl_bitlinear5_forward_multi(0, w1, x1, y1, 2, 1, None) == B.ERR_SHAPE
    assert L.bitrl_bitlinear5_forward_multi(1, w1, x1, y1, 3, 1, None) == B.ERR_SHAPE
    assert L.bitrl_bitlinear5_forward_multi(1, w1, x1, y1, 2, 9, None) == B.ERR_DTYPE
    assert L.bitrl_bitlinear5_forward_multi(1, w1, (vp * 1)(None), y1, 2, 1, None) == B.ERR_NULL
    assert L.bitrl_bitlinear5_forward_multi(1, w1, x1, y1, 2, 1, None) == B.OK
    B.poll_status()
