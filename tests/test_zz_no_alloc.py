"""The allocation-free packing entry point against the regular one.

``bitrl_pack_ternary_static`` exists for callers that must not allocate device memory (a fixed memory pool, a
stream-ordered section where an allocation would stall the device, a host application that owns the allocator).
It keeps its fp64 partial sums in a fixed array inside the library instead of a caller workspace, so the array is
shared by every call and keeps old contents: the test calls it twice in a row, the second time on a smaller
matrix that uses fewer slots than the first left behind, and demands byte-identical codes and a bit-identical
gamma to ``bitrl_pack_ternary`` both times.  Collected last on purpose, so a run that stops at the first failure has
already run every other test.
"""
import ctypes

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


def test_static_scratch_pack_matches_workspace_pack_twice(B):
    warm = inputs.master_weights(128, 128, 40).cuda()  # first call on the device: looks the scratch address up
    B.pack_ternary_static(warm, torch.empty((128, 32), dtype=torch.uint8, device="cuda"),
                          torch.empty((1,), dtype=torch.float32, device="cuda"))
    for N, K, seed in ((2560, 6912, 41), (384, 256, 42), (2560, 3840, 43)):
        W = inputs.master_weights(N, K, seed).cuda()
        want_packed, want_gamma = B.pack_ternary(W)
        packed = torch.full((N, K // 4), 0xAA, dtype=torch.uint8, device="cuda")
        gamma = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        B.pack_ternary_static(W, packed, gamma)
        B.poll_status()
        # the property the entry point exists for: the device's free memory is what it was (after the first call on the
        # device, which loads nothing either - the scratch array is part of the library image)
        assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.equal(gamma.view(torch.int32), want_gamma.view(torch.int32))  # bit-identical scale
        assert torch.equal(packed, want_packed)                                    # byte-identical codes


def test_static_scratch_pack_rejects_oversize_and_bad_arguments(B):
    L = B.lib()
    W = inputs.master_weights(128, 128, 44).cuda()
    packed = torch.empty((128, 32), dtype=torch.uint8, device="cuda")
    gamma = torch.empty((1,), dtype=torch.float32, device="cuda")
    launches = B.launch_count()
    # 65536 x 8192 = 2^29 weights is beyond the 2^28 limit: refused before anything is launched or read
    assert L.bitrl_pack_ternary_static(W.data_ptr(), 65536, 8192, packed.data_ptr(), gamma.data_ptr(), None) == B.ERR_LIMIT
    assert L.bitrl_pack_ternary_static(None, 128, 128, packed.data_ptr(), gamma.data_ptr(), None) == B.ERR_NULL
    assert L.bitrl_pack_ternary_static(W.data_ptr(), 100, 128, packed.data_ptr(), gamma.data_ptr(), None) == B.ERR_SHAPE
    assert B.launch_count() == launches  # a refused call launches nothing
    assert L.bitrl_status_string(B.ERR_LIMIT) == b"size beyond the fixed maximum of this entry point"
    B.poll_status()
