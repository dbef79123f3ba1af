"""The C-ABI library builds, loads, and exports every symbol that include/bitrl.h declares (no compute calls)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "bitrl.h")).read()
    return sorted(set(re.findall(r"BITRL_API[^;]*?\b(bitrl_\w+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_symbols()
    for must in ("bitrl_pack_ternary", "bitrl_quant_act", "bitrl_bitlinear_forward", "bitrl_encoder_forward"):
        assert must in names
    assert len(names) >= 20


def test_library_exports_every_declared_symbol():
    from paper_2604_24273_b200 import build as lib_build

    path = lib_build.build()
    lib = ctypes.CDLL(str(path))
    for name in declared_symbols():
        assert hasattr(lib, name), f"{name} declared in bitrl.h but not exported"


def test_binding_covers_the_header_and_host_only_calls_work():
    from paper_2604_24273_b200 import bitrl

    assert sorted(bitrl.EXPORTS) == declared_symbols()
    L = bitrl.lib()
    assert L.bitrl_status_string(0) == b"ok"
    assert L.bitrl_status_string(bitrl.ERR_TIMEOUT) == b"device-side wait timed out"
    assert L.bitrl_pack_workspace_bytes(256, 256) >= 8
    assert L.bitrl_workspace_bytes(1, 2560, 3840) == 0          # streaming kernel needs no workspace
    assert L.bitrl_workspace_bytes(4096, 2560, 6912) >= 4096 * 2560 + 2 * 4096 * 4
    # argument validation happens before any CUDA call
    assert L.bitrl_pack_ternary(None, 256, 256, None, None, None, 0, None) == bitrl.ERR_NULL
    assert L.bitrl_quant_act(None, 1, 256, None, None, None, None) == bitrl.ERR_NULL
