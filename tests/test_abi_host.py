"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares, sizes
its buffers as documented, and rejects bad arguments on the host before any launch."""
import ctypes
import os
import re

import pytest

import paper_2606_02823_b200 as qift
from paper_2606_02823_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    if not os.path.exists(binding.LIB_PATH):
        from paper_2606_02823_b200 import build
        build.build()
    return qift.lib()


def test_every_declared_symbol_is_exported(L):
    header = open(os.path.join(ROOT, "include", "qift.h")).read()
    declared = sorted(set(re.findall(r"\b(qift_[a-z0-9_]+)\s*\(", header)))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(L, name), f"{name} declared in qift.h but not exported"
    assert sorted(binding.EXPORTS) == declared


def test_sizes(L):
    assert qift.qift_packed_bytes(4096, 4096, qift.MNZ) == 4096 * 4096 // 4
    assert qift.qift_packed_bytes(4096, 11008, qift.INT4) == 4096 * 11008 // 2
    assert qift.qift_packed_bytes(16, 24, qift.MNZ) == 0          # K not a multiple of 16
    assert qift.qift_packed_bytes(0, 16, qift.MNZ) == 0
    assert qift.qift_workspace_bytes(1, 4096, 4096, qift.MNZ) == 0
    assert qift.qift_workspace_bytes(16, 4096, 4096, qift.POT) == 16 * 4096 + 1024     # re-laid-out activations + token sums, 1 KiB steps
    assert qift.qift_workspace_bytes(64, 4096, 4096, qift.MNZ) == 64 * 4096 + 1024     # row-split route up to 64 rows
    assert qift.qift_workspace_bytes(16, 4096, 4096, qift.POT, qift.ROUTE_DECODE) == 0
    assert qift.qift_workspace_bytes(3, 64, 48, qift.MNZ) == 0                         # K not in whole 16-word slices: generic route
    assert qift.qift_workspace_bytes(512, 4096, 4096, qift.MNZ) == 512 * 4            # per-token sums only
    assert qift.qift_workspace_bytes(2048, 4096, 4096, qift.MNZ) == 4096 * 4096       # int8 scratch
    assert qift.qift_workspace_bytes(65, 3, 16, qift.SYM) == 1024                      # rounded up to 1 KiB
    assert qift.qift_workspace_bytes(2048, 4096, 4096, qift.MNZ, qift.ROUTE_PREFILL_SCRATCH) == 4096 * 4096
    assert qift.qift_workspace_bytes(8, 4096, 4096, qift.MNZ, qift.ROUTE_PREFILL_SCRATCH) == 4096 * 4096
    assert qift.qift_workspace_bytes(8, 4096, 4096, qift.MNZ, qift.ROUTE_GENERIC) == 0
    # the L = 16 mixed stack stores exactly 3 bits per weight
    import synth
    w4 = sum(qift.qift_packed_bytes(n, k, qift.INT4) for _, n, k in synth.LLAMA2_7B)
    w2 = sum(qift.qift_packed_bytes(n, k, qift.MNZ) for _, n, k in synth.LLAMA2_7B)
    weights = sum(n * k for _, n, k in synth.LLAMA2_7B)
    assert (16 * w4 + 16 * w2) * 8 == 3 * 32 * weights


def test_status_strings(L):
    seen = {qift.status_string(s) for s in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert qift.status_string(99) == "unknown status"


def test_bad_arguments_are_rejected_before_any_launch(L):
    p = ctypes.c_void_p(4096)      # never dereferenced: these calls fail validation first
    odd = ctypes.c_void_p(4100)
    null = None
    # null pointers / sizes / enums
    assert L.qift_pack_weights(null, 4, 16, 0, 1, p, p, None) == qift.ERR_INVALID_ARG
    assert L.qift_pack_weights(p, 0, 16, 0, 1, p, p, None) == qift.ERR_INVALID_ARG
    assert L.qift_pack_weights(p, 4, 16, 7, 1, p, p, None) == qift.ERR_INVALID_ARG
    assert L.qift_pack_weights(p, 4, 16, 0, 5, p, p, None) == qift.ERR_INVALID_ARG
    assert L.qift_pack_weights(p, 4, 24, 0, 1, p, p, None) == qift.ERR_UNSUPPORTED_SHAPE
    assert L.qift_pack_weights(p, 4, 32768, 0, 1, p, p, None) == qift.ERR_UNSUPPORTED_SHAPE
    assert L.qift_pack_weights(odd, 4, 16, 0, 1, p, p, None) == qift.ERR_ALIGNMENT
    assert L.qift_quantize_act(p, 0, 1, 256, 96, 0.9, p, p, None) == qift.ERR_UNSUPPORTED_SHAPE   # not a power of two
    assert L.qift_quantize_act(p, 0, 1, 256, 512, 0.9, p, p, None) == qift.ERR_UNSUPPORTED_SHAPE  # does not divide K
    assert L.qift_quantize_act(p, 0, 1, 256, 256, 0.0, p, p, None) == qift.ERR_INVALID_ARG
    assert L.qift_quantize_act(p, 0, 1, 256, 256, 1.5, p, p, None) == qift.ERR_INVALID_ARG
    assert L.qift_quantize_act(p, 3, 1, 256, 256, 0.9, p, p, None) == qift.ERR_INVALID_ARG
    assert L.qift_quantize_act(p, 0, 1, 256, 256, 0.9, odd, p, None) == qift.ERR_ALIGNMENT
    assert L.qift_rotate(p, 1, 256, 0, p, None) == qift.ERR_UNSUPPORTED_SHAPE
    assert L.qift_unpack_codes(p, 1, 12, 0, p, None) == qift.ERR_UNSUPPORTED_SHAPE
    # linear: the W2 entry refuses INT4, K must hold whole words, prefill needs its workspace
    assert L.qift_w2a4_linear(p, p, qift.INT4, p, p, 1, 16, 256, p, 0, None, None, 0, None) == qift.ERR_INVALID_ARG
    assert L.qift_w2a4_linear(p, p, 0, p, p, 1, 16, 40, p, 0, None, None, 0, None) == qift.ERR_UNSUPPORTED_SHAPE
    assert L.qift_w2a4_linear(p, p, 0, p, p, 0, 16, 256, p, 0, None, None, 0, None) == qift.ERR_INVALID_ARG
    assert L.qift_w2a4_linear(p, p, 0, p, p, 1, 16, 256, p, 9, None, None, 0, None) == qift.ERR_INVALID_ARG
    assert L.qift_w2a4_linear(p, p, 0, odd, p, 1, 16, 256, p, 0, None, None, 0, None) == qift.ERR_ALIGNMENT
    assert L.qift_w2a4_linear(p, p, 0, p, p, 64, 16, 256, p, 0, None, None, 0, None) == qift.ERR_WORKSPACE
    assert L.qift_w4a4_linear(p, p, p, p, 64, 16, 256, p, 0, None, p, 16, None) == qift.ERR_WORKSPACE
    assert L.qift_linear_route(p, p, 0, p, p, 32, 16, 256, p, 0, None, None, 0, qift.ROUTE_DECODE, None) \
        == qift.ERR_UNSUPPORTED_SHAPE
    assert L.qift_linear_route(p, p, 0, p, p, 1, 16, 256, p, 0, None, None, 0, 9, None) == qift.ERR_INVALID_ARG
    # three-bit codes: K in whole high words; only the routes that serve the level set; packed size 3 bits per weight
    assert L.qift_pack_weights(p, 16, 48, qift.INT3, 1, p, p, None) == qift.ERR_UNSUPPORTED_SHAPE
    assert L.qift_w3a4_linear(p, p, p, p, 1, 16, 48, p, 0, None, None, 0, None) == qift.ERR_UNSUPPORTED_SHAPE
    assert L.qift_linear_route(p, p, qift.INT3, p, p, 4, 16, 256, p, 0, None, None, 0, qift.ROUTE_DECODE, None) \
        == qift.ERR_UNSUPPORTED_SHAPE
    assert L.qift_w3a4_linear(p, p, p, p, 64, 16, 256, p, 0, None, None, 0, None) == qift.ERR_WORKSPACE
    assert L.qift_packed_bytes(4096, 4096, qift.INT3) == 4096 * 4096 * 3 // 8
    # grouped plans: token-row limits per level set; plans that need tensor maps want a 128-byte aligned device plan
    prob = binding.GroupProblem(4096, 4096, 4096, 4096, 4096, 4096, None, 256, 256, 256, 0)
    n = L.qift_group_plan_bytes(1)
    host = ctypes.create_string_buffer(n + 256)
    hp = ctypes.c_void_p((ctypes.addressof(host) + 255) & ~255)
    plan = lambda M, lv, dev: L.qift_group_plan(ctypes.byref(prob), 1, M, lv, 0, 0, 0.9, hp, ctypes.c_void_p(dev), n, None)
    assert plan(129, qift.MNZ, 4096) == qift.ERR_UNSUPPORTED_SHAPE
    assert plan(17, qift.INT3, 4096) == qift.ERR_UNSUPPORTED_SHAPE
    assert plan(64, qift.MNZ, 4096 + 64) == qift.ERR_ALIGNMENT


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libqift.so"))
    with pytest.raises(FileNotFoundError):
        binding.lib()
