"""Host-only checks of the C-ABI library: it loads, exports every declared symbol, and
rejects bad arguments with a status instead of crashing.  No kernel is launched here."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    import __graft_entry__ as ge
    ge.build()
    from paper_2404_15159_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(B):
    header = open(os.path.join(ROOT, "include", "mixlora.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(mixlora_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(B.lib, name), f"{name} declared in mixlora.h but not exported"
    assert declared == set(B.EXPORTS)


def test_limits_and_status_strings(B):
    lim = B.mixlora_limits()
    assert lim == dict(max_experts=32, max_top_k=8, max_rank=128)
    assert B.status_string(0) == "ok"
    for code in range(1, 6):
        assert B.status_string(code) not in ("ok", "unknown status")


def test_struct_layout_matches_header(B):
    assert C.sizeof(B.mixlora_shape_t) == 44
    assert C.sizeof(B.mixlora_params_t) == 12 * 8
    assert C.sizeof(B.mixlora_grads_t) == 9 * 8 + 8


def test_workspace_bytes_grow_with_tokens_and_reject_bad_shapes(B):
    s1 = B.make_shape(256, 256, 688, 4, 2, 8, 16.0, B.MIXLORA_DTYPE_FP32)
    s2 = B.make_shape(512, 256, 688, 4, 2, 8, 16.0, B.MIXLORA_DTYPE_FP32)
    f1, b1 = B.mixlora_workspace_bytes(s1, False), B.mixlora_workspace_bytes(s1, True)
    assert 0 < f1 < b1 and b1 % 256 == 0
    assert B.mixlora_workspace_bytes(s2, True) > b1
    assert B.mixlora_workspace_bytes(B.make_shape(0, 256, 688, 4, 2, 8, 16.0), True) > 0
    bad = [B.make_shape(256, 250, 688, 4, 2, 8, 16.0),          # d not a multiple of 8
           B.make_shape(256, 256, 688, 4, 5, 8, 16.0),          # k > N
           B.make_shape(256, 256, 688, 64, 2, 8, 16.0),         # N above the limit
           B.make_shape(256, 256, 688, 4, 2, 256, 16.0),        # r above the limit
           B.make_shape(256, 256, 688, 4, 2, 12, 16.0),         # bf16 rank not a multiple of 8
           B.make_shape(-1, 256, 688, 4, 2, 8, 16.0),
           B.make_shape(256, 256, 688, 4, 2, 8, 16.0, dtype=7)]
    for s in bad:
        assert B.mixlora_workspace_bytes(s, True) == 0
    s = B.make_shape(256, 256, 688, 4, 2, 8, 16.0)
    s.struct_size = 12
    assert B.mixlora_workspace_bytes(s, True) == 0


def test_calls_reject_null_and_misaligned_pointers_without_touching_the_device(B):
    s = B.make_shape(16, 64, 128, 4, 2, 8, 16.0)
    p = B.mixlora_params_t()                                     # all NULL
    st = B.lib.mixlora_ffn_forward(C.byref(s), C.byref(p), 256, 256, 1 << 30, None)
    assert st == 1
    for name, _ in B.mixlora_params_t._fields_:
        setattr(p, name, 4096)
    p.w_gate = 4100                                              # misaligned
    assert B.lib.mixlora_ffn_forward(C.byref(s), C.byref(p), 4096, 4096, 1 << 30, None) == 1
    p.w_gate = 4096
    assert B.lib.mixlora_ffn_forward(C.byref(s), C.byref(p), None, 4096, 1 << 30, None) == 1      # y NULL
    assert B.lib.mixlora_ffn_forward(C.byref(s), C.byref(p), 4096, None, 1 << 30, None) == 3      # workspace NULL
    assert B.lib.mixlora_ffn_forward(C.byref(s), C.byref(p), 4096, 4096 + 16, 1 << 30, None) == 3  # misaligned ws
    assert B.lib.mixlora_ffn_forward(C.byref(s), C.byref(p), 4096, 4096, 16, None) == 3           # too small
    g = B.mixlora_grads_t()
    assert B.lib.mixlora_ffn_backward(C.byref(s), C.byref(p), None, 0.0, 4096, 1 << 30, C.byref(g), None) == 1
    g.accumulate = 3
    assert B.lib.mixlora_ffn_backward(C.byref(s), C.byref(p), 4096, 0.0, 4096, 1 << 30, C.byref(g), None) == 1
    g.accumulate = 0
    assert B.lib.mixlora_ffn_backward(C.byref(s), C.byref(p), 4096, 0.0, 4096, 16, C.byref(g), None) == 3
    assert B.lib.mixlora_aux_loss(C.byref(s), None, 0.01, 4096, None, None, None) == 3
    assert B.lib.mixlora_aux_loss(C.byref(s), 4096, 0.01, None, None, None, None) == 1
    assert B.lib.mixlora_gemm_bf16(None, 4096, 4096, 8, 8, 8, 0, None, None) == 1
    assert B.lib.mixlora_gemm_bf16(4096, 4096, 4096, 8, 12, 8, 0, None, None) == 2
    bad = B.make_shape(16, 64, 128, 4, 9, 8, 16.0)
    assert B.lib.mixlora_ffn_forward(C.byref(bad), C.byref(p), 4096, 4096, 1 << 30, None) == 1
    big = B.make_shape(16, 64, 128, 40, 2, 8, 16.0)
    assert B.lib.mixlora_ffn_forward(C.byref(big), C.byref(p), 4096, 4096, 1 << 30, None) == 2
