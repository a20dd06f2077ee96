"""The C-ABI library: it loads, exports what include/d2moe.h declares, and rejects bad arguments on
the host before any launch.  No kernel runs here."""
import ctypes
import os
import re

import pytest

from paper_2504_15299_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "d2moe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(d2moe_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert set(names) == set(binding.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def good():
    return binding.Config(256, 512, 4, 2, 64, (2, 4, 8))


def test_status_strings(lib):
    assert binding.status_string(0) == "ok"
    assert "NULL" in binding.status_string(1)
    assert binding.status_string(99) == "unknown status"


@pytest.mark.parametrize("mutate,code", [
    (lambda c: setattr(c, "top_k", 5), 2),
    (lambda c: setattr(c, "top_k", 0), 2),
    (lambda c: setattr(c, "bits", (4, 2, 8)), 2),
    (lambda c: setattr(c, "bits", (2, 4, 9)), 2),
    (lambda c: setattr(c, "bits", (0, 4)), 2),
    (lambda c: setattr(c, "group_size", 48), 2),
    (lambda c: setattr(c, "group_size", 128), 0),
    (lambda c: setattr(c, "d_model", 200), 2),
    (lambda c: setattr(c, "scale_mode", 1), 0),
    (lambda c: setattr(c, "scale_mode", 2), 2),
    (lambda c: setattr(c, "renormalize", 2), 2),
    (lambda c: setattr(c, "kernel_path", 7), 2),
    (lambda c: setattr(c, "n_experts", 300), 2),
    (lambda c: setattr(c, "d_ffn", 1 << 19), 2),       # beyond D2MOE_MAX_DIM: no launch could take it
    (lambda c: setattr(c, "d_ffn", 1 << 18), 0),
])
def test_check_config(lib, mutate, code):
    c = good()
    mutate(c)
    assert binding.check_config(c) == code


def test_packed_bytes_is_the_top_width_only(lib):
    rows, cols = 512, 256
    a = binding.packed_bytes(binding.Config(256, 512, 4, 2, 64, (2, 3, 4, 8)), rows, cols)
    b = binding.packed_bytes(binding.Config(256, 512, 4, 2, 64, (2, 4, 8)), rows, cols)
    c = binding.packed_bytes(binding.Config(256, 512, 4, 2, 64, (8,)), rows, cols)
    assert a == b == c
    total, code, meta = a
    assert code == rows * cols and meta == rows * (cols // 64) * 4 and total == 256 + code + meta
    # so do lists whose steps are not powers of two: 5 = 4 + 1, 3 = 2 + 1, 7 = 4 + 2 + 1 bits, eight one-bit steps
    for bits in ((5, 6, 7, 8), (3, 8), (1, 8), (1, 2, 3, 4, 5, 6, 7, 8), (7, 8), (6, 8)):
        assert binding.packed_bytes(binding.Config(256, 512, 4, 2, 64, bits), rows, cols) == a, bits
    assert binding.packed_bytes(binding.Config(256, 512, 4, 2, 64, (3, 5)), rows, cols)[1] == rows * cols * 5 // 8
    # a 4-bit top width stores half of that
    assert binding.packed_bytes(binding.Config(256, 512, 4, 2, 64, (2, 3, 4)), rows, cols)[1] == rows * cols // 2
    # rows are padded to the 64-row tile
    assert binding.packed_bytes(good(), 100, 256)[1] == 128 * 256
    with pytest.raises(binding.D2MoEError):
        binding.packed_bytes(good(), 64, 100)
    # free residual scales: the same code bytes, six more fp16 scales per (row, group)
    free = binding.Config(256, 512, 4, 2, 64, (2, 3, 4, 8), scale_mode=1)
    t1, c1, m1 = binding.packed_bytes(free, rows, cols)
    assert c1 == code and m1 == rows * (cols // 64) * (4 + 2 * 6) and t1 == 256 + c1 + m1


def test_null_and_short_buffers_are_rejected_before_launch(lib):
    c = good().c()
    L = lib
    # pack: NULL pointers
    assert L.d2moe_pack_mwq(ctypes.byref(c), None, 64, 64, None, 0, None) == 1
    # pack: short output, misaligned output (fake non-null pointers are never dereferenced)
    assert L.d2moe_pack_mwq(ctypes.byref(c), 4096, 64, 64, 8192, 10, None) == 5
    assert L.d2moe_pack_mwq(ctypes.byref(c), 4096, 64, 64, 8192 + 16, 1 << 20, None) == 3
    # unpack: width outside [b1, top]
    assert L.d2moe_unpack_codes(ctypes.byref(c), 4096, 64, 64, 1, 4096, None, None, None) == 3
    # workspace query
    assert binding.workspace_bytes(good(), 16) > 0
    # a workspace sized for max_tokens serves every smaller batch, whichever expert kernel it takes
    big = binding.Config(4096, 14336, 8, 2, 128, (2, 3, 4, 8))
    sizes = [binding.workspace_bytes(big, t) for t in (1, 8, 64, 256, 257, 512, 2048)]
    assert all(a <= b for a, b in zip(sizes, sizes[1:])), sizes
    bad = good(); bad.top_k = 9
    assert L.d2moe_workspace_bytes(ctypes.byref(bad.c()), 16) == 0
    # route: both / neither of gate_w and logits
    args_tail = [4096] * 6 + [None, 4096, 1 << 30, None]
    assert L.d2moe_route(ctypes.byref(c), 4, 4096, None, None, None, 4096, *args_tail) == 1
    assert L.d2moe_route(ctypes.byref(c), 4, 4096, 4096, 4096, None, 4096, *args_tail) == 1
    assert L.d2moe_route(ctypes.byref(c), 4, 4096, 4096, None, None, None, *args_tail) == 1
    # route: short workspace
    assert L.d2moe_route(ctypes.byref(c), 4, 4096, 4096, None, None, 4096, *([4096] * 6), None, 4096, 16, None) == 5
    # forward: T == 0 is a no-op, negative T is a shape error, missing expert pointer is NULL
    assert L.d2moe_moe_forward(ctypes.byref(c), 0, None, None, None, None, None, None, None, 0, None) == 0
    assert L.d2moe_moe_forward(ctypes.byref(c), -1, None, None, None, None, None, None, None, 0, None) == 3
    assert L.d2moe_moe_forward(ctypes.byref(c), (1 << 20) + 1, None, None, None, None, None, None, None, 0, None) == 3
    ptrs = (ctypes.c_void_p * 12)(*([4096] * 11 + [None]))
    rin = binding._RouteIn(4096, None, None, 4096)
    assert L.d2moe_moe_forward(ctypes.byref(c), 4, 4096, ptrs, ctypes.byref(rin), None, 4096, None, 4096,
                               1 << 30, None) == 1
    ptrs = (ctypes.c_void_p * 12)(*([4096] * 12))
    assert L.d2moe_moe_forward(ctypes.byref(c), 4, 4096, ptrs, ctypes.byref(rin), None, 4096, None, 4096,
                               16, None) == 5
    # stack layer: argument errors are found before the normalisation kernel would be launched
    assert L.d2moe_stack_layer(ctypes.byref(c), 4, 4096, 4096, ctypes.c_float(1e-5), ptrs, ctypes.byref(rin),
                               None, 4096, 16, None) == 5


def test_static_scratch_routing_refuses_what_its_array_cannot_hold(lib):
    # more assignments than the built-in scratch array holds: refused before any launch (the fake non-null
    # pointers are never dereferenced); the key limit equals the most (expert, width) pairs a valid
    # configuration can have (256 experts x 8 widths), so it can never be exceeded
    args = [4096, 4096, None, None, 4096] + [4096] * 6 + [None, None]
    c = good().c()
    assert lib.d2moe_route_static_scratch(ctypes.byref(c), -1, *args) == 3
    too_many_tokens = binding.STATIC_MAX_ASSIGNMENTS // c.top_k + 1
    assert lib.d2moe_route_static_scratch(ctypes.byref(c), too_many_tokens, *args) == 5
    assert binding.STATIC_MAX_KEYS == 256 * 8
