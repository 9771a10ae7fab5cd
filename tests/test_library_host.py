"""CPU-side checks of the C-ABI library: it loads without a GPU and exports what include/lrq.h declares."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2508_03485_b200 import build, binding
    build.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "lrq.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(lrq_[a-z0-9_]+)\s*\(", hdr))
    assert {"lrq_tlq_quantize_weights", "lrq_rotate_quantize_act", "lrq_qlinear", "lrq_qlinear_stack"} <= declared
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in lrq.h but not exported"
    from paper_2508_03485_b200.binding import EXPORTS
    assert declared == set(EXPORTS)


def test_status_strings_and_version(lib):
    assert lib.lrq_version() >= 100
    seen = {lib.lrq_status_string(i).decode() for i in range(6)}
    assert len(seen) == 6 and "ok" in seen


def test_argument_checks_run_before_any_launch(lib):
    # null pointers and bad sizes are rejected on the host; nothing touches a device
    import ctypes as C
    from paper_2508_03485_b200.binding import _ActParams, _TlqParams
    p = _ActParams(1, 128, None, 8, 0)
    assert lib.lrq_rotate_quantize_act(None, 4, 128, 128, C.byref(p), None, None, None, None, 0, None) == 1
    fake = C.c_void_p(0x1000)   # never dereferenced: the size checks fail first
    assert lib.lrq_rotate_quantize_act(fake, 4, 130, 130, C.byref(p), fake, fake, fake, None, 0, None) == 2
    p2 = _ActParams(1, 96, None, 8, 0)      # not a power of two
    assert lib.lrq_rotate_quantize_act(fake, 4, 192, 192, C.byref(p2), fake, fake, fake, None, 0, None) == 2
    p3 = _ActParams(1, 128, None, 5, 0)     # unsupported bit-width
    assert lib.lrq_rotate_quantize_act(fake, 4, 128, 128, C.byref(p3), fake, fake, fake, None, 0, None) == 2
    p4 = _ActParams(2, 0, 0x1000, 8, 0)     # dense rotation without workspace
    assert lib.lrq_rotate_quantize_act(fake, 4, 128, 128, C.byref(p4), fake, fake, fake, None, 0, None) == 3
    assert lib.lrq_act_workspace_bytes(5, 128, C.byref(p4)) == 2560
    assert lib.lrq_act_workspace_bytes(5, 128, C.byref(p)) == 0
    a = (C.c_double * 1)(1.0)
    t = _TlqParams(5, 0, 7, 1, 1, a, a, 0)
    assert lib.lrq_tlq_quantize_weights(fake, 8, 64, C.byref(t), fake, fake, None, fake, None, 0, None) == 2
    t = _TlqParams(4, 48, 7, 1, 1, a, a, 0)    # group does not divide K
    assert lib.lrq_tlq_quantize_weights(fake, 8, 64, C.byref(t), fake, fake, None, fake, None, 0, None) == 2
    h = C.c_void_p()
    assert lib.lrq_layer_create(C.byref(h), 8, 64, 4, 0, 0, None, fake, fake, None, None, C.byref(p)) == 1
    assert lib.lrq_layer_create(C.byref(h), 8, 64, 4, 0, 0, fake, fake, fake, None, None, C.byref(p)) == 2  # 128 does not divide 64
    p5 = _ActParams(1, 64, None, 8, 0)
    assert lib.lrq_layer_create(C.byref(h), 8, 64, 4, 0, 0, fake, fake, fake, None, None, C.byref(p5)) == 0
    assert lib.lrq_workspace_bytes(h, 10) == 768 + 256 + 256
    assert lib.lrq_qlinear(h, fake, 10, 64, fake, 0, 8, None, 0, None) == 3       # workspace missing
    assert lib.lrq_qlinear(h, fake, 10, 64, fake, 0, 4, fake, 1 << 20, None) == 1  # ldy < N
    assert lib.lrq_qlinear(h, fake, 0, 64, fake, 0, 64, fake, 1 << 20, None) == 1  # no tokens: an argument error, nothing launched
    lib.lrq_layer_destroy(h)
    assert lib.lrq_rotate_quantize_act(fake, 0, 128, 128, C.byref(p), fake, fake, fake, None, 0, None) == 1
    # weight rotation: block size must be a power of two dividing K; a dense rotation needs R and cannot run in place
    assert lib.lrq_rotate_weights(fake, 8, 192, 192, None, 1, 128, None, fake, 192, None) == 1
    assert lib.lrq_rotate_weights(fake, 8, 128, 128, None, 2, 0, None, fake, 128, None) == 1
    assert lib.lrq_rotate_weights(fake, 8, 128, 128, None, 2, 0, fake, fake, 128, None) == 1
    assert lib.lrq_rotate_weights(fake, 8, 128, 64, None, 0, 0, None, fake, 128, None) == 1      # ldw < K
    # dual transformation: all three factors, blocks of 128, K a multiple of 128, scratch of 10 bytes per element
    d = _ActParams(3, 0, None, 8, 0, None, 128, 0x1000, 0x1000, 0x1000)
    assert lib.lrq_act_workspace_bytes(5, 256, C.byref(d)) == 5120 + 7680
    assert lib.lrq_rotate_quantize_act(fake, 4, 256, 256, C.byref(d), fake, fake, fake, None, 0, None) == 3
    assert lib.lrq_rotate_quantize_act(fake, 4, 192, 192, C.byref(d), fake, fake, fake, fake, 1 << 20, None) == 2
    d_missing = _ActParams(3, 0, None, 8, 0, None, 128, 0x1000, None, 0x1000)
    assert lib.lrq_rotate_quantize_act(fake, 4, 256, 256, C.byref(d_missing), fake, fake, fake, fake, 1 << 20, None) == 1
    d64 = _ActParams(3, 0, None, 8, 0, None, 64, 0x1000, 0x1000, 0x1000)
    assert lib.lrq_rotate_quantize_act(fake, 4, 256, 256, C.byref(d64), fake, fake, fake, fake, 1 << 20, None) == 2
    assert lib.lrq_rotate_weights_dual(fake, 8, 256, 256, None, 128, fake, None, fake, fake, 256, None) == 1
    assert lib.lrq_rotate_weights_dual(fake, 8, 200, 200, None, 128, fake, fake, fake, fake, 200, None) == 1
    assert lib.lrq_static_scratch_bytes() == 8 << 20
    # rotation choice: 8 bytes of workspace, K a multiple of 16
    assert lib.lrq_ars_select(fake, 4, 128, 128, 1.0, fake, fake, None, 0, None) == 3
    assert lib.lrq_ars_select(fake, 4, 120, 120, 1.0, fake, fake, fake, 8, None) == 2


def test_calling_without_a_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    import paper_2508_03485_b200 as P
    with pytest.raises(ValueError):
        P.lrq_rotate_quantize_act(torch.zeros(4, 128, dtype=torch.bfloat16), P.ROT_HADAMARD, 8, 128)
