"""The allocation-free entry point lrq_rotate_quantize_act_static against the ordinary one.

Some callers of this library cannot allocate device memory when they call it (a host whose memory is planned
by another runtime, or one that forbids cudaMalloc after start-up); for them the dense rotation's scratch is a
fixed array inside the library.  The two entry points run the same kernels, so their results must agree bit
for bit, on two calls in a row (the array keeps the previous call's contents) and whatever ran before."""
import numpy as np
import pytest
import torch

import parity as PU
from lrq_workloads import f32_to_bf16_bits, make_activations, make_orthogonal

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2508_03485_b200 as P
    P.load_library()
    return P


def _free_bytes():
    return torch.cuda.mem_get_info()[0]


def test_static_scratch_matches_workspace_path_twice(P):
    K = 384
    R = PU.bf16_to_device(f32_to_bf16_bits(make_orthogonal(11, K).astype(np.float32)))
    warm = PU.bf16_to_device(make_activations(9, 1, K))
    P.lrq_rotate_quantize_act_static(warm, P.ROT_DENSE, 8, R=R)                # start-up call: loads the module
    torch.cuda.synchronize()
    # second call: fewer tokens and other data, so stale scratch rows from the first call lie beyond it
    for M, seed, a_bits in [(300, 1, 8), (77, 2, 4)]:
        X = PU.bf16_to_device(make_activations(seed, M, K, n_salient=16, salient_x=100.0))
        ref = P.lrq_rotate_quantize_act(X, P.ROT_DENSE, a_bits, R=R)
        # the caller's own result buffers, as a host that may not allocate would pass them
        out = (torch.empty((M, K * a_bits // 8), dtype=torch.uint8, device="cuda"),
               torch.empty((M,), dtype=torch.float32, device="cuda"),
               torch.empty((M,), dtype=torch.int32, device="cuda"))
        got = None                                                             # drop the previous round's buffers now
        torch.cuda.synchronize()
        held, reserved, free = torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), _free_bytes()
        got = P.lrq_rotate_quantize_act_static(X, P.ROT_DENSE, a_bits, R=R, out=out)
        torch.cuda.synchronize()
        # nothing was allocated: neither through torch's allocator nor behind its back on the device
        assert torch.cuda.memory_allocated() == held and torch.cuda.memory_reserved() == reserved
        assert _free_bytes() == free
        assert all(g is o for g, o in zip(got, out))
        for g, r in zip(got, ref):
            assert torch.equal(g, r)
    assert P.lrq_device_status() == 0


def test_static_scratch_other_kinds_and_limit(P):
    X = PU.bf16_to_device(make_activations(3, 64, 1152))
    ref = P.lrq_rotate_quantize_act(X, P.ROT_HADAMARD, 8, 128)
    got = P.lrq_rotate_quantize_act_static(X, P.ROT_HADAMARD, 8, 128)
    torch.cuda.synchronize()
    for g, r in zip(got, ref):
        assert torch.equal(g, r)
    # one token too many for the fixed array: refused with the workspace status, nothing launched
    K = 1024
    M = P.lrq_static_scratch_bytes() // (4 * K) + 1
    Xb = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    Rb = torch.zeros((K, K), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.LrqError) as e:
        P.lrq_rotate_quantize_act_static(Xb, P.ROT_DENSE, 8, R=Rb)
    assert e.value.code == 3
    out = P.lrq_rotate_quantize_act_static(Xb[:-1], P.ROT_DENSE, 8, R=Rb)   # exactly at the limit
    torch.cuda.synchronize()
    assert int(out[2].abs().max()) == 0


def test_static_scratch_serves_the_dual_transformation(P):
    # kind DUAL needs 10 bytes of scratch per element (fp32 rotated values and three bf16 panels)
    from lrq_workloads import LayerSpec
    spec = LayerSpec("dual", 17, 300, 384, 8, 4, 8, 0, "dual", 128, n_salient=8)
    dual = PU.dual_to_device(P, spec.dual_factors())
    X = PU.bf16_to_device(spec.activations())
    ref = P.lrq_rotate_quantize_act(X, P.ROT_DUAL, 8, dual=dual)
    got = P.lrq_rotate_quantize_act_static(X, P.ROT_DUAL, 8, dual=dual)
    torch.cuda.synchronize()
    for g, r in zip(got, ref):
        assert torch.equal(g, r)
    M = P.lrq_static_scratch_bytes() // (10 * 384) + 2
    with pytest.raises(P.LrqError) as e:
        P.lrq_rotate_quantize_act_static(torch.zeros((M, 384), dtype=torch.bfloat16, device="cuda"), P.ROT_DUAL, 8, dual=dual)
    assert e.value.code == 3
