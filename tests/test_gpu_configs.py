"""GPU parity at the full workload sizes, in the launch configuration the bench times: every layer is
run in full through lrq_qlinear; activation codes are compared for all tokens where the oracle's rotation is
cheap (Hadamard) and for sampled tokens otherwise; outputs are compared on sampled token rows; TLQ codes and
tables on sampled weight rows."""
import numpy as np
import pytest
import torch

import parity as PU
from lrq_workloads import bf16_bits_to_f64, config_layers

pytestmark = pytest.mark.gpu

N_TOK = 256      # sampled token rows per layer
N_ROW = 192      # sampled weight rows per layer


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2508_03485_b200 as P
    P.load_library()
    return P


def _run_layer(P, orc, spec, M=None):
    rng = np.random.default_rng(spec.seed)
    W, xb = spec.weights(), spec.activations(M)
    M = xb.shape[0]
    layer, tl = PU.gpu_layer(spec, W, P)
    rows = np.sort(rng.choice(spec.N, size=min(N_ROW, spec.N), replace=False))
    # oracle TLQ on sampled rows; the contraction below then only yields those output columns
    T = PU.check_tlq(orc, W, tl, spec.w_bits, spec.group, rows=rows, what=spec.name)
    X = PU.bf16_to_device(xb)
    Y = P.lrq_qlinear(layer, X, P.F32)
    assert P.lrq_device_status() == 0
    toks = np.sort(rng.choice(M, size=min(N_TOK, M), replace=False))
    Rb = spec.rotation_bf16()
    Yo, oq, os_, oz = PU.oracle_layer_rows(orc, spec, xb[toks], T, Rb)
    Yg = Y[torch.from_numpy(toks).cuda()][:, torch.from_numpy(rows).cuda()].cpu().numpy()
    # activation codes of the same input through lrq_rotate_quantize_act (same kernels as inside lrq_qlinear)
    q, s, z = P.lrq_rotate_quantize_act(X, layer.kind, spec.a_bits, spec.had_block, layer.R)
    qn = PU.act_codes_to_numpy(q[torch.from_numpy(toks).cuda()], spec.a_bits)
    gz = z.cpu().numpy()[toks]
    frac, zf = PU.check_act(qn, s.cpu().numpy()[toks], gz, oq, os_, oz, spec.name)
    fro, mabs, nbound = PU.check_layer_out(orc, spec, T, Yg, qn, gz, Yo, oq, os_, oz, spec.name)
    print(f"{spec.name}: rel_fro={fro:.2e} maxabs/rms={mabs:.2e} code_flips={frac:.2e} z_flips={zf} boundary_tokens={nbound}")
    layer.close()
    return fro, mabs, frac, zf


def test_config0_all_tokens(P, orc):
    spec = config_layers(0)[0]
    W, xb = spec.weights(), spec.activations()
    layer, tl = PU.gpu_layer(spec, W, P)
    T = PU.check_tlq(orc, W, tl, spec.w_bits, spec.group, what="cfg0")
    Yo, oq, os_, oz = PU.oracle_layer_rows(orc, spec, xb, T)
    X = PU.bf16_to_device(xb)
    Y = P.lrq_qlinear(layer, X, P.F32)
    q, s, z = P.lrq_rotate_quantize_act(X, P.ROT_HADAMARD, 4, 1024)
    gq, gz = PU.act_codes_to_numpy(q, 4), z.cpu().numpy()
    PU.check_act(gq, s.cpu().numpy(), gz, oq, os_, oz, "cfg0")
    PU.check_layer_out(orc, spec, T, Y.cpu().numpy(), gq, gz, Yo, oq, os_, oz, "cfg0")


@pytest.mark.parametrize("i", range(4))
def test_config1_layers(P, orc, i):
    _run_layer(P, orc, config_layers(1)[i])


@pytest.mark.parametrize("i", range(4))
def test_config2_layers(P, orc, i):
    _run_layer(P, orc, config_layers(2)[i])


@pytest.mark.parametrize("i", range(3))
def test_config3_layers(P, orc, i):
    _run_layer(P, orc, config_layers(3)[i])


def test_config4_sampled_layers(P, orc):
    # all four shapes and both rotation kinds of the video-DiT stack, at the stack's M
    layers = config_layers(4)
    dense = [l for l in layers if l.rot == "dense"]
    pick = layers[:4] + dense[:1]
    assert {l.name.split(".")[1] for l in pick} >= {"qkv", "proj", "fc1", "fc2"} and dense
    for spec in pick:
        _run_layer(P, orc, spec)
