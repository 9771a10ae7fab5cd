"""GPU parity at the full workload sizes, in the launch configuration the bench times.

Single layers (workloads 0-3): each layer runs in full through lrq_qlinear; TLQ codes and tables are compared for
every weight; activation codes, scales and zero-points for sampled tokens (all tokens for workload 0); outputs on
the sampled token rows over all N output columns, which the oracle computes one row at a time (tokens are
independent).

The stack (workload 4): one lrq_qlinear_stack call over the 112 layers with one shared workspace, as the bench
issues it; TLQ results of every layer against the oracle; activation codes of every distinct (activations,
rotation) pair, all tokens for the Hadamard layers and sampled tokens for the dense ones; outputs of a seeded
subset of layers (all four shapes, both rotation kinds, first and last block) on sampled token rows, read from
the buffers the stack call itself wrote."""
import numpy as np
import pytest
import torch

import parity as PU
from lrq_workloads import bf16_bits_to_f64, config_layers

pytestmark = pytest.mark.gpu

N_TOK = 256      # sampled token rows per layer


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
    T = PU.check_tlq(orc, W, tl, spec.w_bits, spec.group, what=spec.name)      # every row, no tie exemption
    X = PU.bf16_to_device(xb)
    Y = P.lrq_qlinear(layer, X, P.F32)
    assert P.lrq_device_status() == 0
    toks = np.sort(rng.choice(M, size=min(N_TOK, M), replace=False))
    Rb = spec.rotation_bf16()
    Yo, oq, os_, oz, Yr = PU.oracle_layer_rows(orc, spec, xb[toks], T, Rb)
    Yg = Y[torch.from_numpy(toks).cuda()].cpu().numpy()
    # activation codes of the same input through lrq_rotate_quantize_act (same kernels as inside lrq_qlinear)
    q, s, z = P.lrq_rotate_quantize_act(X, layer.kind, spec.a_bits, spec.had_block, layer.R)
    qn = PU.act_codes_to_numpy(q[torch.from_numpy(toks).cuda()], spec.a_bits)
    gz = z.cpu().numpy()[toks]
    act = PU.check_act(qn, s.cpu().numpy()[toks], gz, oq, os_, oz, Yr, spec.rot, spec.had_block, spec.name)
    fro, mabs, nbound = PU.check_layer_out(orc, T, Yg, qn, gz, Yo, os_, act, spec.name)
    print(f"{spec.name}: rel_fro={fro:.2e} maxabs/rms={mabs:.2e} code_flips={act.flip_fraction:.2e} ties={act.tie_fraction:.2e} "
          f"z_flips={act.z_flips} boundary_tokens={nbound} worst_boundary={act.worst_boundary:.2f} worst_scale={act.worst_scale:.2f}")
    layer.close()


def test_config0_all_tokens(P, orc):
    spec = config_layers(0)[0]
    W, xb = spec.weights(), spec.activations()
    layer, tl = PU.gpu_layer(spec, W, P)
    T = PU.check_tlq(orc, W, tl, spec.w_bits, spec.group, what="cfg0")
    Yo, oq, os_, oz, Yr = PU.oracle_layer_rows(orc, spec, xb, T)
    X = PU.bf16_to_device(xb)
    Y = P.lrq_qlinear(layer, X, P.F32)
    q, s, z = P.lrq_rotate_quantize_act(X, P.ROT_HADAMARD, 4, 1024)
    gq, gz = PU.act_codes_to_numpy(q, 4), z.cpu().numpy()
    act = PU.check_act(gq, s.cpu().numpy(), gz, oq, os_, oz, Yr, "hadamard", 1024, "cfg0")
    PU.check_layer_out(orc, T, Y.cpu().numpy(), gq, gz, Yo, os_, act, "cfg0")


@pytest.mark.parametrize("i", range(4))
def test_config1_layers(P, orc, i):
    _run_layer(P, orc, config_layers(1)[i])


@pytest.mark.parametrize("i", range(4))
def test_config2_layers(P, orc, i):
    _run_layer(P, orc, config_layers(2)[i])


@pytest.mark.parametrize("i", range(3))
def test_config3_layers(P, orc, i):
    _run_layer(P, orc, config_layers(3)[i])


def test_config4_stack_against_oracle(P, orc):
    specs = config_layers(4)
    rng = np.random.default_rng(12)
    dense_idx = [i for i, s in enumerate(specs) if s.rot == "dense"]
    assert dense_idx, "the seeded draw of workload 4 has dense-rotation layers"
    # layers whose outputs are compared: first and last block, every dense layer, one more of each shape
    checked = sorted(set(list(range(4)) + list(range(len(specs) - 4, len(specs))) + dense_idx +
                         [4 * int(b) + j for j, b in enumerate(rng.choice(np.arange(1, 27), size=4, replace=False))]))
    assert {specs[i].name.split(".")[1] for i in checked} == {"qkv", "proj", "fc1", "fc2"}
    M = specs[0].M

    # one activation buffer per distinct K, shared by every layer of that K (as the bench does)
    xbits, Xdev = {}, {}
    for s in specs:
        if s.K not in xbits:
            xbits[s.K] = s.activations()
            Xdev[s.K] = PU.bf16_to_device(xbits[s.K])

    layers, tls, oracle_T = [], [], {}
    for i, s in enumerate(specs):
        W = s.weights()
        layer, tl = PU.gpu_layer(s, W, P)
        T = PU.check_tlq(orc, W, tl, s.w_bits, s.group, what=s.name)           # every weight of every layer
        if i in checked:
            oracle_T[i] = T
        layers.append(layer); tls.append(tl)
        del W

    # outputs: checked layers own a buffer; the others share one per N (their results are overwritten, as in the bench)
    shared, Ys = {}, []
    for i, s in enumerate(specs):
        if i in checked:
            Ys.append(torch.empty((M, s.N), dtype=torch.float32, device="cuda"))
        else:
            if s.N not in shared:
                shared[s.N] = torch.empty((M, s.N), dtype=torch.float32, device="cuda")
            Ys.append(shared[s.N])
    Xs = [Xdev[s.K] for s in specs]
    plan = P.StackPlan(layers, Xs, Ys, P.F32)
    ws = torch.empty(plan.need, dtype=torch.uint8, device="cuda")
    P.lrq_qlinear_stack(plan, ws)                      # the one call under test
    torch.cuda.synchronize()
    assert P.lrq_device_status() == 0

    toks = np.sort(rng.choice(M, size=N_TOK, replace=False))
    tok_dev = torch.from_numpy(toks).cuda()

    # activation codes of every distinct (activations, rotation): Hadamard pairs over all tokens, in chunks
    for K in sorted(xbits):
        s = next(sp for sp in specs if sp.K == K and sp.rot == "hadamard")
        q, sc, z = P.lrq_rotate_quantize_act(Xdev[K], P.ROT_HADAMARD, s.a_bits, s.had_block)
        gs, gz = sc.cpu().numpy(), z.cpu().numpy()
        flips = 0.0
        for m0 in range(0, M, 4096):
            sl = slice(m0, min(M, m0 + 4096))
            Yr = orc.rotate_hadamard_fwht(bf16_bits_to_f64(xbits[K][sl]), s.had_block)
            oq, os_, oz = orc.quantize_act(Yr, s.a_bits)
            r = PU.check_act(PU.act_codes_to_numpy(q[sl], s.a_bits), gs[sl], gz[sl], oq, os_, oz, Yr, "hadamard", s.had_block,
                             f"cfg4 K={K} tokens {m0}..")
            flips = max(flips, r.flip_fraction)
        print(f"cfg4 activations K={K}: all {M} tokens, worst chunk flip fraction {flips:.2e}")

    # outputs of the checked layers, from the buffers the stack call wrote
    for i in checked:
        s, T = specs[i], oracle_T[i]
        Rb = s.rotation_bf16()
        Yo, oq, os_, oz, Yr = PU.oracle_layer_rows(orc, s, xbits[s.K][toks], T, Rb)
        q, sc, z = P.lrq_rotate_quantize_act(Xdev[s.K], layers[i].kind, s.a_bits, s.had_block, layers[i].R)
        qn = PU.act_codes_to_numpy(q[tok_dev], s.a_bits)
        gz = z.cpu().numpy()[toks]
        act = PU.check_act(qn, sc.cpu().numpy()[toks], gz, oq, os_, oz, Yr, s.rot, s.had_block, s.name)
        fro, mabs, nb = PU.check_layer_out(orc, T, Ys[i][tok_dev].cpu().numpy(), qn, gz, Yo, os_, act, f"cfg4 stack {s.name}")
        print(f"cfg4 stack {s.name} ({s.rot}): rel_fro={fro:.2e} maxabs/rms={mabs:.2e} flips={act.flip_fraction:.2e} "
              f"boundary_tokens={nb} worst_boundary={act.worst_boundary:.2f}")
    for layer in layers:
        layer.close()
