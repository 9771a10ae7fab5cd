"""GPU parity: every step of the CUDA path, called through the C ABI, against the fp64 oracle on the same
seeded inputs.  Small shapes are compared element by element (several tiles plus a ragged tail); the
full-size workload layers are run in full on the GPU and compared on sampled token rows, which the oracle
computes one by one (tokens are independent)."""
import numpy as np
import pytest
import torch

import parity as PU
from lrq_workloads import (LayerSpec, bf16_bits_to_f64, config_layers, default_clip_grid, f32_to_bf16_bits,
                           make_activations, make_orthogonal, make_weights)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2508_03485_b200 as P
    P.load_library()
    return P


# --------------------------------------------------------------------------------------------- rotq
@pytest.mark.parametrize("M,K,B,a_bits,mode", [
    (1, 128, 128, 8, 0), (7, 1152, 128, 8, 0), (129, 1024, 1024, 4, 0), (33, 1536, 512, 4, 0),
    (5, 6144, 2048, 4, 0), (3, 12288, 4096, 4, 0), (17, 3072, 1024, 4, 1), (64, 4608, 128, 8, 1),
    (9, 64, 8, 8, 0), (12, 256, 16, 4, 0), (300, 1152, 128, 4, 0), (2, 512, 64, 8, 0),
    # large blocks (register-butterfly kernel): 8-bit codes, several blocks per token, several groups per CTA
    (4001, 1024, 1024, 8, 0), (70, 2048, 2048, 8, 0), (130, 8192, 4096, 8, 1), (257, 2048, 1024, 4, 0),
])
def test_rotate_quantize_hadamard(P, orc, M, K, B, a_bits, mode):
    xb = make_activations(100 + M + K, M, K)
    q, s, z = P.lrq_rotate_quantize_act(PU.bf16_to_device(xb), P.ROT_HADAMARD, a_bits, B, mode=mode)
    Yr = orc.rotate_hadamard_fwht(bf16_bits_to_f64(xb), B)
    oq, os_, oz = orc.quantize_act(Yr, a_bits, mode)
    PU.check_act(PU.act_codes_to_numpy(q, a_bits), s.cpu().numpy(), z.cpu().numpy(), oq, os_, oz, Yr, "hadamard", B,
                 f"rotq {M}x{K} B{B}")


def test_rotate_quantize_edge_tokens(P, orc):
    # constant token, all-zero token, a single spike (Lemma 1), values at the bf16 extremes of the workload
    K, B = 256, 128
    x = np.zeros((5, K), dtype=np.float32)
    x[0] = 2.0
    x[2, 37], x[2, 0], x[2, 128] = 245.0, 100.0, 100.0   # spike plus an offset: a symmetric range would put every
    x[3] = np.linspace(-300, 200, K)                      # element exactly on a rounding boundary (min/s = -7.5)
    x[4, ::2] = 1.0
    xb = f32_to_bf16_bits(x)
    for a_bits in (4, 8):
        q, s, z = P.lrq_rotate_quantize_act(PU.bf16_to_device(xb), P.ROT_HADAMARD, a_bits, B)
        Yr = orc.rotate_hadamard_fwht(bf16_bits_to_f64(xb), B)
        oq, os_, oz = orc.quantize_act(Yr, a_bits)
        PU.check_act(PU.act_codes_to_numpy(q, a_bits), s.cpu().numpy(), z.cpu().numpy(), oq, os_, oz, Yr, "hadamard", B, "edge")
        assert s[1].item() == 1.0 and z[1].item() == 0          # empty range: unit step


def test_rotate_quantize_strided_rows_and_no_rotation(P, orc):
    M, K = 20, 384
    xb = make_activations(5, M, 512)
    xd = PU.bf16_to_device(xb)[:, :K]                          # ldx = 512 > K
    q, s, z = P.lrq_rotate_quantize_act(xd, P.ROT_NONE, 8)
    Yn = bf16_bits_to_f64(xb[:, :K])
    oq, os_, oz = orc.quantize_act(Yn, 8)
    # Without a rotation the inputs sit on the coarse bf16 grid, where x/s lands exactly on a rounding boundary
    # for a visible share of the elements.  Those are exact ties (the oracle's own choice there is decided by the
    # last bit of its fp64 s): check_act verifies each differing element is one, and does not count exact ties
    # against the 1e-4 allowance; everything else gets the ordinary allowance.
    r = PU.check_act(PU.act_codes_to_numpy(q, 8), s.cpu().numpy(), z.cpu().numpy(), oq, os_, oz, Yn, "none", 0, "none")
    assert r.tie_fraction <= 5e-3
    q, s, z = P.lrq_rotate_quantize_act(xd, P.ROT_HADAMARD, 4, 128)
    Yr = orc.rotate_hadamard_fwht(Yn, 128)
    oq, os_, oz = orc.quantize_act(Yr, 4)
    PU.check_act(PU.act_codes_to_numpy(q, 4), s.cpu().numpy(), z.cpu().numpy(), oq, os_, oz, Yr, "hadamard", 128, "strided")


@pytest.mark.parametrize("M,K,a_bits", [(70, 192, 4), (130, 1152, 8), (33, 1536, 4),
                                        # ragged shapes of the tensor-core rotation: K not a multiple of the 64-deep
                                        # k-block (last block zero-filled by TMA) nor of the 32-column epilogue chunk
                                        (130, 136, 4), (130, 136, 8), (130, 200, 4), (130, 200, 8)])
def test_rotate_quantize_dense(P, orc, M, K, a_bits):
    xb = make_activations(7, M, K, n_salient=16, salient_x=100.0)
    Rb = f32_to_bf16_bits(make_orthogonal(3, K).astype(np.float32))
    q, s, z = P.lrq_rotate_quantize_act(PU.bf16_to_device(xb), P.ROT_DENSE, a_bits, R=PU.bf16_to_device(Rb))
    Yr = orc.rotate_dense(bf16_bits_to_f64(xb), bf16_bits_to_f64(Rb))
    oq, os_, oz = orc.quantize_act(Yr, a_bits)
    PU.check_act(PU.act_codes_to_numpy(q, a_bits), s.cpu().numpy(), z.cpu().numpy(), oq, os_, oz, Yr, "dense", 0, "dense")


# --------------------------------------------------------------------------------------------- tlqw
@pytest.mark.parametrize("N,K,bits,G", [(16, 128, 3, 0), (33, 1152, 4, 0), (8, 1536, 3, 128), (5, 4608, 4, 0),
                                        (3, 12288, 4, 0), (64, 256, 2, 64), (7, 64, 4, 8)])
def test_tlq_quantize_weights(P, orc, N, K, bits, G):
    W = make_weights(200 + N + K, N, K)
    W[0, :3] = 0.0
    g = default_clip_grid()
    tl = P.lrq_tlq_quantize_weights(torch.from_numpy(W).cuda(), bits, G, 7, g, g)
    PU.check_tlq(orc, W, tl, bits, G, what=f"tlq {N}x{K} b{bits} G{G}")


def test_tlq_degenerate_rows(P, orc):
    W = np.zeros((4, 64), dtype=np.float32)
    W[1] = 0.25
    W[2, ::2], W[2, 1::2] = 0.5, -0.125
    W[3] = -np.abs(make_weights(1, 1, 64)[0])
    tl = P.lrq_tlq_quantize_weights(torch.from_numpy(W).cuda(), 3, 0, 7, [1.0, 1.2], [1.0, 1.2])
    T = orc.tlq_quantize(W.astype(np.float64), 3, 0, 7, [1.0, 1.2], [1.0, 1.2])
    assert np.array_equal(PU.unpack4(tl.codes.cpu().numpy()).astype(np.int32) - 4, T.codes.astype(np.int32))
    assert np.array_equal(tl.levels.cpu().numpy().astype(np.float64), T.levels)


# --------------------------------------------------------------------------------------------- qgemm
def _small_layer(P, orc, M, K, N, w_bits, a_bits, G, B, seed, rot="hadamard"):
    spec = LayerSpec("t", seed, M, K, N, w_bits, a_bits, G, rot, B)
    W, xb = spec.weights(), spec.activations()
    layer, tl = PU.gpu_layer(spec, W, P)
    T = PU.check_tlq(orc, W, tl, w_bits, G, what="small layer")
    return spec, W, xb, layer, tl, T


@pytest.mark.parametrize("impl", [1, 0, 2, 3])
@pytest.mark.parametrize("M,K,N,w_bits,a_bits,G,B", [
    (70, 256, 72, 4, 8, 0, 128), (129, 1152, 200, 4, 8, 0, 128), (33, 512, 136, 3, 4, 128, 512),
    (256, 1024, 1024, 3, 4, 0, 1024), (5, 128, 8, 4, 4, 64, 64),
])
def test_qgemm_from_oracle_codes(P, orc, impl, M, K, N, w_bits, a_bits, G, B):
    # the contraction alone: the GPU gets the oracle's activation codes, so only Eq. 10 is compared
    spec, W, xb, layer, tl, T = _small_layer(P, orc, M, K, N, w_bits, a_bits, G, B, 31)
    Yo, oq, os_, oz, _ = PU.oracle_layer_rows(orc, spec, xb, T)
    if a_bits == 8:
        qd = torch.from_numpy(oq.astype(np.uint8)).cuda()
    else:
        qd = torch.from_numpy((oq[:, 0::2] | (oq[:, 1::2] << 4)).astype(np.uint8)).cuda()
    sd = torch.from_numpy(os_.astype(np.float32)).cuda()
    zd = torch.from_numpy(oz.astype(np.int32)).cuda()
    try:
        Y = P.lrq_qgemm_codes(layer, qd, sd, zd, P.F32, impl)
    except P.LrqError as e:
        if impl in (0, 2) and e.code == 2:
            pytest.skip("shape not taken by this tensor-core kernel")
        raise
    assert P.lrq_device_status() == 0
    fro, _ = PU.check_out(Y.cpu().numpy(), Yo, f"qgemm impl{impl}", rel=1e-5, mx=1e-4)
    if impl == 3:
        # the integer form of Eq. 10 sums exactly; what is left is the fp32 rounding of the sum, of the stored row sums
        # that the zero-point term multiplies (acc and z * wsum partly cancel) and of the epilogue's products
        assert fro <= 1e-6, fro


@pytest.mark.parametrize("M,K,N,w_bits,a_bits,G,B,rot", [
    (70, 256, 72, 4, 8, 0, 128, "hadamard"), (300, 1152, 392, 4, 8, 0, 128, "hadamard"),
    (129, 1536, 264, 3, 4, 128, 512, "hadamard"), (65, 384, 136, 3, 4, 128, 0, "dense"),
])
def test_qlinear_small(P, orc, M, K, N, w_bits, a_bits, G, B, rot):
    spec, W, xb, layer, tl, T = _small_layer(P, orc, M, K, N, w_bits, a_bits, G, B, 41, rot)
    Rb = spec.rotation_bf16()
    Yo, oq, os_, oz, Yr = PU.oracle_layer_rows(orc, spec, xb, T, Rb)
    X = PU.bf16_to_device(xb)
    q, s, z = P.lrq_rotate_quantize_act(X, layer.kind, a_bits, B, layer.R)
    gq, gz = PU.act_codes_to_numpy(q, a_bits), z.cpu().numpy()
    act = PU.check_act(gq, s.cpu().numpy(), gz, oq, os_, oz, Yr, rot, B, "qlinear codes")
    Y = P.lrq_qlinear(layer, X, P.F32)
    PU.check_layer_out(orc, T, Y.cpu().numpy(), gq, gz, Yo, os_, act, "qlinear f32")
    Yh = P.lrq_qlinear(layer, X, P.F16)
    PU.check_layer_out(orc, T, Yh.float().cpu().numpy(), gq, gz, Yo, os_, act, "qlinear f16")
    Yb = P.lrq_qlinear(layer, X, P.BF16).float().cpu().numpy()
    # bf16 output: the fp32 result rounded to bf16 (half an ulp = 2^-9 relative)
    Yf = Y.cpu().numpy().astype(np.float64)
    assert (np.abs(Yb - Yf) <= np.abs(Yf) * 2.0 ** -8).all()
    assert P.lrq_device_status() == 0


def test_qlinear_scale_and_bias(P, orc):
    spec, W, xb, layer, tl, T = _small_layer(P, orc, 40, 256, 96, 4, 8, 0, 128, 43)
    rng = np.random.default_rng(0)
    ws, bs = rng.uniform(0.5, 2, 96).astype(np.float32), rng.standard_normal(96).astype(np.float32)
    layer2 = P.QLayer(tl, 96, 256, P.ROT_HADAMARD, 8, 128, wscale=torch.from_numpy(ws).cuda(),
                      bias=torch.from_numpy(bs).cuda())
    X = bf16_bits_to_f64(xb)
    Yo, *_ = orc.qlinear(X, T, 8, "hadamard", 128, wscale=ws.astype(np.float64), bias=bs.astype(np.float64))
    Y = P.lrq_qlinear(layer2, PU.bf16_to_device(xb), P.F32)
    PU.check_out(Y.cpu().numpy(), Yo, "scale+bias")


def test_qlinear_stack_matches_single_calls(P):
    specs = [LayerSpec("a", 51, 64, 256, 72, 4, 8, 0, "hadamard", 128),
             LayerSpec("b", 52, 48, 512, 40, 3, 4, 128, "hadamard", 512),
             LayerSpec("c", 53, 33, 128, 136, 4, 8, 0, "dense", 0)]
    layers, Xs, Ys, refs = [], [], [], []
    for sp in specs:
        layer, _ = PU.gpu_layer(sp, sp.weights(), P)
        X = PU.bf16_to_device(sp.activations())
        layers.append(layer); Xs.append(X)
        refs.append(P.lrq_qlinear(layer, X, P.F32))
        Ys.append(torch.zeros_like(refs[-1]))
    plan = P.StackPlan(layers, Xs, Ys, P.F32)
    P.lrq_qlinear_stack(plan)
    torch.cuda.synchronize()
    for y, r in zip(Ys, refs):
        assert torch.equal(y, r)


# ------------------------------------------------------------------ tensor-core kernel at full size
@pytest.mark.parametrize("cfg,li", [(1, 0), (2, 0), (3, 1)])
def test_qgemm_tensor_core_matches_cuda_core_everywhere(P, cfg, li):
    # Every output element of the tcgen05 kernel against the plain CUDA-core kernel of the same library on a
    # full-size workload layer: several tiles per CTA pair, grouped and per-channel tables, 4- and 8-bit codes.
    # The oracle checks sampled rows elsewhere; this one looks at all of them, twice (a hand-over race
    # between the kernel's warps shows up as a few wrong tiles that differ from run to run).
    spec = config_layers(cfg)[li]
    layer, tl = PU.gpu_layer(spec, spec.weights(), P)
    X = PU.bf16_to_device(spec.activations())
    kind = P.ROT_HADAMARD
    q, s, z = P.lrq_rotate_quantize_act(X, kind, spec.a_bits, spec.had_block)
    ref = P.lrq_qgemm_codes(layer, q, s, z, P.F32, 1)
    first = None
    for _ in range(3):
        Y = P.lrq_qgemm_codes(layer, q, s, z, P.F32, 0)
        torch.cuda.synchronize()
        assert P.lrq_device_status() == 0
        rms = ref.pow(2).mean().sqrt()
        assert ((Y - ref).abs().max() / rms).item() <= 2e-3          # fp32 summation order only
        if first is None:
            first = Y.clone()
        else:
            assert torch.equal(Y, first)                             # fixed accumulation order: bit-identical
    layer.close()


def test_qlinear_stack_replays_from_a_cuda_graph(P):
    # The stack is a fixed sequence of launches (kernels with by-value tensor maps, two memsets for a dense
    # rotation): captured once, replayed on new activations, it must give what direct calls give.
    specs = [LayerSpec("a", 61, 200, 1152, 264, 4, 8, 0, "hadamard", 128),
             LayerSpec("b", 62, 130, 512, 136, 3, 4, 128, "dense", 0)]
    layers, Xs, Ys = [], [], []
    for sp in specs:
        layer, _ = PU.gpu_layer(sp, sp.weights(), P)
        layers.append(layer)
        Xs.append(PU.bf16_to_device(sp.activations()))
        Ys.append(torch.zeros((sp.M, sp.N), dtype=torch.float32, device="cuda"))
    plan = P.StackPlan(layers, Xs, Ys, P.F32)
    ws = torch.empty(plan.need, dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        P.lrq_qlinear_stack(plan, ws)                # first-call set-up happens outside the capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        P.lrq_qlinear_stack(plan, ws)
    for seed in (71, 72):
        for sp, X in zip(specs, Xs):
            X.copy_(PU.bf16_to_device(make_activations(seed, sp.M, sp.K, n_salient=8 if sp.rot == "dense" else 0)))
        g.replay()
        torch.cuda.synchronize()
        for layer, X, Y in zip(layers, Xs, Ys):
            assert torch.equal(Y, P.lrq_qlinear(layer, X, P.F32))
    assert P.lrq_device_status() == 0


# --------------------------------------------------------------------------------- smoothing, ARS metric
@pytest.mark.parametrize("M,K,B,a_bits", [(40, 1152, 128, 8), (33, 1536, 512, 4), (9, 72, 8, 8), (5, 6144, 2048, 4)])
def test_rotate_quantize_with_smoothing(P, orc, M, K, B, a_bits):
    # Sec. 5.1: channel-wise multipliers applied before the rotation (fast and generic kernels)
    xb = make_activations(300 + K, M, K, n_salient=8, salient_x=60.0)
    rng = np.random.default_rng(K)
    p = (1.0 / np.sqrt(np.abs(bf16_bits_to_f64(xb)).max(axis=0) + 1e-3) * rng.uniform(0.8, 1.25, K)).astype(np.float32)
    q, s, z = P.lrq_rotate_quantize_act(PU.bf16_to_device(xb), P.ROT_HADAMARD, a_bits, B,
                                        prescale=torch.from_numpy(p).cuda())
    Yr = orc.rotate_hadamard_fwht(orc.smooth(bf16_bits_to_f64(xb), p.astype(np.float64)), B)
    oq, os_, oz = orc.quantize_act(Yr, a_bits)
    PU.check_act(PU.act_codes_to_numpy(q, a_bits), s.cpu().numpy(), z.cpu().numpy(), oq, os_, oz, Yr, "hadamard", B,
                 f"smooth {M}x{K}")


def test_smoothing_is_refused_for_a_dense_rotation(P):
    X = torch.zeros((8, 128), dtype=torch.bfloat16, device="cuda")
    R = torch.zeros((128, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.LrqError) as e:
        P.lrq_rotate_quantize_act(X, P.ROT_DENSE, 8, R=R, prescale=torch.ones(128, device="cuda"))
    assert e.value.code == 2


@pytest.mark.parametrize("M,K,n_sal,thr", [(256, 1152, 0, 1.0), (300, 1536, 16, 1.0), (4096, 4608, 0, 1.0), (17, 64, 2, 5.0)])
def test_ars_metric_and_choice(P, orc, M, K, n_sal, thr):
    # Eq. 11 / Eq. 12 against the oracle; tolerance 1e-6: squares of bf16 are exact in fp32 and at most 16 of them
    # are summed in fp32 (relative error below 16 * 2^-24) before everything goes on in fp64
    xb = make_activations(400 + K, M, K, n_salient=n_sal, salient_x=100.0)
    J, kind = P.lrq_ars_select(PU.bf16_to_device(xb), thr)
    Jo, ko = orc.fluctuation_metric(bf16_bits_to_f64(xb), thr)
    assert abs(J.item() - Jo) <= 1e-6 * Jo
    assert abs(Jo - thr) > 1e-4 * thr and kind.item() == ko


# ------------------------------------------------------------------------------- layouts and edges
@pytest.mark.parametrize("dt", ["F32", "F16", "BF16"])
def test_qlinear_strided_input_and_output(P, dt):
    # X and Y as column slices of wider buffers (ldx > K, ldy > N; N = 264 ends inside a 32- and a 64-column store
    # tile): the TMA store path must honour ldy and must not touch the columns beside Y
    code = getattr(P, dt)
    tdt = {"F32": torch.float32, "F16": torch.float16, "BF16": torch.bfloat16}[dt]
    spec = LayerSpec("s", 81, 300, 512, 264, 4, 8, 0, "hadamard", 128)
    layer, _ = PU.gpu_layer(spec, spec.weights(), P)
    Xc = PU.bf16_to_device(spec.activations())
    ref = P.lrq_qlinear(layer, Xc, code)
    Xw = torch.zeros((300, 640), dtype=torch.bfloat16, device="cuda")
    Xw[:, 64:576] = Xc
    Yw = torch.full((300, 320), -7.0, dtype=tdt, device="cuda")
    out = P.lrq_qlinear(layer, Xw[:, 64:576], code, out=Yw[:, 32:296])
    torch.cuda.synchronize()
    assert torch.equal(out, ref)
    assert (Yw[:, :32] == -7.0).all() and (Yw[:, 296:] == -7.0).all()
    assert P.lrq_device_status() == 0


@pytest.mark.parametrize("M", [1, 127, 128, 129, 257])
def test_qlinear_token_counts_around_a_tile(P, M):
    # one token, and counts just below / at / above the 128-row CTA tile and the 256-row pair tile; the rows of
    # a larger batch are independent, so each must equal the first M rows of the M = 300 result
    spec = LayerSpec("m", 82, 300, 256, 264, 3, 4, 128, "hadamard", 256)
    layer, _ = PU.gpu_layer(spec, spec.weights(), P)
    X = PU.bf16_to_device(spec.activations())
    full = P.lrq_qlinear(layer, X, P.F32)
    part = P.lrq_qlinear(layer, X[:M].contiguous(), P.F32)
    torch.cuda.synchronize()
    assert torch.equal(part, full[:M])
    assert P.lrq_device_status() == 0


@pytest.mark.parametrize("N,K,rot,B,smooth", [(37, 1152, "hadamard", 128, True), (5, 12288, "hadamard", 4096, False),
                                              (70, 384, "dense", 0, True), (130, 200, "dense", 0, False),
                                              (9, 72, "none", 0, True), (16, 1536, "hadamard", 512, True)])
def test_rotate_weights(P, orc, N, K, rot, B, smooth):
    # W diag(colmul) R (Eq. 2, weight side; Sec. 5.1) against the oracle.  Both evaluate in fp64 and differ only in
    # summation order (1e-13 relative); after the one rounding to fp32 that shows as at most one ulp, and only
    # where the fp64 value sits next to a rounding boundary.
    rng = np.random.default_rng(N + K)
    W = make_weights(31, N, K)
    c = rng.uniform(0.3, 3.0, K).astype(np.float32) if smooth else None
    R = Rb = None
    if rot == "dense":
        Rb = f32_to_bf16_bits(make_orthogonal(7, K).astype(np.float32))
        R = PU.bf16_to_device(Rb)
    kind = {"hadamard": P.ROT_HADAMARD, "dense": P.ROT_DENSE, "none": P.ROT_NONE}[rot]
    out = P.lrq_rotate_weights(torch.from_numpy(W).cuda(), kind, B, R, None if c is None else torch.from_numpy(c).cuda())
    ref = orc.rotate_weights(W.astype(np.float64), None if c is None else c.astype(np.float64), rot, B,
                             None if Rb is None else bf16_bits_to_f64(Rb))
    got = out.cpu().numpy()
    ref32 = ref.astype(np.float32)
    ulp = np.spacing(np.abs(ref32)).astype(np.float64)
    assert (np.abs(got.astype(np.float64) - ref) <= 0.5 * ulp + 1e-12 * np.abs(ref).max()).all()
    assert (got != ref32).mean() < 1e-3
    if rot == "hadamard":          # in place is allowed for this kind
        Wd = torch.from_numpy(W).cuda()
        P.lrq_rotate_weights(Wd, kind, B, None, None if c is None else torch.from_numpy(c).cuda(), out=Wd)
        assert torch.equal(Wd, out)


def test_rotated_and_smoothed_layer_reproduces_the_plain_product(P):
    # End to end on the GPU: weights rotated by lrq_rotate_weights with colmul = 1/p, activations smoothed by p and
    # rotated inside lrq_qlinear.  With 8-bit activations and 4-bit TLQ the result is a quantized estimate of X W^T;
    # its error must be that of the quantizers (a few per cent of the output scale), far from what a mismatch of
    # the two sides of Eq. 2 would give (order one).
    rng = np.random.default_rng(3)
    M, K, N, B = 200, 1152, 264, 128
    W = make_weights(51, N, K)
    xb = make_activations(52, M, K)
    X = bf16_bits_to_f64(xb)
    p = (1.0 / np.sqrt(np.abs(X).max(axis=0) + 1e-3)).astype(np.float32)
    Wr = P.lrq_rotate_weights(torch.from_numpy(W).cuda(), P.ROT_HADAMARD, B, None, torch.from_numpy(1.0 / p).cuda())
    grid = default_clip_grid()
    tl = P.lrq_tlq_quantize_weights(Wr, 4, 0, 7, grid, grid)
    layer = P.QLayer(tl, N, K, P.ROT_HADAMARD, 8, B, prescale=torch.from_numpy(p).cuda())
    Y = P.lrq_qlinear(layer, PU.bf16_to_device(xb), P.F32).cpu().numpy().astype(np.float64)
    ref = X @ W.astype(np.float64).T
    err = np.linalg.norm(Y - ref) / np.linalg.norm(ref)
    assert err < 0.2, err       # the oracle gives 0.117 on these inputs; without colmul it is 0.92
    assert P.lrq_device_status() == 0


def _sweep_shapes():
    rng = np.random.default_rng(2024)
    out = []
    for i in range(28):
        K = 64 * int(rng.integers(1, 25))
        G = 128 if (K % 128 == 0 and rng.random() < 0.5) else 0
        M = int(rng.integers(1, 900))
        N = 8 * int(rng.integers(1, 180))
        w_bits, a_bits = int(rng.choice([3, 4])), int(rng.choice([4, 8]))
        dt = ["F32", "F16", "BF16"][i % 3]
        out.append((M, K, N, w_bits, a_bits, G, dt))
    return out


@pytest.mark.parametrize("M,K,N,w_bits,a_bits,G,dt", _sweep_shapes())
def test_qgemm_shape_sweep_against_cuda_core(P, M, K, N, w_bits, a_bits, G, dt):
    # Seeded random shapes (ragged M and N, one to 24 k-blocks, both tile widths, every output type): the tcgen05
    # kernel against the plain CUDA-core kernel on the same codes.  fp32: summation order only; 16-bit outputs:
    # one more rounding of a value that may differ in its last fp32 bits (one 16-bit ulp).
    B = 1
    while K % (2 * B) == 0 and B < 128:
        B *= 2
    spec = LayerSpec("w", 900 + M, M, K, N, w_bits, a_bits, G, "hadamard", B)
    layer, _ = PU.gpu_layer(spec, spec.weights(), P)
    X = PU.bf16_to_device(spec.activations())
    q, s, z = P.lrq_rotate_quantize_act(X, P.ROT_HADAMARD, a_bits, B)
    code = getattr(P, dt)
    ref = P.lrq_qgemm_codes(layer, q, s, z, code, 1).float()
    Y = P.lrq_qgemm_codes(layer, q, s, z, code, 0).float()
    torch.cuda.synchronize()
    assert P.lrq_device_status() == 0
    rms = ref.pow(2).mean().sqrt().item()
    tol = 2e-3 * rms if dt == "F32" else (2e-3 * rms + ref.abs() * (2.0 ** -7 if dt == "BF16" else 2.0 ** -10))
    assert ((Y - ref).abs() <= tol).all()
    layer.close()


# ------------------------------------------------------------------------------------ host-side behaviour
def test_bounded_wait_runs_out_and_is_reported(P, orc):
    # The one place where a device-side wait is made to expire: the library's diagnostic kernel (one warp, one
    # barrier nothing arrives on, no copy or tensor memory in flight) calls the same bounded-wait routine the
    # tensor-core kernels use, with a budget of 100 000 cycles.  The code must show up once in the status word,
    # the word must then be clear, and the path must work as before.
    assert P.lrq_device_status() == 0
    P.lrq_selftest_wait_timeout(100000)
    assert P.lrq_device_status() == P.SELFTEST_WAIT_CODE
    assert P.lrq_device_status() == 0
    spec, W, xb, layer, tl, T = _small_layer(P, orc, 70, 256, 72, 4, 8, 0, 128, 45)
    Yo, *_ = PU.oracle_layer_rows(orc, spec, xb, T)
    Y = P.lrq_qlinear(layer, PU.bf16_to_device(xb), P.F32)
    PU.check_out(Y.cpu().numpy(), Yo, "after the expired wait")
    assert P.lrq_device_status() == 0
    with pytest.raises(P.LrqError):
        P.lrq_selftest_wait_timeout(0)


def test_two_host_threads_on_two_streams(P):
    # Calls on different streams with different workspaces may run concurrently, from different host threads, on the
    # same layer handle or on handles created concurrently.
    import threading
    spec = LayerSpec("t", 91, 300, 1152, 264, 4, 8, 0, "hadamard", 128)
    W = spec.weights()
    X = PU.bf16_to_device(spec.activations())
    shared_layer, _ = PU.gpu_layer(spec, W, P)
    ref = P.lrq_qlinear(shared_layer, X, P.F32)
    torch.cuda.synchronize()
    results, errors = {}, []

    def work(i):
        try:
            torch.cuda.set_device(0)
            st = torch.cuda.Stream()
            own_layer, _ = PU.gpu_layer(spec, W, P)                      # created on this thread
            ws = torch.empty(shared_layer.workspace_bytes(spec.M), dtype=torch.uint8, device="cuda")
            outs = []
            with torch.cuda.stream(st):
                for r in range(20):
                    L = shared_layer if r % 2 else own_layer
                    outs.append(P.lrq_qlinear(L, X, P.F32, workspace=ws, stream=st))
            st.synchronize()
            results[i] = outs
        except Exception as e:                                           # surfaced in the main thread
            errors.append(e)

    ts = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    assert not errors, errors
    for outs in results.values():
        for y in outs:
            assert torch.equal(y, ref)
    assert P.lrq_device_status() == 0


# --------------------------------------------------------------- packed 3-bit codes, small-tile contraction
@pytest.mark.parametrize("M,K,N,a_bits,G,B", [(256, 1024, 1024, 4, 0, 1024), (70, 256, 72, 8, 0, 128), (33, 512, 136, 4, 128, 512),
                                              (300, 1152, 392, 8, 128, 128), (1, 128, 8, 4, 64, 64)])
def test_packed3_codes_and_small_tile_kernel(P, orc, M, K, N, a_bits, G, B):
    # W3 weights stored as the b-bit codes of Eq. 5 really need: eight codes in three bytes.  TLQ must emit the same
    # codes and tables as for the nibble layout (compared with the oracle bit for bit through the 3-bit unpacking), and
    # the layer - taken by the small-tile contraction - must reproduce the oracle's outputs element by element.
    spec = LayerSpec("p3", 33, M, K, N, 3, a_bits, G, "hadamard", B)
    W, xb = spec.weights(), spec.activations()
    layer, tl = PU.gpu_layer(spec, W, P, code_layout=P.CODES_PACKED3)
    assert tl.codes.shape == (N, 3 * K // 8)
    T = PU.check_tlq(orc, W, tl, 3, G, what="packed3", packed3=True)
    Yo, oq, os_, oz, Yr = PU.oracle_layer_rows(orc, spec, xb, T)
    X = PU.bf16_to_device(xb)
    q, s, z = P.lrq_rotate_quantize_act(X, P.ROT_HADAMARD, a_bits, B)
    gq, gz = PU.act_codes_to_numpy(q, a_bits), z.cpu().numpy()
    act = PU.check_act(gq, s.cpu().numpy(), gz, oq, os_, oz, Yr, "hadamard", B, "packed3 codes")
    for dt in (P.F32, P.F16):
        Y = P.lrq_qlinear(layer, X, dt)
        PU.check_layer_out(orc, T, Y.float().cpu().numpy(), gq, gz, Yo, os_, act, "packed3 qlinear")
    # the same contraction on the CUDA cores reads the packed layout too
    Yc = P.lrq_qgemm_codes(layer, q, s, z, P.F32, 1)
    Ys = P.lrq_qgemm_codes(layer, q, s, z, P.F32, 2)
    rms = Yc.pow(2).mean().sqrt().item()
    assert ((Ys - Yc).abs().max().item() <= 2e-3 * rms)
    with pytest.raises(P.LrqError) as e:
        P.lrq_qgemm_codes(layer, q, s, z, P.F32, 0)          # the large-tile kernel does not read this layout
    assert e.value.code == 2
    assert P.lrq_device_status() == 0


def test_packed3_needs_three_bit_codes(P):
    Wd = torch.zeros((8, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(P.LrqError) as e:
        P.lrq_tlq_quantize_weights(Wd, 4, 0, 7, [1.0], [1.0], code_layout=P.CODES_PACKED3)
    assert e.value.code == 2


@pytest.mark.parametrize("M", [1, 100, 256, 300])
@pytest.mark.parametrize("w_bits,a_bits", [(4, 8), (3, 4), (4, 4)])
def test_small_batches_take_the_small_tile_kernel(P, orc, M, w_bits, a_bits):
    # lrq_qlinear on a few hundred tokens (the automatic choice) against the oracle, nibble layout
    spec = LayerSpec("sm", 35, M, 512, 264, w_bits, a_bits, 128, "hadamard", 128)
    W, xb = spec.weights(), spec.activations()
    layer, tl = PU.gpu_layer(spec, W, P)
    T = PU.check_tlq(orc, W, tl, w_bits, 128, what="small")
    Yo, oq, os_, oz, Yr = PU.oracle_layer_rows(orc, spec, xb, T)
    X = PU.bf16_to_device(xb)
    q, s, z = P.lrq_rotate_quantize_act(X, P.ROT_HADAMARD, a_bits, 128)
    gq, gz = PU.act_codes_to_numpy(q, a_bits), z.cpu().numpy()
    act = PU.check_act(gq, s.cpu().numpy(), gz, oq, os_, oz, Yr, "hadamard", 128, "small codes")
    Y = P.lrq_qlinear(layer, X, P.F32)
    PU.check_layer_out(orc, T, Y.cpu().numpy(), gq, gz, Yo, os_, act, "small qlinear")
    Y2 = P.lrq_qgemm_codes(layer, q, s, z, P.F32, 2)
    assert torch.equal(Y, Y2)                                # lrq_qlinear took the small-tile kernel
    assert P.lrq_device_status() == 0
