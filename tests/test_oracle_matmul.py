"""Pins of the oracle's quantized contraction and of the whole layer (Sec. 4.1 Eq. 10, Sec. 3.2 Eq. 2)."""
from fractions import Fraction

import numpy as np

from lrq_workloads import default_clip_grid


def _tiny(orc, bits_w=3, bits_a=4, M=3, K=16, N=4, G=0, seed=0):
    rng = np.random.default_rng(seed)
    W = (rng.standard_t(4, size=(N, K)) * 0.014).astype(np.float32).astype(np.float64)
    X = rng.standard_normal((M, K)).astype(np.float32).astype(np.float64)
    T = orc.tlq_quantize(W, bits_w, G, 7, default_clip_grid(), default_clip_grid())
    Q, S, Z = orc.quantize_act(X, bits_a)
    return W, X, T, Q, S, Z


def test_contraction_equals_exact_rational_arithmetic(orc):
    # every factor is a dyadic rational: evaluate Eq. 10 exactly with Fractions
    for G in (0, 8):
        W, X, T, Q, S, Z = _tiny(orc, G=G, seed=G)
        rng = np.random.default_rng(1)
        wscale = rng.uniform(0.5, 2.0, size=W.shape[0])
        bias = rng.standard_normal(W.shape[0])
        Y = orc.qmatmul(Q, S, Z, T, wscale, bias)
        half, Gs = 4, (G or W.shape[1])
        for m in range(X.shape[0]):
            for n in range(W.shape[0]):
                acc = Fraction(0)
                for k in range(W.shape[1]):
                    lvl = Fraction(float(T.levels[n, k // Gs, int(T.codes[n, k]) + half]))
                    acc += (Fraction(int(Q[m, k])) + Fraction(int(Z[m]))) * lvl
                exact = Fraction(float(S[m])) * acc * Fraction(float(wscale[n])) + Fraction(float(bias[n]))
                assert abs(Y[m, n] - float(exact)) <= 1e-14 * max(1e-30, abs(float(exact)) + abs(bias[n]))


def test_contraction_is_the_product_of_the_dequantized_operands(orc):
    # Eq. 10 == X_f W_f^T with X_f from Eq. 1 and W_f the table entries: library matmul in fp64
    W, X, T, Q, S, Z = _tiny(orc, bits_w=4, bits_a=8, M=9, K=64, N=11, G=32, seed=3)
    Wf = np.take_along_axis(T.levels.repeat(32, axis=1), (T.codes.astype(int) + 8)[:, :, None], axis=2)[:, :, 0]
    Xf = orc.dequantize_act(Q, S, Z)
    Y = orc.qmatmul(Q, S, Z, T)
    ref = Xf @ Wf.T
    assert np.abs(Y - ref).max() <= 1e-13 * np.abs(ref).max()
    # zero-point identity: sum (q+z) w = sum q w + z sum w
    assert np.allclose(T.wsum, Wf.sum(axis=1), rtol=1e-13)
    # a transposed or mis-indexed weight operand would not survive a non-square check
    assert Y.shape == (9, 11)


def test_contraction_with_identity_quantizers_is_a_plain_matmul(orc):
    # integer activations on a unit grid and power-of-two weights: both quantizers are lossless,
    # so the layer reduces to numpy.matmul
    rng = np.random.default_rng(4)
    K, N, M = 32, 5, 6
    expo = rng.integers(1, 9, size=(N, K))
    sign = np.where(rng.random((N, K)) < 0.5, -1.0, 1.0)
    W = sign * 2.0 ** (-expo)
    for n in range(N):                                   # make both sides span their full unit grids
        W[n, :8] = 2.0 ** -np.arange(1, 9)
        W[n, 8:17] = -(2.0 ** -np.arange(1, 10))
    X = rng.integers(-100, 156, size=(M, K)).astype(np.float64)
    X[:, 0], X[:, 1] = -100, 155
    T = orc.tlq_quantize(W, 4, 0, 7)
    Y, Q, S, Z = orc.qlinear(X, T, 8, "none")
    lossy = (T.codes == 0) & (W < 0)                    # negative elements folded into code 0 (smallest levels)
    Wd = np.where(lossy, 2.0 ** -8, W)
    assert np.array_equal(S, np.ones(M))
    assert np.abs(Y - X @ Wd.T).max() < 1e-12
    assert lossy.sum() <= N * 3


def test_all_ones_codes_one_level_table(orc):
    from oracle import TLQResult
    K, N, M = 40, 3, 2
    lv = np.zeros((N, 1, 8))
    lv[:, 0, 5] = [0.375, -1.5, 2.0 ** -20]
    T = TLQResult(np.ones((N, K), dtype=np.int8), lv, np.zeros((N, 1, 6)), np.zeros(N), np.zeros((N, 1)), 3, K)
    Q = np.ones((M, K), dtype=np.int32)
    Y = orc.qmatmul(Q, np.array([1.0, 2.0]), np.array([0, 3], dtype=np.int32), T)
    assert np.array_equal(Y[0], K * lv[:, 0, 5])
    assert np.array_equal(Y[1], 2.0 * (K * lv[:, 0, 5] + 3 * K * lv[:, 0, 5]))


def test_layer_output_converges_to_the_full_precision_product(orc):
    # trend only: with more bits the layer approaches X W^T
    rng = np.random.default_rng(5)
    W = (rng.standard_normal((16, 128)) * 0.02).astype(np.float32).astype(np.float64)
    W = np.sign(W) * np.maximum(np.abs(W), 1e-3)          # bounded log-range so the log grid can refine
    X = rng.standard_normal((8, 128))
    ref = orc.rotate_hadamard_fwht(X, 128) @ W.T          # weights are given in the rotated basis
    errs = []
    for b in (3, 5, 8):
        T = orc.tlq_quantize(W, b, 0, -1)
        Y, *_ = orc.qlinear(X, T, b + 4, "hadamard", 128)
        errs.append(np.linalg.norm(Y - ref) / np.linalg.norm(ref))
    assert errs[0] > errs[1] > errs[2] and errs[2] < 0.02


def test_layer_rotation_invariance_with_fine_quantizers(orc):
    # Eq. 2 end to end: rotating activations and weights by the same R leaves the product (nearly) unchanged
    rng = np.random.default_rng(6)
    W = rng.standard_normal((8, 64))
    W = np.sign(W) * np.maximum(np.abs(W), 0.05)
    X = rng.standard_normal((4, 64))
    Wr = orc.rotate_hadamard_fwht(W, 64)
    T = orc.tlq_quantize(Wr, 8, 0, -1)
    Y, *_ = orc.qlinear(X, T, 12, "hadamard", 64)
    ref = X @ W.T
    assert np.linalg.norm(Y - ref) / np.linalg.norm(ref) < 0.05


def test_integer_shift_form_of_eq10_equals_the_level_table_product(orc):
    # Eq. 10 as printed: (mantissa of the level x integer of the activation) << (f - I), with Python integers.  A level
    # is II * 2^(f - I), II = rint(2^r * 2^I) (Eqs. 8-9, I = 7), so II and f come back exactly from the level's value.
    import math
    for G in (0, 8):
        W, X, T, Q, S, Z = _tiny(orc, G=G, seed=10 + G)
        Y = orc.qmatmul(Q, S, Z, T)
        half, Gs = 4, (G or W.shape[1])
        for n in range(W.shape[0]):
            lv = T.levels[n].ravel()
            exps = [math.frexp(abs(v))[1] for v in lv if v != 0.0]
            emin = min(exps)                                   # common factor: keeps every shift non-negative
            for m in range(X.shape[0]):
                acc = 0
                for k in range(W.shape[1]):
                    v = float(T.levels[n, k // Gs, int(T.codes[n, k]) + half])
                    f, e = math.frexp(abs(v))
                    mant = int(f * 256)
                    assert mant == f * 256 and 128 <= mant <= 255          # an 8-bit mantissa
                    ix = int(Q[m, k]) + int(Z[m])                           # the activation's integer: x = s (q + z)
                    acc += (-1 if v < 0 else 1) * ((mant * ix) << (e - emin)) if ix >= 0 else \
                           (-1 if v < 0 else 1) * -((mant * -ix) << (e - emin))
                exact = Fraction(float(S[m])) * Fraction(acc) * Fraction(2) ** (emin - 8)
                assert abs(Y[m, n] - float(exact)) <= 1e-14 * max(1e-30, abs(float(exact)))
