"""Pins of the oracle's per-token quantizer (Sec. 3.1, Eq. 1) and of TLQ (Sec. 4.1, Eqs. 4-9)."""
import itertools

import numpy as np
import pytest

from lrq_workloads import bf16_bits_to_f32, f32_to_bf16_bits, default_clip_grid


# ----------------------------------------------------------------------------- Eq. 1
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_act_quantizer_range_and_error_bound(orc, bits):
    rng = np.random.default_rng(bits)
    Y = rng.standard_normal((16, 200)) * rng.uniform(0.1, 30, size=(16, 1)) + rng.uniform(-5, 5, size=(16, 1))
    Q, S, Z = orc.quantize_act(Y, bits)
    qmax = 2 ** bits - 1
    assert Q.min() >= 0 and Q.max() <= qmax
    for m in range(Y.shape[0]):
        assert S[m] == (Y[m].max() - Y[m].min()) / qmax
        assert Z[m] == np.rint(Y[m].min() / S[m])
        assert Q[m, Y[m].argmin()] == 0                              # min -> code 0
        assert Q[m, Y[m].argmax()] in (qmax, qmax - 1)               # max -> top code, or one below when z rounded up
    Xf = orc.dequantize_act(Q, S, Z)
    err = np.abs(Xf - Y)
    # inside the code range the error is at most half a step; the clamp at the ends adds at most half a step more
    assert (err <= S[:, None] * (1.0 + 1e-12)).all()
    inner = (Q > 0) & (Q < qmax)
    assert (err[inner] <= 0.5 * S[:, None].repeat(Y.shape[1], 1)[inner] * (1 + 1e-12)).all()
    assert (Q.max(axis=1) >= qmax - 1).all()                         # max lands on the top code or one below


def test_act_quantizer_is_idempotent(orc):
    rng = np.random.default_rng(11)
    Y = rng.standard_normal((8, 64)) * 3
    Q, S, Z = orc.quantize_act(Y, 4)
    Xf = orc.dequantize_act(Q, S, Z)
    # re-quantizing the grid points with the same (s, z): every point maps to itself
    Q2 = np.clip(np.rint(Xf / S[:, None]) - Z[:, None], 0, 15).astype(np.int32)
    assert np.array_equal(Q, Q2)


def test_act_quantizer_brute_force_nearest_grid_point(orc):
    rng = np.random.default_rng(12)
    Y = rng.standard_normal((6, 9)) * 2
    for bits in (2, 3, 4):
        Q, S, Z = orc.quantize_act(Y, bits)
        for m, k in itertools.product(range(Y.shape[0]), range(Y.shape[1])):
            grid = S[m] * (np.arange(2 ** bits) + Z[m])
            d = np.abs(grid - Y[m, k])
            assert d[Q[m, k]] <= d.min() + 1e-12 * S[m]


def test_act_quantizer_lossless_on_integer_ramp(orc):
    # b = 8 on integers spanning exactly 255 steps: s = 1, codes = values - min
    base = np.arange(-100, 156, dtype=np.float64)
    Y = np.stack([base, base[::-1] + 7])
    Q, S, Z = orc.quantize_act(Y, 8)
    assert np.array_equal(S, [1.0, 1.0]) and np.array_equal(Z, [-100, -93])
    assert np.array_equal(orc.dequantize_act(Q, S, Z), Y)


def test_act_quantizer_symmetric_mode_and_degenerate_tokens(orc):
    Y = np.array([[1.0, -7.0, 3.5, 0.0], [2.0, 2.0, 2.0, 2.0], [0.0, 0.0, 0.0, 0.0]])
    Q, S, Z = orc.quantize_act(Y, 4, mode=1)
    assert S[0] == 1.0 and Z[0] == -8
    assert np.array_equal(Q[0], [9, 1, 12, 8])                       # rint(3.5) = 4 (ties to even)
    Qa, Sa, Za = orc.quantize_act(Y, 4, mode=0)
    assert Sa[1] == 1.0 and Za[1] == 2 and np.array_equal(Qa[1], [0, 0, 0, 0])   # constant token: s = 1
    assert Sa[2] == 1.0 and Za[2] == 0 and S[2] == 1.0


def test_rounding_is_ties_to_even(orc):
    Y = np.array([[0.0, 0.5, 1.5, 2.5, 3.0]])                        # s = 1 with b such that range/qmax = 1
    Q, S, Z = orc.quantize_act(Y, 2)
    assert S[0] == 1.0 and np.array_equal(Q[0], [0, 0, 2, 2, 3])


# ----------------------------------------------------------------------------- Eqs. 8-9
def test_level_value_integerization_bound(orc):
    rng = np.random.default_rng(13)
    for e in rng.uniform(-30, 4, size=400):
        f = np.floor(e)
        for I in (6, 7, 8):
            v = orc.level_value(e, I)
            assert abs(v - 2.0 ** e) <= 2.0 ** (f - I - 1) * (1 + 1e-12)          # |II 2^-I - 2^r| <= 2^-(I+1)
            II = v / 2.0 ** (f - I)
            assert II == np.rint(II) and 2 ** I <= II <= 2 ** (I + 1)
        assert abs(orc.level_value(e, -1) / 2.0 ** e - 1) < 1e-15
        v7 = np.float32(orc.level_value(e, 7))
        assert bf16_bits_to_f32(f32_to_bf16_bits(np.array([v7])))[0] == v7       # I = 7 levels are bf16 numbers
    assert orc.level_value(3.0, 7) == 8.0 and orc.level_value(-2.0, 7) == 0.25


# ----------------------------------------------------------------------------- Eqs. 4-7
def _rand_w(rng, N, K):
    return (rng.standard_t(4, size=(N, K)) * 0.014).astype(np.float32).astype(np.float64)


@pytest.mark.parametrize("bits,G", [(3, 0), (4, 0), (3, 32), (4, 64), (2, 16)])
def test_tlq_structure(orc, bits, G):
    rng = np.random.default_rng(100 + bits + G)
    W = _rand_w(rng, 12, 128)
    W[0, :5] = 0.0
    T = orc.tlq_quantize(W, bits, G, 7, default_clip_grid(), default_clip_grid())
    half, Gs = 2 ** (bits - 1), (G or 128)
    assert T.codes.min() >= -half and T.codes.max() <= half - 1
    assert (T.codes[W > 0] >= 0).all() and (T.codes[W < 0] <= 0).all() and (T.codes[W == 0] == 0).all()
    for n in range(W.shape[0]):
        for g in range(128 // Gs):
            lv = T.levels[n, g]
            assert len(np.unique(lv)) <= 2 ** bits                    # at most 2^b distinct levels
            assert (lv[half + 1:] > 0).all() and (lv[:half] < 0).all() and lv[half] >= 0
            assert (np.diff(lv[half:]) > 0).all() and (np.diff(lv[:half]) > 0).all()   # monotone in the code
            w = W[n, g * Gs:(g + 1) * Gs]
            c = T.codes[n, g * Gs:(g + 1) * Gs].astype(int)
            o = np.argsort(w, kind="stable")
            assert (np.diff(c[o]) >= 0).all()                         # code is monotone non-decreasing in w
    # wsum is the row sum of the de-quantized weights
    deq = np.take_along_axis(T.levels.reshape(12, -1, 2 ** bits).repeat(Gs, axis=1),
                             (T.codes.astype(int) + half)[:, :, None], axis=2)[:, :, 0]
    assert np.allclose(T.wsum, deq.sum(axis=1), rtol=1e-13, atol=0)


def test_tlq_brute_force_nearest_level_in_log_domain(orc):
    # With Eq. 7 levels (I < 0) each code is the nearest point of the side's log-domain grid s (q + z).
    rng = np.random.default_rng(14)
    W = _rand_w(rng, 6, 24)
    for bits in (3, 4):
        T = orc.tlq_quantize(W, bits, 0, -1, [1.0, 1.1, 1.3], [1.0, 1.2])
        half = 2 ** (bits - 1)
        for n in range(W.shape[0]):
            sp, zp, sn, zn = T.meta[n, 0, :4]
            for k in range(W.shape[1]):
                w, c = W[n, k], int(T.codes[n, k])
                if w > 0:
                    grid = sp * (np.arange(half) + zp)
                    d = np.abs(grid - np.log2(w))
                    assert d[c] <= d.min() + 1e-12
                    if c > 0:
                        assert abs(T.levels[n, 0, c + half] / 2.0 ** grid[c] - 1) < 1e-15
                else:
                    grid = sn * (np.arange(half + 1) + zn)
                    d = np.abs(grid - np.log2(-w))
                    assert d[-c] <= d.min() + 1e-12
                    if c < 0:
                        assert abs(T.levels[n, 0, c + half] / -(2.0 ** grid[-c]) - 1) < 1e-15
            assert abs(T.levels[n, 0, half] / 2.0 ** (sp * zp) - 1) < 1e-15              # code 0 carries the lowest positive level


def test_tlq_no_clipping_is_the_plain_minmax_log_quantizer(orc):
    rng = np.random.default_rng(15)
    W = _rand_w(rng, 4, 64)
    T = orc.tlq_quantize(W, 4, 0, -1)                                    # alpha = beta = 1
    for n in range(4):
        lp = np.log2(W[n][W[n] > 0])
        ln = np.log2(-W[n][W[n] < 0])
        assert T.meta[n, 0, 0] == (lp.max() - lp.min()) / 7 and T.meta[n, 0, 2] == (ln.max() - ln.min()) / 8
        assert T.meta[n, 0, 1] == np.rint(lp.min() / T.meta[n, 0, 0])
        assert T.meta[n, 0, 3] == np.rint(ln.min() / T.meta[n, 0, 2])
        assert T.meta[n, 0, 4] == 1.0 and T.meta[n, 0, 5] == 1.0
        # extremes of each side land on the end codes
        assert T.codes[n, np.argmax(W[n])] == 7 and T.codes[n, np.argmin(W[n])] == -8


def test_tlq_powers_of_two_are_lossless(orc):
    # weights +-2^-j on a unit log grid: s = 1 and exact reconstruction (the textbook log2 quantizer)
    bits = 4
    pos = [2.0 ** -j for j in range(1, 9)]                               # 8 values -> codes 0..7
    neg = [-(2.0 ** -j) for j in range(1, 10)]                           # 9 values -> codes 0..8
    W = np.array([pos + neg + pos[::-1] + neg[::-1]])
    for I in (-1, 7):
        T = orc.tlq_quantize(W, bits, 0, I)
        assert T.meta[0, 0, 0] == 1.0 and T.meta[0, 0, 2] == 1.0
        deq = T.levels[0, 0][T.codes[0].astype(int) + 8]
        ok = T.codes[0] != 0
        assert np.array_equal(deq[ok], W[0][ok])
        # the only lossy elements are the negative ones that share code 0 with the lowest positive level
        assert set(W[0][~ok]) == {2.0 ** -8, -(2.0 ** -9)}
        assert T.levels[0, 0, 8] == 2.0 ** -8


def test_tlq_dequantize_quantize_is_idempotent(orc):
    rng = np.random.default_rng(16)
    W = _rand_w(rng, 8, 96)
    g = default_clip_grid()
    for bits in (3, 4):
        T = orc.tlq_quantize(W, bits, 0, -1, g, g)
        half = 2 ** (bits - 1)
        deq = np.take_along_axis(T.levels[:, 0, :], T.codes.astype(int) + half, axis=1)
        # re-quantize the de-quantized weights on the same grids: every level maps back to its code
        for n in range(W.shape[0]):
            sp, zp, sn, zn = T.meta[n, 0, :4]
            for k in range(W.shape[1]):
                v, c = deq[n, k], int(T.codes[n, k])
                if c > 0:
                    assert np.clip(np.rint(np.log2(v) / sp) - zp, 0, half - 1) == c
                elif c < 0:
                    assert np.clip(np.rint(np.log2(-v) / sn) - zn, 0, half) == -c


def test_tlq_search_picks_the_best_candidate(orc):
    rng = np.random.default_rng(17)
    W = _rand_w(rng, 5, 256)
    g = default_clip_grid()
    T = orc.tlq_quantize(W, 4, 0, 7, g, g)
    one = [orc.tlq_quantize(W, 4, 0, 7, [a], [a]) for a in g]           # 1-point grids: no search
    half = 8
    for n in range(W.shape[0]):
        w = W[n]
        def side_err(R, pos):
            deq = R.levels[n, 0][R.codes[n].astype(int) + half]
            m = (w > 0) if pos else (w < 0)
            if not pos:                                                   # the negative side's own lowest level
                s, z = R.meta[n, 0, 2:4]
                deq = np.where(R.codes[n] == 0, -orc.level_value(s * z, 7), deq)
            return ((w[m] - deq[m]) ** 2).sum()
        ep = np.array([side_err(R, True) for R in one])
        en = np.array([side_err(R, False) for R in one])
        assert T.meta[n, 0, 4] == g[ep.argmin()] and T.meta[n, 0, 5] == g[en.argmin()]
        best = one[int(ep.argmin())]
        assert np.array_equal(T.codes[n][w > 0], best.codes[n][w > 0])
    assert (T.margin > 1e-9).all()


def test_tlq_group_equals_per_slice_quantization(orc):
    rng = np.random.default_rng(18)
    W = _rand_w(rng, 3, 256)
    g = default_clip_grid()
    T = orc.tlq_quantize(W, 3, 128, 7, g, g)
    for j in range(2):
        Tj = orc.tlq_quantize(W[:, j * 128:(j + 1) * 128], 3, 0, 7, g, g)
        assert np.array_equal(T.codes[:, j * 128:(j + 1) * 128], Tj.codes)
        assert np.array_equal(T.levels[:, j], Tj.levels[:, 0])


def test_tlq_one_sided_and_tiny_groups(orc):
    W = np.array([[0.5, 0.25, 0.125, 0.0625], [-0.5, -0.5, -0.5, -0.5], [0.0, 0.0, 0.0, 0.0], [0.3, -0.2, 0.0, 0.3]])
    T = orc.tlq_quantize(W, 3, 0, 7)
    assert np.array_equal(T.codes[0], [3, 2, 1, 0]) and (T.levels[0, 0, :4] == 0).all()
    assert np.array_equal(T.levels[0, 0, 4:], [0.0625, 0.125, 0.25, 0.5])
    assert (T.codes[1] == 0).all() or (T.codes[1] <= 0).all()
    assert (T.codes[2] == 0).all() and (T.levels[2] == 0).all() and T.wsum[2] == 0.0
    assert np.isfinite(T.levels).all() and np.isfinite(T.wsum).all()
