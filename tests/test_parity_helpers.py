"""The comparison rules of tests/parity.py, exercised on the CPU with the oracle on both sides: a stand-in for the
GPU result is made from the oracle's own output with a planted difference, and check_act must accept it only
when Eq. 1's rounding really allows two answers there."""
import numpy as np
import pytest

import parity as PU


def _token_batch(orc, seed=0, M=24, K=256, bits=8):
    rng = np.random.default_rng(seed)
    Y = rng.standard_normal((M, K)) * 3.0
    Q, S, Z = orc.quantize_act(Y, bits)
    return Y, Q, S, Z


def test_identical_results_pass(orc):
    Y, Q, S, Z = _token_batch(orc)
    r = PU.check_act(Q, S.astype(np.float32), Z, Q, S, Z, Y, "hadamard", 128, "same")
    assert r.flip_fraction == 0 and r.z_flips == 0 and not r.diff_tokens.any()


def test_flip_away_from_a_boundary_is_an_error(orc):
    Y, Q, S, Z = _token_batch(orc)
    t = Y / S[:, None]
    hd = np.abs(t - np.floor(t) - 0.5)
    inner = (Q > 0) & (Q < 255)
    m, k = np.unravel_index(np.argmax(np.where(inner, hd, -1)), hd.shape)      # as far from a boundary as it gets
    G = Q.copy()
    G[m, k] += 1
    with pytest.raises(AssertionError, match="away from a rounding boundary"):
        PU.check_act(G, S.astype(np.float32), Z, Q, S, Z, Y, "hadamard", 128, "planted")


def test_flip_on_a_boundary_is_accepted_and_counted(orc):
    Y, Q, S, Z = _token_batch(orc)
    # move one element to within 1e-7 code steps of a rounding boundary and re-run the oracle on it
    m, k = 3, 17
    t = Y[m, k] / S[m]
    Y2 = Y.copy()
    Y2[m, k] = (np.floor(t) + 0.5 - 1e-7) * S[m]
    Q2, S2, Z2 = orc.quantize_act(Y2, 8)
    assert np.array_equal(S2, S)                                               # the extremes were not touched
    G = Q2.copy()
    G[m, k] += 1                                                              # the other side of the boundary
    r = PU.check_act(G, S2.astype(np.float32), Z2, Q2, S2, Z2, Y2, "hadamard", 128, "boundary")
    assert r.flip_fraction == pytest.approx(1.0 / Q.size) and r.diff_tokens.sum() == 1 and r.diff_tokens[m]
    assert 0 < r.worst_boundary <= 1
    G[m, k] += 1                                                              # two codes away is never valid
    with pytest.raises(AssertionError, match="more than one"):
        PU.check_act(G, S2.astype(np.float32), Z2, Q2, S2, Z2, Y2, "hadamard", 128, "two away")


def test_exact_ties_are_valid_but_not_counted(orc):
    # integer-valued tokens with a unit step: x/s + 0 is an integer; shifting by half a step makes every element a tie
    base = np.arange(-100, 156, dtype=np.float64)
    Y = np.stack([base + 0.5, base[::-1] + 0.5])
    Q, S, Z = orc.quantize_act(Y, 8)
    assert np.array_equal(S, [1.0, 1.0])
    G = Q.copy()
    sel = (Q > 0) & (Q < 255)
    k = np.nonzero(sel[0])[0][:5]
    t = Y[0, k] / S[0]
    # the other valid rounding of an exact tie
    G[0, k] = np.where(np.rint(t) > t, Q[0, k] - 1, Q[0, k] + 1)
    r = PU.check_act(G, S.astype(np.float32), Z, Q, S, Z, Y, "none", 0, "ties")
    assert r.flip_fraction == 0 and r.tie_fraction == pytest.approx(5 / Q.size)


def test_too_many_boundary_flips_fail(orc):
    Y, Q, S, Z = _token_batch(orc, M=4, K=64)
    Y2 = Y.copy()
    ks = [5, 9, 33]                                                           # 3 of 256 elements > 1e-4
    for k in ks:
        t = Y[1, k] / S[1]
        Y2[1, k] = (np.floor(t) + 0.5 - 1e-7) * S[1]
    Q2, S2, Z2 = orc.quantize_act(Y2, 8)
    G = Q2.copy()
    G[1, ks] += 1
    with pytest.raises(AssertionError, match="of the codes differ"):
        PU.check_act(G, S2.astype(np.float32), Z2, Q2, S2, Z2, Y2, "hadamard", 64, "many")


def test_zero_point_flip_needs_min_on_a_boundary(orc):
    Y, Q, S, Z = _token_batch(orc, M=6, K=128)
    G, GZ = Q.copy(), Z.copy()
    GZ[2] += 1
    G[2] = np.clip(Q[2] - 1, 0, 255)                                          # q + z unchanged except where clamped
    with pytest.raises(AssertionError, match="zero-point differs"):
        PU.check_act(G, S.astype(np.float32), GZ, Q, S, Z, Y, "hadamard", 128, "z")


def test_scale_tolerance_is_per_path(orc):
    Y, Q, S, Z = _token_batch(orc)
    Sg = (S * (1 + 2e-6)).astype(np.float32)
    with pytest.raises(AssertionError, match="scales differ"):
        PU.check_act(Q, Sg, Z, Q, S, Z, Y, "hadamard", 128, "s")
    # a dense rotation of K = 3072 carries the tensor-core accumulation error in its extremes: wider bound
    assert PU.scale_rtol("dense", 3072) > 2e-5 > PU.scale_rtol("dense", 1152) > PU.scale_rtol("hadamard", 12288)


def test_unpack3_layout():
    codes = np.arange(16, dtype=np.uint8) % 8
    w0 = sum(int(c) << (3 * j) for j, c in enumerate(codes[:8]))
    w1 = sum(int(c) << (3 * j) for j, c in enumerate(codes[8:]))
    packed = np.array([[w0 & 255, (w0 >> 8) & 255, w0 >> 16, w1 & 255, (w1 >> 8) & 255, w1 >> 16]], dtype=np.uint8)
    assert np.array_equal(PU.unpack3(packed)[0], codes)
