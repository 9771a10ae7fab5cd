"""Pins of the oracle's rotations (Sec. 3.2 Eqs. 2-3, Sec. 4.2 Eq. 12, Sec. 4.3 Lemma 1)."""
import os

import numpy as np
import pytest
import scipy.linalg

HERE = os.path.dirname(os.path.abspath(__file__))


def _golden():
    mats, cur = {}, None
    for line in open(os.path.join(HERE, "golden", "hadamard_eq3.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("H"):
            cur = line
            mats[cur] = []
        else:
            mats[cur].append([float(v) for v in line.split()])
    return {k: np.array(v) for k, v in mats.items()}


def test_printed_h2_and_h4(orc):
    g = _golden()
    assert np.allclose(orc.hadamard_matrix(2) * np.sqrt(2), g["H2"], atol=1e-15)
    assert np.allclose(orc.hadamard_matrix(4) * 2.0, g["H4"], atol=1e-15)


@pytest.mark.parametrize("n", [1, 2, 4, 8, 64, 128, 512, 1024])
def test_hadamard_orthogonal_and_closed_form(orc, n):
    H = orc.hadamard_matrix(n)
    assert np.abs(H @ H.T - np.eye(n)).max() < 1e-13               # H H^T = I (Eq. 2)
    U = H * np.sqrt(n)
    assert np.abs(U @ U.T - n * np.eye(n)).max() < 1e-10           # unnormalised: n I
    i, j = np.meshgrid(np.arange(n), np.arange(n), indexing="ij")
    pop = np.array([bin(v).count("1") for v in (i & j).ravel()]).reshape(n, n)
    assert np.array_equal(np.rint(U), (-1.0) ** pop)                # entry (-1)^popcount(i&j)
    assert np.array_equal(np.rint(U), scipy.linalg.hadamard(n) if n > 1 else np.ones((1, 1)))
    assert np.array_equal(H, H.T)


def test_hadamard_rejects_non_power_of_two(orc):
    with pytest.raises(ValueError):
        orc.hadamard_matrix(12)
    with pytest.raises(ValueError):
        orc.rotate_hadamard_fwht(np.zeros((1, 12)), 12)
    with pytest.raises(ValueError):
        orc.rotate_hadamard_fwht(np.zeros((1, 12)), 8)


@pytest.mark.parametrize("n", [2, 4, 16, 128, 1024, 4096])
def test_fwht_equals_explicit_product(orc, n):
    rng = np.random.default_rng(n)
    X = rng.standard_normal((3, n))
    a = orc.rotate_hadamard_fwht(X, n)
    b = orc.rotate_hadamard_explicit(X, n)
    c = X @ (scipy.linalg.hadamard(n) / np.sqrt(n))                 # library matrix, library matmul
    assert np.abs(a - b).max() < 1e-12 * np.sqrt(n)
    assert np.abs(a - c).max() < 1e-12 * np.sqrt(n)
    assert np.abs(orc.rotate_hadamard_fwht(a, n) - X).max() < 1e-12 * np.sqrt(n)   # involution


def test_fwht_spike_is_flattened_exactly(orc):
    # Lemma 1: a vector dominated by one entry alpha maps to entries of magnitude alpha / sqrt(C).
    for C, j, alpha in [(64, 5, 245.0), (1024, 1000, 300.0), (4096, 0, 3.0)]:
        x = np.zeros((1, C))
        x[0, j] = alpha
        y = orc.rotate_hadamard_fwht(x, C)
        assert np.array_equal(np.abs(y), np.full((1, C), alpha / np.sqrt(C)))
        assert abs(np.linalg.norm(y) - alpha) < 1e-12 * alpha


def test_block_diagonal_blocks_are_independent(orc):
    rng = np.random.default_rng(3)
    K, B = 1152, 128
    X = rng.standard_normal((4, K))
    y = orc.rotate_hadamard_fwht(X, B)
    for j in range(K // B):
        yj = orc.rotate_hadamard_fwht(X[:, j * B:(j + 1) * B], B)
        assert np.array_equal(y[:, j * B:(j + 1) * B], yj)
    X2 = X.copy()
    X2[:, :B] += 1.0                                                # touching block 0 moves block 0 only
    y2 = orc.rotate_hadamard_fwht(X2, B)
    assert np.array_equal(y2[:, B:], y[:, B:]) and not np.array_equal(y2[:, :B], y[:, :B])
    assert np.abs(np.linalg.norm(y, axis=1) - np.linalg.norm(X, axis=1)).max() < 1e-12


def test_dense_rotation_matches_library_matmul_and_keeps_norm(orc):
    from lrq_workloads import make_orthogonal
    rng = np.random.default_rng(4)
    K = 96
    R = make_orthogonal(7, K)
    assert np.abs(R @ R.T - np.eye(K)).max() < 1e-12
    X = rng.standard_normal((5, K))
    y = orc.rotate_dense(X, R)
    assert np.abs(y - X @ R).max() < 1e-13
    assert np.abs(np.linalg.norm(y, axis=1) - np.linalg.norm(X, axis=1)).max() < 1e-12   # Lemma 1
    # not symmetric: a transposed operand would fail here
    assert np.abs(y - X @ R.T).max() > 1e-3


def test_dense_rotation_with_hadamard_matrix_equals_fwht(orc):
    rng = np.random.default_rng(5)
    X = rng.standard_normal((3, 256))
    Hd = np.kron(np.eye(2), orc.hadamard_matrix(128))
    assert np.abs(orc.rotate_dense(X, Hd) - orc.rotate_hadamard_fwht(X, 128)).max() < 1e-12


def test_rotation_invariance_of_the_product(orc):
    # Eq. 2: (X R)(W R)^T = X W^T for orthogonal R (both rotation kinds).
    from lrq_workloads import make_orthogonal
    rng = np.random.default_rng(6)
    K = 128
    X = rng.standard_normal((4, K))
    W = rng.standard_normal((7, K))
    ref = X @ W.T
    for rot in (lambda A: orc.rotate_hadamard_fwht(A, 64), lambda A: orc.rotate_dense(A, make_orthogonal(1, K))):
        assert np.abs(rot(X) @ rot(W).T - ref).max() < 1e-12


# ------------------------------------------------------------------ the dual transformation in its factors (Sec. 4.2)
def _dual_inputs(K=256, Bd=64, seed=3):
    from lrq_workloads import make_block_rotations, make_staggered_permutation
    R1 = make_block_rotations(seed, K, Bd)
    R2 = make_block_rotations(seed + 1, K, Bd)
    perm = make_staggered_permutation(seed, K, Bd, np.array([5, 70, 7, 200]))
    return R1, perm, R2


def test_dual_rotation_worked_example(orc):
    # K = 4, blocks of 2, worked by hand: u = x R1 = [-2, 1, 3, 4]; v_i = u[perm[i]] = [3, -2, 4, 1];
    # y = v R2 = [2, 3, 1, -4].  A transposed block or a scatter instead of a gather gives other numbers.
    q = np.array([[0.0, 1.0], [-1.0, 0.0]])                       # x q = [-x1, x0]
    R1 = np.stack([q, np.eye(2)])
    R2 = np.stack([q, q.T])
    y = orc.rotate_dual(np.array([[1.0, 2.0, 3.0, 4.0]]), 2, R1, [2, 0, 3, 1], R2)
    assert np.array_equal(y, [[2.0, 3.0, 1.0, -4.0]])


def test_dual_rotation_equals_dense_rotation_by_the_composed_matrix(orc):
    K, Bd = 256, 64
    R1, perm, R2 = _dual_inputs(K, Bd)
    Pm = np.zeros((K, K))
    Pm[perm, np.arange(K)] = 1.0                                  # (u P)_i = u[perm[i]]
    R = scipy.linalg.block_diag(*R1) @ Pm @ scipy.linalg.block_diag(*R2)
    assert np.abs(R @ R.T - np.eye(K)).max() < 1e-12              # the composition is a rotation
    X = np.random.default_rng(0).standard_normal((9, K)) * 4.0
    Yd = orc.rotate_dual(X, Bd, R1, perm, R2)
    assert np.abs(Yd - orc.rotate_dense(X, R)).max() < 1e-12
    assert np.abs(Yd - X @ R).max() < 1e-12
    assert np.allclose(np.linalg.norm(Yd, axis=1), np.linalg.norm(X, axis=1), rtol=1e-13)   # Lemma 1: norms kept


def test_dual_rotation_special_cases(orc):
    K, Bd = 256, 64
    R1, perm, R2 = _dual_inputs(K, Bd)
    X = np.random.default_rng(1).standard_normal((5, K))
    eye = np.broadcast_to(np.eye(Bd), R1.shape)
    ident = np.arange(K)
    # R2 = I, P = I: the blocks of R1 act on their own channels only
    Y = orc.rotate_dual(X, Bd, R1, ident, eye)
    assert np.abs(Y - np.einsum("mjl,jli->mji", X.reshape(5, K // Bd, Bd), R1).reshape(5, K)).max() < 1e-13
    # R1 = R2 = I: a pure reordering, exactly
    assert np.array_equal(orc.rotate_dual(X, Bd, eye, perm, eye), X[:, perm])
    # one block of K channels and no reordering: two dense rotations in a row
    Q1 = _dual_inputs(K, K, 8)[0]
    Q2 = _dual_inputs(K, K, 9)[0]
    assert np.abs(orc.rotate_dual(X, K, Q1, ident, Q2) - X @ Q1[0] @ Q2[0]).max() < 1e-12


def test_dual_rotation_spreads_leading_channels_over_blocks():
    from lrq_workloads import make_staggered_permutation
    K, Bd = 1152, 128
    first = np.array([3, 4, 5, 6, 7, 8, 9, 10, 11, 600])          # nine neighbours of one block, and one more
    perm = make_staggered_permutation(0, K, Bd, first)
    assert np.array_equal(np.sort(perm), np.arange(K))
    where = {int(c): i // Bd for i, c in enumerate(perm)}
    assert sorted(where[int(c)] for c in first[:9]) == list(range(9))   # one per block
    assert where[600] == 8                                        # the second pass runs backwards


def test_dual_rotation_rejects_a_non_permutation(orc):
    R1, perm, R2 = _dual_inputs()
    bad = perm.copy()
    bad[0] = bad[1]
    with pytest.raises(ValueError):
        orc.rotate_dual(np.zeros((1, 256)), 64, R1, bad, R2)
    with pytest.raises(ValueError):
        orc.rotate_dual(np.zeros((1, 256)), 64, R1, np.arange(256) + 1, R2)
