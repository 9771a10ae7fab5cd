"""Pins of the two oracle routines around the rotation choice: the smoothing multipliers (Sec. 5.1) and the
fluctuation metric J with its threshold rule (Sec. 4.2, Eqs. 11-12)."""
import numpy as np
import pytest

from lrq_workloads import make_activations, make_orthogonal, make_weights, bf16_bits_to_f64


def test_smoothing_leaves_the_product_unchanged(orc):
    # Sec. 5.1 / SmoothQuant identity: (X diag(p)) (W diag(1/p))^T = X W^T, also through a rotation (Eq. 2)
    rng = np.random.default_rng(0)
    X = bf16_bits_to_f64(make_activations(1, 9, 256))
    W = make_weights(2, 7, 256).astype(np.float64)
    p = rng.uniform(0.05, 3.0, 256)
    Xs = orc.smooth(X, p)
    assert np.array_equal(Xs, X * p[None, :])                 # the definition itself, element by element
    Ws = W / p[None, :]
    ref = X @ W.T
    assert np.allclose(Xs @ Ws.T, ref, rtol=1e-12, atol=1e-12 * np.abs(ref).max())
    Yr = orc.rotate_hadamard_fwht(Xs, 128) @ orc.rotate_hadamard_fwht(Ws, 128).T
    assert np.allclose(Yr, ref, rtol=1e-11, atol=1e-11 * np.abs(ref).max())
    assert np.array_equal(orc.smooth(X, np.ones(256)), X)     # unit multipliers change nothing


@pytest.mark.parametrize("rot,B", [("hadamard", 64), ("hadamard", 256), ("dense", 0), ("none", 0)])
def test_rotated_weights_keep_the_layer_product(orc, rot, B):
    # Eq. 2 with the smoothing of Sec. 5.1: (X diag(p) R)(W diag(1/p) R)^T = X W^T for an orthogonal R.  A dropped
    # multiplier, a transposed R or a missing 1/sqrt(B) on either side breaks the identity.
    rng = np.random.default_rng(5)
    K = 256
    X = bf16_bits_to_f64(make_activations(11, 6, K))
    W = make_weights(12, 10, K).astype(np.float64)
    p = rng.uniform(0.2, 4.0, K)
    R = make_orthogonal(13, K) if rot == "dense" else None
    Wr = orc.rotate_weights(W, 1.0 / p, rot, B, R)
    Xs = orc.smooth(X, p)
    Xr = {"hadamard": lambda: orc.rotate_hadamard_fwht(Xs, B), "dense": lambda: orc.rotate_dense(Xs, R),
          "none": lambda: Xs}[rot]()
    ref = X @ W.T
    assert np.allclose(Xr @ Wr.T, ref, rtol=1e-11, atol=1e-11 * np.abs(ref).max())
    # against the explicit matrices (library product), and the norm of every row is kept by the rotation
    if rot == "hadamard":
        Hb = np.kron(np.eye(K // B), orc.hadamard_matrix(B))
        assert np.allclose(Wr, (W / p) @ Hb, rtol=1e-12, atol=1e-15)
    if rot == "dense":
        assert np.allclose(Wr, (W / p) @ R, rtol=1e-12, atol=1e-15)
    assert np.allclose(np.linalg.norm(Wr, axis=1), np.linalg.norm(W / p, axis=1), rtol=1e-12)
    assert np.array_equal(orc.rotate_weights(W, None, "none"), W)


def test_smoothing_tames_salient_channels(orc):
    # dividing a salient channel by its own magnitude brings it back to the others' range
    X = bf16_bits_to_f64(make_activations(3, 64, 128, n_salient=4, salient_x=60.0))
    amax = np.abs(X).max(axis=0)
    p = 1.0 / np.sqrt(amax)                                  # migration strength 0.5 with unit weight ranges
    Xs = orc.smooth(X, p)
    assert np.abs(Xs).max() < np.abs(X).max() / 4
    assert np.allclose(np.abs(Xs).max(axis=0), np.sqrt(amax))


def test_metric_closed_forms(orc):
    # Eq. 11 on inputs whose Frobenius norm is known in closed form
    J, kind = orc.fluctuation_metric(np.full((5, 8), -3.0), 1.0)
    assert J == 3.0 and kind == 2
    X = np.zeros((4, 4)); X[1, 2] = 8.0
    J, kind = orc.fluctuation_metric(X, 2.5)                  # ||X||_F = 8, sqrt(16) = 4
    assert J == 2.0 and kind == 1
    rng = np.random.default_rng(1)
    X = rng.standard_normal((300, 200))
    J, _ = orc.fluctuation_metric(X)
    assert abs(J - np.linalg.norm(X) / np.sqrt(X.size)) <= 1e-13 * J          # library norm
    assert abs(J - np.sqrt(X.var() + X.mean() ** 2)) <= 1e-12                 # rms = sqrt(var + mean^2)
    J2, _ = orc.fluctuation_metric(-2.5 * X)
    assert abs(J2 - 2.5 * J) <= 1e-13 * J2                                    # homogeneous of degree one
    Jt, _ = orc.fluctuation_metric(X.T.copy())
    assert abs(Jt - J) <= 1e-13 * J                                           # only the element count matters


def test_threshold_rule_separates_the_two_activation_families(orc):
    # Eq. 12 with the paper's threshold 1: mild-outlier layers stay near J = 1 (unit-variance base), layers with
    # salient channels sit far above it.  The threshold itself: J < thr -> Hadamard, J >= thr -> dense.
    mild = bf16_bits_to_f64(make_activations(5, 256, 512, n_salient=0, mild_p=0.0))
    sal = bf16_bits_to_f64(make_activations(6, 256, 512, n_salient=16, salient_x=100.0))
    Jm, km = orc.fluctuation_metric(mild, 1.05)
    Js, ks = orc.fluctuation_metric(sal, 1.05)
    assert 0.95 < Jm < 1.05 and km == 1
    assert Js > 10 and ks == 2
    X = np.ones((2, 2))
    assert orc.fluctuation_metric(X, 1.0)[1] == 2 and orc.fluctuation_metric(X, 1.0 + 1e-12)[1] == 1
