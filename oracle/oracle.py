"""ctypes front-end of the fp64 CPU oracle in ``lrq_oracle.c``.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the bench's
CPU-baseline leg.  It shares nothing with the CUDA library and never imports it.
All arrays are numpy, double precision unless stated; every function cites the passage of the
paper its C routine follows.  Parity-unpinned readings are listed in the C file's header.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lrq_oracle.c")
_LIB = os.path.join(_HERE, "liblrq_oracle.so")

__all__ = [
    "build", "num_threads", "hadamard_matrix", "rotate_hadamard_explicit", "rotate_hadamard_fwht",
    "rotate_dense", "rotate_dual", "quantize_act", "dequantize_act", "level_value", "tlq_quantize", "qmatmul",
    "TLQResult", "qlinear", "smooth", "fluctuation_metric", "rotate_weights",
]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-D_GNU_SOURCE",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None
_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int32)
_bp = ctypes.POINTER(ctypes.c_int8)


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_level_value.restype = ctypes.c_double
        _lib.orc_level_value.argtypes = [ctypes.c_double, ctypes.c_int]
        _lib.orc_fluctuation_metric.restype = ctypes.c_double
        _lib.orc_fluctuation_metric.argtypes = [_dp, ctypes.c_int, ctypes.c_int, ctypes.c_double, _ip]
    return _lib


def _d(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(_dp)


def num_threads() -> int:
    return int(_L().orc_num_threads())


def hadamard_matrix(n: int) -> np.ndarray:
    """Normalised Sylvester matrix H_n by the Kronecker recursion (Sec. 3.2, Eq. 3)."""
    H = np.zeros((n, n))
    rc = _L().orc_hadamard_matrix(int(n), H.ctypes.data_as(_dp))
    if rc:
        raise ValueError("n must be a power of two")
    return H


def _rot(fn, X, B):
    X, xp = _d(X)
    M, K = X.shape
    Y = np.empty_like(X)
    rc = fn(xp, M, K, int(B), Y.ctypes.data_as(_dp))
    if rc:
        raise ValueError("block size must be a power of two dividing K")
    return Y


def rotate_hadamard_explicit(X, B):
    """y = x . blockdiag(H_B) as an explicit matrix product (Sec. 4.2, Eq. 12, first case)."""
    return _rot(_L().orc_rotate_hadamard_explicit, X, B)


def rotate_hadamard_fwht(X, B):
    """The same map through the butterfly factorisation of Eq. 3."""
    return _rot(_L().orc_rotate_hadamard_fwht, X, B)


def rotate_dense(X, R):
    """y = x . R for a dense K x K rotation (Sec. 4.2, Eq. 12, second case)."""
    X, xp = _d(X)
    R, rp = _d(R)
    M, K = X.shape
    assert R.shape == (K, K)
    Y = np.empty_like(X)
    _L().orc_rotate_dense(xp, M, K, rp, Y.ctypes.data_as(_dp))
    return Y


def rotate_dual(X, Bd: int, R1, perm, R2):
    """y = x . R1hat . P . R2hat, the dual transformation of Sec. 4.2 in its factors: R1hat and R2hat
    block-diagonal with blocks R1[j], R2[j] of Bd x Bd (arrays [K/Bd, Bd, Bd]); P as the index map
    (u P)_i = u[perm[i]]."""
    X, xp = _d(X)
    R1, r1p = _d(R1)
    R2, r2p = _d(R2)
    M, K = X.shape
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    assert K % Bd == 0 and R1.shape == (K // Bd, Bd, Bd) and R2.shape == R1.shape and perm.shape == (K,)
    Y = np.empty_like(X)
    rc = _L().orc_rotate_dual(xp, M, K, int(Bd), r1p, perm.ctypes.data_as(_ip), r2p, Y.ctypes.data_as(_dp))
    if rc:
        raise ValueError("Bd must divide K and perm must be a permutation of range(K)")
    return Y


def smooth(X, p):
    """X diag(p): the channel-wise smoothing multipliers applied to the activations (Sec. 5.1)."""
    X, xp = _d(X)
    p, pp = _d(p)
    M, K = X.shape
    assert p.shape == (K,)
    Y = np.empty_like(X)
    _L().orc_smooth(xp, M, K, pp, Y.ctypes.data_as(_dp))
    return Y


def rotate_weights(W, colmul=None, rot: str = "hadamard", had_block: int = 0, R=None, dual=None):
    """The weight side of Eq. 2, (X R)(W R)^T = X W^T: the rows of W diag(colmul) mapped by the layer's rotation
    (Sec. 3.2; colmul is the reciprocal of the activations' smoothing multipliers, Sec. 5.1).  The same maps the
    activations take, applied to weight rows."""
    W = np.asarray(W, dtype=np.float64)
    if colmul is not None:
        W = smooth(W, np.asarray(colmul, dtype=np.float64))
    if rot == "hadamard":
        return rotate_hadamard_fwht(W, had_block)
    if rot == "dense":
        return rotate_dense(W, R)
    if rot == "dual":
        return rotate_dual(W, *dual)
    if rot == "none":
        return W.copy()
    raise ValueError(rot)


def fluctuation_metric(X, thr: float = 1.0):
    """J = ||X||_F / sqrt(B N C) (Sec. 4.2, Eq. 11) and the rotation kind Eq. 12 picks:
    1 = Hadamard (J < thr), 2 = outlier-aware dense rotation.  Returns (J, kind)."""
    X, xp = _d(X)
    M, K = X.shape
    kind = ctypes.c_int32(0)
    J = _L().orc_fluctuation_metric(xp, M, K, float(thr), ctypes.byref(kind))
    return float(J), int(kind.value)


def quantize_act(Y, bits: int, mode: int = 0):
    """Per-token uniform quantizer (Sec. 3.1, Eq. 1).  Returns (codes int32 [M,K], s [M], z int32 [M])."""
    Y, yp = _d(Y)
    M, K = Y.shape
    Q = np.empty((M, K), dtype=np.int32)
    S = np.empty(M)
    Z = np.empty(M, dtype=np.int32)
    rc = _L().orc_quantize_act(yp, M, K, int(bits), int(mode), Q.ctypes.data_as(_ip), S.ctypes.data_as(_dp),
                               Z.ctypes.data_as(_ip))
    if rc:
        raise ValueError("bad bit-width")
    return Q, S, Z


def dequantize_act(Q, S, Z):
    """x_f = s (q + z) (Eq. 1, second line)."""
    Q = np.ascontiguousarray(Q, dtype=np.int32)
    S, sp = _d(S)
    Z = np.ascontiguousarray(Z, dtype=np.int32)
    M, K = Q.shape
    X = np.empty((M, K))
    _L().orc_dequantize_act(Q.ctypes.data_as(_ip), sp, Z.ctypes.data_as(_ip), M, K, X.ctypes.data_as(_dp))
    return X


def level_value(e: float, I: int) -> float:
    """Value of the level with log-domain exponent e (Eqs. 8-9; I < 0: Eq. 7)."""
    return float(_L().orc_level_value(float(e), int(I)))


@dataclass
class TLQResult:
    codes: np.ndarray    # int8 [N,K], signed code c
    levels: np.ndarray   # float64 [N,K/G,2^b], entry u = c + 2^(b-1)
    meta: np.ndarray     # float64 [N,K/G,6]: s+, z+, s-, z-, alpha, beta
    wsum: np.ndarray     # float64 [N]
    margin: np.ndarray   # float64 [N,K/G]
    bits: int
    group: int


def tlq_quantize(W, bits: int, group: int = 0, I: int = 7, alpha=(1.0,), beta=(1.0,)) -> TLQResult:
    """Twin-log quantization with search-based clipping (Sec. 4.1, Eqs. 4-9)."""
    W, wp = _d(W)
    N, K = W.shape
    G = K if group <= 0 else int(group)
    if K % G:
        raise ValueError("group must divide K")
    ng, nl = K // G, 1 << bits
    al, alp = _d(np.atleast_1d(alpha))
    be, bep = _d(np.atleast_1d(beta))
    codes = np.empty((N, K), dtype=np.int8)
    levels = np.empty((N, ng, nl))
    meta = np.empty((N, ng, 6))
    wsum = np.empty(N)
    margin = np.empty((N, ng))
    rc = _L().orc_tlq_quantize(wp, N, K, int(bits), G, int(I), alp, al.size, bep, be.size,
                               codes.ctypes.data_as(_bp), levels.ctypes.data_as(_dp), meta.ctypes.data_as(_dp),
                               wsum.ctypes.data_as(_dp), margin.ctypes.data_as(_dp))
    if rc:
        raise ValueError("bad TLQ arguments")
    return TLQResult(codes, levels, meta, wsum, margin, int(bits), G)


def qmatmul(Q, S, Z, tlq: TLQResult, wscale=None, bias=None):
    """Quantized contraction and epilogue (Sec. 4.1, Eq. 10 evaluated exactly)."""
    Q = np.ascontiguousarray(Q, dtype=np.int32)
    S, sp = _d(S)
    Z = np.ascontiguousarray(Z, dtype=np.int32)
    M, K = Q.shape
    N = tlq.codes.shape[0]
    assert tlq.codes.shape[1] == K
    Y = np.empty((M, N))
    ws = wsp = bs = bsp = None
    if wscale is not None:
        ws, wsp = _d(wscale)
    if bias is not None:
        bs, bsp = _d(bias)
    lv, lvp = _d(tlq.levels)
    cd = np.ascontiguousarray(tlq.codes, dtype=np.int8)
    rc = _L().orc_qmatmul(Q.ctypes.data_as(_ip), sp, Z.ctypes.data_as(_ip), M, K, cd.ctypes.data_as(_bp), lvp,
                          N, tlq.group, tlq.bits, wsp, bsp, Y.ctypes.data_as(_dp))
    if rc:
        raise ValueError("bad qmatmul arguments")
    return Y


def qlinear(X, tlq: TLQResult, a_bits: int, rot: str, had_block: int = 0, R=None, mode: int = 0,
            wscale=None, bias=None, prescale=None, return_rotated: bool = False, dual=None):
    """The whole layer on already-widened inputs: [smooth (Sec. 5.1) ->] rotate (Eq. 12) -> per-token
    quantize (Eq. 1) -> contraction with the TLQ table and epilogue (Eq. 10).  Returns (Y, codes, s, z), and with
    return_rotated also the rotated activations that Eq. 1 quantized."""
    if prescale is not None:
        X = smooth(X, prescale)
    if rot == "hadamard":
        Yr = rotate_hadamard_fwht(X, had_block)
    elif rot == "dense":
        Yr = rotate_dense(X, R)
    elif rot == "dual":
        Yr = rotate_dual(X, *dual)                     # dual = (Bd, R1, perm, R2)
    elif rot == "none":
        Yr = np.ascontiguousarray(X, dtype=np.float64)
    else:
        raise ValueError(rot)
    Q, S, Z = quantize_act(Yr, a_bits, mode)
    Y = qmatmul(Q, S, Z, tlq, wscale, bias)
    return (Y, Q, S, Z, Yr) if return_rotated else (Y, Q, S, Z)
