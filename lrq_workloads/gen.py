"""Seeded generators for the five DiT-shaped workloads.

Everything here is a random draw or a number-format conversion.  The shapes follow the
public architectures the paper evaluates (PixArt, MMDiT/FLUX-style joint attention, a
video DiT); the value distributions follow the paper's description of DiT tensors:
long-tailed, zero-mean weights (Sec. 4.1, "Motivation"), mild activation outliers that
rarely exceed 5 and salient outliers confined to fixed channels on every token
(Sec. 4.2, "Motivation").  Generator: numpy ``Generator(PCG64(seed))``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import numpy as np


# ----------------------------------------------------------------------------- formats
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# ----------------------------------------------------------------------------- draws
def make_weights(seed: int, N: int, K: int, nu: float = 4.0, std: float = 0.02) -> np.ndarray:
    """[N, K] float32, Student-t with ``nu`` degrees of freedom scaled to standard deviation ``std``.

    These are the weights *in the rotated basis* (the array handed to TLQ); the un-rotated
    matrix is never needed by the inference path.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    w = rng.standard_t(nu, size=(N, K)) * (std / np.sqrt(nu / (nu - 2.0)))
    return w.astype(np.float32)


def make_activations(seed: int, M: int, K: int, mild_p: float = 0.005, mild_x: float = 5.0,
                     n_salient: int = 8, salient_x: float = 60.0, chunk: int = 4096) -> np.ndarray:
    """[M, K] bfloat16 bit patterns (uint16).

    N(0,1) base; a Bernoulli(``mild_p``) subset of entries multiplied by ``mild_x`` (mild
    outliers); ``n_salient`` channels, drawn once, multiplied by ``salient_x`` on every token
    (salient outliers).  Rows are produced in chunks so that M = 32768 x K = 4608 stays cheap.
    """
    rng = np.random.Generator(np.random.PCG64(seed + 1_000_003))
    sal = rng.choice(K, size=n_salient, replace=False) if n_salient > 0 else np.zeros(0, dtype=np.int64)
    out = np.empty((M, K), dtype=np.uint16)
    for m0 in range(0, M, chunk):
        m1 = min(M, m0 + chunk)
        x = rng.standard_normal(size=(m1 - m0, K), dtype=np.float32)
        if mild_p > 0:
            mask = rng.random(size=x.shape, dtype=np.float32) < mild_p
            x[mask] *= np.float32(mild_x)
        if n_salient > 0:
            x[:, sal] *= np.float32(salient_x)
        out[m0:m1] = f32_to_bf16_bits(x)
    return out


def make_orthogonal(seed: int, K: int) -> np.ndarray:
    """[K, K] float64 orthogonal matrix: Q of the QR factorisation of a seeded Gaussian matrix,
    column signs fixed so that diag(R) > 0 (Haar-distributed).  Stands in for the composed
    outlier-aware rotation, which the inference path receives as one dense matrix."""
    rng = np.random.Generator(np.random.PCG64(seed + 2_000_003))
    a = rng.standard_normal(size=(K, K))
    q, r = np.linalg.qr(a)
    q *= np.sign(np.diag(r))[None, :]
    return q


def salient_channels(seed: int, K: int, n_salient: int) -> np.ndarray:
    """The channels make_activations(seed, ., K, n_salient=...) scales up on every token (its first draw)."""
    rng = np.random.Generator(np.random.PCG64(seed + 1_000_003))
    return rng.choice(K, size=n_salient, replace=False) if n_salient > 0 else np.zeros(0, dtype=np.int64)


def make_block_rotations(seed: int, K: int, Bd: int) -> np.ndarray:
    """[K/Bd, Bd, Bd] float64: one Haar-distributed orthogonal matrix per block of Bd channels.  Stands in for a
    block-diagonal outlier-aware rotation, whose construction from calibration data is outside the path."""
    assert K % Bd == 0
    rng = np.random.Generator(np.random.PCG64(seed + 3_000_017))
    out = np.empty((K // Bd, Bd, Bd))
    for j in range(K // Bd):
        q, r = np.linalg.qr(rng.standard_normal(size=(Bd, Bd)))
        out[j] = q * np.sign(np.diag(r))[None, :]
    return out


def make_staggered_permutation(seed: int, K: int, Bd: int, first: np.ndarray | None = None) -> np.ndarray:
    """int32 [K] index map of a staggered channel reordering: position i of the reordered vector takes channel
    perm[i].  The channels are put in a ranking (those of ``first`` lead, in the given order; the rest follow in a
    seeded random order, standing in for a ranking by calibrated range) and dealt over the K/Bd blocks back and
    forth: ranks 0..nb-1 to blocks 0..nb-1, ranks nb..2nb-1 to blocks nb-1..0, and so on, each pass filling the
    next slot of every block.  So the leading channels end up spread over different blocks."""
    assert K % Bd == 0
    nb = K // Bd
    rng = np.random.Generator(np.random.PCG64(seed + 4_000_037))
    first = np.zeros(0, dtype=np.int64) if first is None else np.asarray(first, dtype=np.int64)
    rest = np.setdiff1d(np.arange(K), first)
    ranking = np.concatenate([first, rng.permutation(rest)])
    perm = np.empty(K, dtype=np.int32)
    for r, ch in enumerate(ranking):
        p, pos = divmod(r, nb)
        b = pos if p % 2 == 0 else nb - 1 - pos
        perm[b * Bd + p] = ch
    return perm


def default_clip_grid() -> np.ndarray:
    """Grid of clipping factors handed to the TLQ search: 1.00, 1.02, ..., 1.60."""
    return np.round(1.0 + 0.02 * np.arange(31), 2)


# ----------------------------------------------------------------------------- configs
@dataclass
class LayerSpec:
    name: str
    seed: int
    M: int
    K: int
    N: int
    w_bits: int
    a_bits: int
    group: int            # 0 => per output channel
    rot: str              # "hadamard" | "dense" | "dual" (a dense layer with its rotation kept in factors)
    had_block: int        # block size of the block-diagonal Hadamard (0 for dense)
    nu: float = 4.0
    w_std: float = 0.02
    mild_p: float = 0.005
    mild_x: float = 5.0
    n_salient: int = 8
    salient_x: float = 60.0

    def weights(self) -> np.ndarray:
        return make_weights(self.seed, self.N, self.K, self.nu, self.w_std)

    def activations(self, M: int | None = None) -> np.ndarray:
        return make_activations(self.seed, self.M if M is None else M, self.K, self.mild_p,
                                self.mild_x, self.n_salient, self.salient_x)

    def rotation_bf16(self) -> np.ndarray | None:
        """Dense rotation as bf16 bit patterns [K, K] (y = x @ R), or None for Hadamard layers."""
        if self.rot != "dense":
            return None
        return f32_to_bf16_bits(make_orthogonal(self.seed, self.K).astype(np.float32))


    def dual_factors(self, Bd: int = 128):
        """(Bd, R1 bf16 bits [K/Bd,Bd,Bd], perm int32 [K], R2 bf16 bits [K/Bd,Bd,Bd]) of a seeded dual transformation
        y = x . blockdiag(R1) . P . blockdiag(R2); the permutation leads with this layer's salient channels."""
        R1 = f32_to_bf16_bits(make_block_rotations(self.seed, self.K, Bd).astype(np.float32))
        R2 = f32_to_bf16_bits(make_block_rotations(self.seed + 7, self.K, Bd).astype(np.float32))
        perm = make_staggered_permutation(self.seed, self.K, Bd, salient_channels(self.seed, self.K, self.n_salient))
        return Bd, R1, perm, R2


def _largest_pow2_divisor(k: int) -> int:
    return k & (-k)


def _cfg0() -> List[LayerSpec]:
    return [LayerSpec("linear", 0, 256, 1024, 1024, 3, 4, 0, "hadamard", 1024)]


def _cfg1() -> List[LayerSpec]:
    shapes = [("qkv", 1152, 3456), ("proj", 1152, 1152), ("fc1", 1152, 4608), ("fc2", 4608, 1152)]
    return [LayerSpec(n, 1 + i, 4096, k, o, 4, 8, 0, "hadamard", 128) for i, (n, k, o) in enumerate(shapes)]


def _cfg2() -> List[LayerSpec]:
    M = 4096 + 333
    mk = lambda n, s, k, o, rot: LayerSpec(
        n, s, M, k, o, 3, 4, 128, rot, 0 if rot == "dense" else _largest_pow2_divisor(k),
        n_salient=16 if rot == "dense" else 0, salient_x=100.0)
    return [mk("qkv", 5, 1536, 4608, "hadamard"), mk("proj", 6, 1536, 1536, "dense"),
            mk("fc1", 7, 1536, 6144, "dense"), mk("fc2", 8, 6144, 1536, "hadamard")]


def _cfg3() -> List[LayerSpec]:
    M = 4096 + 512
    mk = lambda n, s, k, o, rot: LayerSpec(
        n, s, M, k, o, 4, 4, 0, rot, 0 if rot == "dense" else min(4096, _largest_pow2_divisor(k)),
        nu=3.0, w_std=0.015, mild_p=0.01, mild_x=6.0,
        n_salient=32 if rot == "dense" else 0, salient_x=80.0)
    return [mk("qkv", 9, 3072, 9216, "dense"), mk("fc1", 10, 3072, 12288, "hadamard"),
            mk("fc2", 11, 12288, 3072, "hadamard")]


def _cfg4(n_blocks: int = 28, p_dense: float = 0.05) -> List[LayerSpec]:
    M = 2 * 16 * 1024
    rng = np.random.Generator(np.random.PCG64(12))
    shapes = [("qkv", 1152, 3456), ("proj", 1152, 1152), ("fc1", 1152, 4608), ("fc2", 4608, 1152)]
    out = []
    for b in range(n_blocks):
        for j, (n, k, o) in enumerate(shapes):
            dense = bool(rng.random() < p_dense) and k == 1152
            out.append(LayerSpec(f"b{b}.{n}", 1200 + 4 * b + j, M, k, o, 4, 8, 0,
                                 "dense" if dense else "hadamard", 0 if dense else 128))
    return out


CONFIGS = {0: _cfg0, 1: _cfg1, 2: _cfg2, 3: _cfg3, 4: _cfg4}


def config_layers(cfg: int, **kw) -> List[LayerSpec]:
    """Layer list of workload ``cfg`` (0..4)."""
    return CONFIGS[cfg](**kw)
