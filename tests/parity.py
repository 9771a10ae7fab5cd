"""Helpers of the GPU parity tests: run a layer through the CUDA library (via the C ABI) and through
the oracle on the same seeded arrays, and compare with the stated tolerances.

Tolerances (from the benchmark spec of this path):
  * TLQ weight codes and level tables: bit-exact;
  * activation codes: exact except 1-code differences on at most 1e-4 of the elements;
  * outputs: relative Frobenius error <= 1e-3 and max-abs error <= 1e-2 x RMS of the oracle output.
"""
from __future__ import annotations

import numpy as np
import torch

from lrq_workloads import LayerSpec, bf16_bits_to_f64, default_clip_grid

ACT_FLIP_FRACTION = 1e-4
OUT_REL_FRO = 1e-3
OUT_MAXABS_RMS = 1e-2


def bf16_to_device(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def unpack4(packed: np.ndarray) -> np.ndarray:
    """[R, C/2] uint8 -> [R, C] with element 2j in the low nibble of byte j."""
    lo = packed & 0xF
    hi = packed >> 4
    return np.stack([lo, hi], axis=-1).reshape(packed.shape[0], -1)


def act_codes_to_numpy(codes: torch.Tensor, a_bits: int) -> np.ndarray:
    c = codes.cpu().numpy()
    return (unpack4(c) if a_bits == 4 else c).astype(np.int32)


def check_act(gpu_q, gpu_s, gpu_z, orc_q, orc_s, orc_z, what="", flip_fraction=ACT_FLIP_FRACTION):
    """Compare activation codes / scales / zero-points.  A token whose zero-point differs by one has all
    its codes shifted by one while q + z is unchanged; such tokens are compared on q + z."""
    gpu_q = np.asarray(gpu_q, dtype=np.int64)
    orc_q = np.asarray(orc_q, dtype=np.int64)
    gz, oz = np.asarray(gpu_z, dtype=np.int64), np.asarray(orc_z, dtype=np.int64)
    assert np.allclose(np.asarray(gpu_s, dtype=np.float64), orc_s, rtol=2e-5, atol=0), f"{what}: scales differ"
    zflip = gz != oz
    assert np.abs(gz - oz).max() <= 1, f"{what}: zero-point off by more than one"
    assert zflip.sum() <= max(1, 0.01 * zflip.size), f"{what}: too many zero-point flips ({zflip.sum()})"
    d = (gpu_q + gz[:, None]) - (orc_q + oz[:, None])        # difference of q + z (equals q diff when z agrees)
    # clamping at the ends can hide a shift on z-flipped tokens; allow it there
    bad = np.abs(d) > 1
    assert not bad[~zflip].any(), f"{what}: a code differs by more than one"
    frac = (d[~zflip] != 0).mean() if (~zflip).any() else 0.0
    assert frac <= flip_fraction, f"{what}: {frac:.2e} of the codes differ (limit {flip_fraction})"
    return float(frac), int(zflip.sum())


def check_out(y_gpu: np.ndarray, y_orc: np.ndarray, what="", rel=OUT_REL_FRO, mx=OUT_MAXABS_RMS):
    y_gpu = np.asarray(y_gpu, dtype=np.float64)
    fro = np.linalg.norm(y_gpu - y_orc) / max(np.linalg.norm(y_orc), 1e-300)
    rms = np.sqrt(np.mean(y_orc ** 2))
    mabs = np.abs(y_gpu - y_orc).max() / max(rms, 1e-300)
    assert fro <= rel, f"{what}: relative Frobenius error {fro:.3e} > {rel}"
    assert mabs <= mx, f"{what}: max-abs error {mabs:.3e} x RMS > {mx}"
    return float(fro), float(mabs)


def check_layer_out(orc, spec, T, y_gpu, gpu_q, gpu_z, Yo, oq, os_, oz, what="", **tol):
    """Output parity of a whole layer.  A token whose activation codes (or zero-point) differ from the oracle's
    sits on a rounding boundary of Eq. 1, where both roundings are valid; its reference row is the oracle's
    contraction (Eq. 10) evaluated on the codes the GPU chose.  All other rows are the oracle's own pipeline.
    The number of such tokens is bounded separately by check_act."""
    gpu_q = np.asarray(gpu_q, dtype=np.int32)
    diff = (gpu_q != oq).any(axis=1) | (np.asarray(gpu_z) != oz)
    ref = Yo
    if diff.any():
        ref = Yo.copy()
        idx = np.nonzero(diff)[0]
        ref[idx] = orc.qmatmul(gpu_q[idx], os_[idx], np.asarray(gpu_z, dtype=np.int32)[idx], T)
    fro, mabs = check_out(y_gpu, ref, what, **tol)
    return fro, mabs, int(diff.sum())


def check_tlq(orc, W: np.ndarray, tl, bits: int, group: int, rows=None, what=""):
    """Bit-exact comparison of GPU TLQ results `tl` (TLQWeights) against the oracle on W[rows]."""
    g = default_clip_grid()
    rows = np.arange(W.shape[0]) if rows is None else np.asarray(rows)
    T = orc.tlq_quantize(W[rows].astype(np.float64), bits, group, 7, g, g)
    half = 1 << (bits - 1)
    # A (row, group) whose best and second-best clipping factors tie to within fp64 summation noise has two
    # valid answers (the order of the sum decides); such rows are compared only if the same factor was chosen.
    gm = tl.meta.cpu().numpy()[rows]
    tie = (T.margin < 1e-10).any(axis=1) & ~(gm[..., 4:] == T.meta[..., 4:]).all(axis=(1, 2))
    assert tie.sum() <= max(1, len(rows) // 100), f"{what}: too many tied searches resolved differently"
    keep = ~tie
    gc = unpack4(tl.codes.cpu().numpy())[rows].astype(np.int32) - half
    assert np.array_equal(gc[keep], T.codes.astype(np.int32)[keep]), \
        f"{what}: {np.count_nonzero(gc[keep] != T.codes[keep])} TLQ codes differ"
    gl = tl.levels.cpu().numpy()[rows]
    assert np.array_equal(gl[keep], T.levels.astype(np.float32)[keep]), f"{what}: level tables differ"
    assert np.array_equal(gl.astype(np.float64)[keep], T.levels[keep]), f"{what}: a level is not exactly an fp32 number"
    assert np.allclose(gm[keep], T.meta[keep], rtol=1e-13, atol=0), f"{what}: TLQ parameters differ"
    assert np.array_equal(gm[keep][..., 4:], T.meta[keep][..., 4:]), f"{what}: chosen clipping factors differ"
    gw = tl.wsum.cpu().numpy()[rows].astype(np.float64)
    scale = np.abs(T.levels).max(axis=(1, 2)) * np.sqrt(W.shape[1])
    assert (np.abs(gw - T.wsum) <= 1e-6 * scale + 1e-30)[keep].all(), f"{what}: wsum differs"
    return T


def gpu_layer(spec: LayerSpec, W: np.ndarray, P):
    """Quantize weights on the GPU and build the layer handle.  Returns (QLayer, TLQWeights)."""
    g = default_clip_grid()
    Wd = torch.from_numpy(W).cuda()
    tl = P.lrq_tlq_quantize_weights(Wd, spec.w_bits, spec.group, 7, g, g)
    R = None
    if spec.rot == "dense":
        R = bf16_to_device(spec.rotation_bf16())
    kind = P.ROT_DENSE if spec.rot == "dense" else P.ROT_HADAMARD
    return P.QLayer(tl, spec.N, spec.K, kind, spec.a_bits, spec.had_block, R), tl


def oracle_layer_rows(orc, spec: LayerSpec, Xbits_rows: np.ndarray, T, R_bits=None):
    X = bf16_bits_to_f64(Xbits_rows)
    R = None if R_bits is None else bf16_bits_to_f64(R_bits)
    return orc.qlinear(X, T, spec.a_bits, spec.rot, spec.had_block, R)
