"""Helpers of the GPU parity tests: run a layer through the CUDA library (via the C ABI) and through
the oracle on the same seeded arrays, and compare with the stated tolerances.

Tolerances:
  * TLQ weight codes, level tables, chosen clipping factors: bit-exact;
  * activation codes: exact, except that an element whose exact y/s lies on a rounding boundary of Eq. 1
    (within the fp32 error of the path, derived below) may take the neighbouring code, on at most 1e-4 of
    the elements;
  * outputs: relative Frobenius error <= 1e-3 and max-abs error <= 1e-2 x RMS of the oracle output.

Where two answers are valid (Eq. 1 rounds y/s, and the kernels hold y/s in fp32):
  * the oracle's own fp64 t = y/s of a differing element must satisfy |frac(t) - 1/2| <= boundary_tol: the
    element is on a rounding boundary to within what fp32 arithmetic can resolve.  Anything else is an error.
  * an exact tie (|frac(t) - 1/2| below fp64 noise: the inputs sit on a coarse grid and s divides them) has two
    equally valid codes even in exact arithmetic; such elements are checked for validity (one code apart) and
    not counted against the 1e-4 allowance.
  * a token whose min/s is on a boundary may take the neighbouring zero-point; all its codes then shift by
    one while q + z is unchanged.  Such tokens are compared on q + z (which is unique), need the same boundary
    proof on min/s, and may be at most 1e-4 of the tokens (plus one).

boundary_tol, in code steps, for an element with t = y/s of a token with zero-point z (fp32 unit u = 2^-24):
    the quantizer evaluates fma(y_fp32, (float)(1/s), -z): the reciprocal's rounding and the fma's rounding each
      move t by at most u * (|t| + |z|); the step s itself comes from fp32 extremes (another u * |t| each);
    the rotation that produced y_fp32:
      Hadamard, log2(B) butterfly stages: every add rounds by u relative to its result; summed over the stages
        the error of an output has rms u * sqrt(log2(B) / 3) * rms(y) (independent roundings, each stage's
        errors spread over the later stages' outputs with the same gain as the signal);
      dense, K products (exact) accumulated in fp32 on the tensor cores in K/16 chained instructions whose adds
        round toward zero: each loses up to one ulp (2u) of the running sum, half of that on average.  The part
        common to a token's elements (a uniform shrink) cancels in y/s; what is left is bounded here by
        (K/32) * u * rms(y), half an ulp per chained add (measured worst case: 0.45 of it at K = 3072);
      dual (two block-diagonal products of Bd-wide blocks, the second over the three bf16 terms of the first one's
        fp32 result): Bd/16 chained adds, then 3 Bd/16 of them, counted as for the dense product: (4 Bd / 32) * u *
        rms(y) (the second rotation is orthogonal, so the first product's error keeps its size on the way through;
        what the three-term split drops, 2^-25 of each element, is below one rounding);
      none: y is the bf16 input, exact.
    tol = u * (4 * (|t| + |z| + 1) + g * rms(y)/s),  g = sqrt(log2 B), K/32, Bd/8 or 0
    (the first term is a worst-case bound; measured on the five workloads, differing elements sit within 0.2 tol).
Scale tolerance: s is (max - min) / (2^b - 1) of fp32 extremes, evaluated in fp64 and rounded to fp32 once:
    Hadamard / none: 5e-7 relative = 8 u (the fp32 rounding of s itself is u; the extremes' rotation error is a few u
    of their magnitude; measured 1e-7);
    dense: the extremes carry the tensor-core accumulation error; if every one of the K/16 accumulations
    truncated in the same direction the relative error would reach (K/16) * 2^-23, which is the bound used
    (2.3e-5 at K = 3072; measured 2.7e-6 at K = 1536); never below 5e-7;
    dual: the same with the 4 Bd / 16 chained accumulations of its two products (3.8e-6 for Bd = 128).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from lrq_workloads import LayerSpec, bf16_bits_to_f64, default_clip_grid

ACT_FLIP_FRACTION = 1e-4
OUT_REL_FRO = 1e-3
OUT_MAXABS_RMS = 1e-2
BOUNDARY_C = 1.0
U32 = 2.0 ** -24
EXACT_TIE = 2.0 ** -40          # |frac(t) - 1/2| below this (relative to |t| + 1) is an exact tie in fp64


def bf16_to_device(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def unpack4(packed: np.ndarray) -> np.ndarray:
    """[R, C/2] uint8 -> [R, C] with element 2j in the low nibble of byte j."""
    lo = packed & 0xF
    hi = packed >> 4
    return np.stack([lo, hi], axis=-1).reshape(packed.shape[0], -1)


def unpack3(packed: np.ndarray) -> np.ndarray:
    """[R, 3C/8] uint8 -> [R, C]: eight 3-bit codes per 3 bytes, code j at bits 3j..3j+2 of the little-endian
    24-bit word."""
    p = packed.reshape(packed.shape[0], -1, 3).astype(np.uint32)
    w = p[..., 0] | (p[..., 1] << 8) | (p[..., 2] << 16)
    return np.stack([(w >> (3 * j)) & 7 for j in range(8)], axis=-1).reshape(packed.shape[0], -1).astype(np.uint8)


def act_codes_to_numpy(codes: torch.Tensor, a_bits: int) -> np.ndarray:
    c = codes.cpu().numpy()
    return (unpack4(c) if a_bits == 4 else c).astype(np.int32)


def rotation_gain(rot: str, K: int, had_block: int = 0) -> float:
    """g of the boundary tolerance (module docstring) for a rotation kind."""
    if rot == "hadamard":
        return float(np.sqrt(max(1.0, np.log2(max(had_block, 2)))))
    if rot == "dense":
        return float(K / 32.0)
    if rot == "dual":                      # had_block carries Bd
        return float(had_block / 8.0)
    if rot == "none":
        return 0.0
    raise ValueError(rot)


def scale_rtol(rot: str, K: int, had_block: int = 0) -> float:
    if rot == "dense":
        return max(5e-7, (K / 16.0) * 2.0 ** -23)
    if rot == "dual":                      # had_block carries Bd
        return max(5e-7, (4 * had_block / 16.0) * 2.0 ** -23)
    return 5e-7


@dataclass
class ActCheck:
    flip_fraction: float        # share of elements whose code differs and that are not exact ties
    tie_fraction: float         # share of elements that differ on an exact tie
    z_flips: int                # tokens whose zero-point differs (boundary-proven)
    diff_tokens: np.ndarray     # bool [M]: tokens with any differing code or zero-point (all boundary-proven)
    worst_boundary: float       # max over differing elements of |frac(t) - 1/2| / boundary_tol   (<= 1)
    worst_scale: float          # max relative scale difference / scale_rtol                       (<= 1)


def _half_distance(t: np.ndarray) -> np.ndarray:
    """|frac(t) - 1/2| for fp64 t: distance of t from the nearest rounding boundary of rint."""
    return np.abs(t - np.floor(t) - 0.5)


def check_act(gpu_q, gpu_s, gpu_z, orc_q, orc_s, orc_z, orc_y, rot, had_block=0, what="",
              flip_fraction=ACT_FLIP_FRACTION) -> ActCheck:
    """Compare activation codes / scales / zero-points with the oracle's.  `orc_y` are the oracle's rotated fp64
    values (the input of Eq. 1) for the same tokens; `rot`, `had_block` name the path for the tolerances above."""
    gpu_q = np.asarray(gpu_q, dtype=np.int64)
    orc_q = np.asarray(orc_q, dtype=np.int64)
    orc_y = np.asarray(orc_y, dtype=np.float64)
    M, K = orc_q.shape
    assert gpu_q.shape == orc_q.shape == orc_y.shape
    gz, oz = np.asarray(gpu_z, dtype=np.int64), np.asarray(orc_z, dtype=np.int64)
    gs, os_ = np.asarray(gpu_s, dtype=np.float64), np.asarray(orc_s, dtype=np.float64)
    rtol = scale_rtol(rot, K, had_block)
    rel_s = np.abs(gs - os_) / os_
    assert (rel_s <= rtol).all(), f"{what}: scales differ by {rel_s.max():.2e} relative (limit {rtol:.1e})"

    g = rotation_gain(rot, K, had_block)
    rms = np.sqrt(np.mean(orc_y ** 2, axis=1))
    tol_rot = BOUNDARY_C * U32 * g * rms / os_                                   # [M]

    def tol_of(t, z):                                                            # boundary_tol, element-wise
        return BOUNDARY_C * U32 * 4.0 * (np.abs(t) + np.abs(z) + 1.0)

    worst = 0.0
    # zero-points: a flip needs min/s (asymmetric mode) on a boundary
    zflip = gz != oz
    if zflip.any():
        assert np.abs(gz - oz).max() <= 1, f"{what}: zero-point off by more than one"
        idx = np.nonzero(zflip)[0]
        tmin = orc_y[idx].min(axis=1) / os_[idx]
        hd, tol = _half_distance(tmin), tol_of(tmin, oz[idx]) + tol_rot[idx]
        assert (hd <= tol).all(), f"{what}: a zero-point differs although min/s is {hd.max():.2e} from a boundary"
        worst = max(worst, float((hd / tol).max()))
        assert zflip.sum() <= int(ACT_FLIP_FRACTION * M) + 1, \
            f"{what}: too many zero-point flips ({zflip.sum()} of {M} tokens)"
    # codes, compared on q + z (equals the code difference wherever z agrees)
    d = (gpu_q + gz[:, None]) - (orc_q + oz[:, None])
    mm, kk = np.nonzero(d)
    n_tie = n_flip = 0
    if mm.size:
        qmax = max(int(orc_q.max()), int(gpu_q.max()))
        # on a z-flipped token the clamp at either end hides the shift: q + z differs by one on clamped elements
        clamped = zflip[mm] & ((orc_q[mm, kk] == 0) | (gpu_q[mm, kk] == 0) | (orc_q[mm, kk] >= qmax) | (gpu_q[mm, kk] >= qmax))
        assert (np.abs(d[mm, kk]) <= 1).all(), f"{what}: a code differs by more than one"
        t = orc_y[mm, kk] / os_[mm]
        hd = _half_distance(t)
        tol = tol_of(t, oz[mm]) + tol_rot[mm]
        bad = (hd > tol) & ~clamped
        assert not bad.any(), (f"{what}: {int(bad.sum())} codes differ away from a rounding boundary "
                               f"(worst |frac(y/s)-1/2| = {hd[bad].max():.3e}, allowed {tol[bad][hd[bad].argmax()]:.3e})")
        live = ~clamped
        if live.any():
            worst = max(worst, float((hd[live] / tol[live]).max()))
        tie = hd <= EXACT_TIE * (np.abs(t) + 1.0)
        n_tie = int((tie & live).sum())
        n_flip = int((~tie & live).sum())
    frac = n_flip / float(M * K)
    # a whole number of elements: a tensor of fewer than 1 / flip_fraction elements may still hold one boundary element
    assert n_flip <= np.ceil(flip_fraction * M * K), f"{what}: {frac:.2e} of the codes differ (limit {flip_fraction})"
    diff_tokens = zflip.copy()
    diff_tokens[np.unique(mm)] = True
    return ActCheck(frac, n_tie / float(M * K), int(zflip.sum()), diff_tokens, worst, float((rel_s / rtol).max()))


def check_out(y_gpu: np.ndarray, y_orc: np.ndarray, what="", rel=OUT_REL_FRO, mx=OUT_MAXABS_RMS):
    y_gpu = np.asarray(y_gpu, dtype=np.float64)
    fro = np.linalg.norm(y_gpu - y_orc) / max(np.linalg.norm(y_orc), 1e-300)
    rms = np.sqrt(np.mean(y_orc ** 2))
    mabs = np.abs(y_gpu - y_orc).max() / max(rms, 1e-300)
    assert fro <= rel, f"{what}: relative Frobenius error {fro:.3e} > {rel}"
    assert mabs <= mx, f"{what}: max-abs error {mabs:.3e} x RMS > {mx}"
    return float(fro), float(mabs)


def check_layer_out(orc, T, y_gpu, gpu_q, gpu_z, Yo, os_, act: ActCheck, what="", **tol):
    """Output parity of a whole layer.  A token that check_act has proven to sit on a rounding boundary of Eq. 1
    (`act.diff_tokens`) has two valid code vectors; its reference row is the oracle's contraction (Eq. 10)
    evaluated on the codes the GPU chose.  All other rows are the oracle's own pipeline, and the codes of those
    rows are identical by check_act.  The number of substituted rows cannot exceed the number of boundary
    elements, itself at most 1e-4 of all elements (plus exact ties)."""
    gpu_q = np.asarray(gpu_q, dtype=np.int32)
    diff = act.diff_tokens
    M, K = gpu_q.shape
    assert diff.sum() <= np.ceil((act.flip_fraction + act.tie_fraction) * M * K) + act.z_flips, \
        f"{what}: more substituted rows than boundary elements"
    ref = Yo
    if diff.any():
        ref = Yo.copy()
        idx = np.nonzero(diff)[0]
        ref[idx] = orc.qmatmul(gpu_q[idx], os_[idx], np.asarray(gpu_z, dtype=np.int32)[idx], T)
    fro, mabs = check_out(y_gpu, ref, what, **tol)
    return fro, mabs, int(diff.sum())


def check_tlq(orc, W: np.ndarray, tl, bits: int, group: int, rows=None, what="", packed3=False):
    """Bit-exact comparison of GPU TLQ results `tl` (TLQWeights) against the oracle on W[rows]: codes, level tables
    and chosen clipping factors of every (row, group), no exemption.

    The clipping search compares fp64 sums of squared errors, and two factors that give the same codes and differ
    only in their lowest level do tie to within 1e-14 relative on the workloads; the winner then depends on how the
    sum was rounded.  The library therefore takes that sum exactly as the definition reads (over the side's
    elements in increasing k, one add after another, products and sums rounded separately), which is also what the
    oracle's plain loop does, so both sides reach the same decision whatever the margin.  The margin is reported
    for the record (`T.margin`) but gates nothing."""
    g = default_clip_grid()
    rows = np.arange(W.shape[0]) if rows is None else np.asarray(rows)
    T = orc.tlq_quantize(W[rows].astype(np.float64), bits, group, 7, g, g)
    half = 1 << (bits - 1)
    gm = tl.meta.cpu().numpy()[rows]
    raw = tl.codes.cpu().numpy()
    gc = (unpack3(raw) if packed3 else unpack4(raw))[rows].astype(np.int32) - half
    assert np.array_equal(gc, T.codes.astype(np.int32)), f"{what}: {np.count_nonzero(gc != T.codes)} TLQ codes differ"
    gl = tl.levels.cpu().numpy()[rows]
    assert np.array_equal(gl, T.levels.astype(np.float32)), f"{what}: level tables differ"
    assert np.array_equal(gl.astype(np.float64), T.levels), f"{what}: a level is not exactly an fp32 number"
    assert np.array_equal(gm[..., 4:], T.meta[..., 4:]), f"{what}: chosen clipping factors differ"
    # steps and zero-points: the same expressions on both sides; log2 comes from two different math libraries
    assert np.allclose(gm, T.meta, rtol=1e-13, atol=0), f"{what}: TLQ parameters differ"
    gw = tl.wsum.cpu().numpy()[rows].astype(np.float64)
    scale = np.abs(T.levels).max(axis=(1, 2)) * np.sqrt(W.shape[1])
    assert (np.abs(gw - T.wsum) <= 1e-6 * scale + 1e-30).all(), f"{what}: wsum differs"
    return T


def dual_to_device(P, factors):
    """(Bd, R1 bits, perm, R2 bits) of LayerSpec.dual_factors -> the binding's DualRotation on the device."""
    Bd, R1, perm, R2 = factors
    return P.DualRotation(Bd, bf16_to_device(R1), torch.from_numpy(np.ascontiguousarray(perm, dtype=np.int32)).cuda(),
                          bf16_to_device(R2))


def dual_to_f64(factors):
    """The same factors as the oracle takes them."""
    Bd, R1, perm, R2 = factors
    return Bd, bf16_bits_to_f64(R1), perm, bf16_bits_to_f64(R2)


def gpu_layer(spec: LayerSpec, W: np.ndarray, P, code_layout: int = 0):
    """Quantize weights on the GPU and build the layer handle.  Returns (QLayer, TLQWeights)."""
    g = default_clip_grid()
    Wd = torch.from_numpy(W).cuda()
    tl = P.lrq_tlq_quantize_weights(Wd, spec.w_bits, spec.group, 7, g, g, code_layout=code_layout)
    R = dual = None
    if spec.rot == "dense":
        R = bf16_to_device(spec.rotation_bf16())
    if spec.rot == "dual":
        dual = dual_to_device(P, spec.dual_factors())
    kind = {"dense": P.ROT_DENSE, "dual": P.ROT_DUAL, "hadamard": P.ROT_HADAMARD}[spec.rot]
    return P.QLayer(tl, spec.N, spec.K, kind, spec.a_bits, spec.had_block, R, dual=dual), tl


def oracle_layer_rows(orc, spec: LayerSpec, Xbits_rows: np.ndarray, T, R_bits=None):
    """The oracle's whole layer on the given token rows: (Y, codes, s, z, rotated values)."""
    X = bf16_bits_to_f64(Xbits_rows)
    R = None if R_bits is None else bf16_bits_to_f64(R_bits)
    dual = dual_to_f64(spec.dual_factors()) if spec.rot == "dual" else None
    return orc.qlinear(X, T, spec.a_bits, spec.rot, spec.had_block, R, return_rotated=True, dual=dual)
