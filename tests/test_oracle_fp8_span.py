"""Why the contraction feeds the tensor cores bf16 and not fp8 (e4m3): measured with the oracle alone.

An e4m3 operand would need every level of an output channel (Eqs. 8-9 with I = 3: a 4-bit significand), after one
power-of-two offset per channel, inside e4m3's 15 binades of normal numbers (2^-6 .. 2^8).  The twin-log quantizer
spaces its levels uniformly in log2|w| between the smallest and the largest magnitude of the row, so a row's levels
span as many octaves as its weights do; this test counts the rows that fit."""
import numpy as np
import pytest

from lrq_workloads import bf16_bits_to_f64, config_layers, default_clip_grid

E4M3_BINADES = 15


def _row_spans(orc, spec, rows=96):
    W = spec.weights()[:rows].astype(np.float64)
    if spec.rot == "dense":
        Wr = orc.rotate_weights(W, None, "dense", R=bf16_bits_to_f64(spec.rotation_bf16()))
    else:
        Wr = orc.rotate_weights(W, None, "hadamard", spec.had_block)
    g = default_clip_grid()
    T = orc.tlq_quantize(Wr, 4, spec.group, 3, g, g)                  # 4-bit codes, I = 3
    lv = np.abs(T.levels.reshape(rows, -1))
    assert (lv > 0).all()
    m, e = np.frexp(lv)
    assert np.array_equal(m * 16, np.rint(m * 16))                     # with I = 3 every level has a 4-bit significand
    return (e.max(axis=1) - e.min(axis=1) + 1).astype(int)


@pytest.mark.parametrize("cfg,layer", [(3, 0), (3, 1), (1, 0), (1, 3)])
def test_tlq_level_sets_do_not_fit_e4m3(orc, cfg, layer):
    spec = config_layers(cfg)[layer]
    span = _row_spans(orc, spec)
    fit = float((span <= E4M3_BINADES).mean())
    print(f"\ncfg{cfg} {spec.name}: octaves spanned by a row's levels: min {span.min()}, median {int(np.median(span))}, "
          f"max {span.max()}; rows that fit e4m3: {fit:.2f}")
    # one row that does not fit makes the layer inexact, and every layer has such rows (heavy-tailed weights: a
    # few rows carry an element far below or above the rest)
    assert fit < 1.0 and span.max() > E4M3_BINADES
