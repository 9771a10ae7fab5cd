"""B200 (sm_100a) quantized-linear path of LRQ-DiT: thin Python binding over the C-ABI library.

Every step of the path (rotation, per-token quantization, TLQ decode + tcgen05 contraction,
epilogue, TLQ weight quantization) runs in the CUDA library ``liblrq_b200.so``; this package only
marshals arguments.  There is no CPU fallback: importing works without a GPU, calling does not.
"""
from .binding import (  # noqa: F401
    StackPlan, lrq_rotate_quantize_act_static, lrq_static_scratch_bytes,
    load_library, LrqError, TLQWeights, QLayer,
    lrq_tlq_quantize_weights, lrq_rotate_quantize_act, lrq_qlinear, lrq_qlinear_stack, lrq_qgemm_codes,
    lrq_ars_select, lrq_rotate_weights, lrq_device_status, lrq_version, ROT_NONE, ROT_HADAMARD, ROT_DENSE, ROT_DUAL,
    DualRotation, lrq_rotate_weights_dual, ACT_ASYM, ACT_SYM, F32, F16, BF16, CODES_NIBBLE, CODES_PACKED3, lrq_selftest_wait_timeout, SELFTEST_WAIT_CODE,
)
