// Pieces shared by the rotate + quantize kernels: the per-token parameters of Eq. 1 and the saturating packers.
#pragma once
#include "lrq_internal.cuh"

namespace lrq_rq {

// Per-token quantization parameters from the token's extremes of the un-normalised transform.
// s_u is the step in the un-normalised domain; the reported scale is s_u * nrm.
struct TokenQ { float inv; float negz; };

__device__ __forceinline__ uint32_t pack_u8x4(int q0, int q1, int q2, int q3) {
    uint32_t t, d;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(q3), "r"(q2), "r"(0));
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(q1), "r"(q0), "r"(t));
    return d;
}

__device__ __forceinline__ uint32_t pack_u4x8(const int* q) {
    uint32_t t = 0;
#pragma unroll
    for (int i = 3; i >= 0; --i)
        asm("cvt.pack.sat.u4.s32.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(q[2 * i + 1]), "r"(q[2 * i]), "r"(t));
    return t;
}

// The same parameters for the fast kernel, where every warp works them out: one fp64 reciprocal refined
// from the fp32 approximation (two Newton steps, relative error below 1e-14) instead of fp64 divisions.
__device__ __forceinline__ TokenQ token_params_fast(float mn, float mx, int a_bits, int mode, double nrm,
                                                    float* scale_out, int32_t* zp_out) {
    const bool asym = mode == LRQ_ACT_ASYM;
    const double qsteps = asym ? (double)((1 << a_bits) - 1) : (double)((1 << (a_bits - 1)) - 1);
    const double range = asym ? (double)mx - (double)mn : (double)fmaxf(fabsf(mn), fabsf(mx));
    const float r0 = __frcp_rn((float)range);
    double s, inv;
    if (range > 0.0 && r0 > 0.f && r0 < 3.0e38f) {
        double r = (double)r0;
        r = fma(r, fma(-range, r, 1.0), r);
        r = fma(r, fma(-range, r, 1.0), r);
        inv = qsteps * r;
        s = range * (1.0 / qsteps);
    } else if (range > 0.0) {      // outside fp32's reciprocal range: plain division
        s = range / qsteps;
        inv = 1.0 / s;
    } else {                       // empty range: unit step in the normalised domain
        s = 1.0 / nrm;
        inv = nrm;
    }
    const double z = asym ? rint((double)mn * inv) : -(double)(1 << (a_bits - 1));
    *scale_out = (float)(s * nrm);
    *zp_out = (int32_t)z;
    TokenQ t;
    t.inv = (float)inv;
    t.negz = (float)(-z);
    return t;
}

}  // namespace lrq_rq
