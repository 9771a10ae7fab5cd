// Rotation + per-token activation quantization (Sec. 4.2 Eq. 12, first case; Sec. 3.1 Eq. 1).
//
// HBM-bound step: each activation is read once (bf16) and written once as a 4- or 8-bit code.
// The block-diagonal Walsh-Hadamard transform runs in fp32: three butterfly stages in registers
// on the 8 elements of one 128-bit load, the remaining stages three at a time through shared
// memory.  The 1/sqrt(B) normalisation is never applied to the elements: it is folded into the
// per-token scale, since rint(y/s) is invariant under a common factor of y and s.
#include "lrq_internal.cuh"

namespace {

__device__ __forceinline__ void bfly8(float* v) {
#pragma unroll
    for (int h = 1; h < 8; h <<= 1)
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (!(i & h)) { float a = v[i], b = v[i | h]; v[i] = a + b; v[i | h] = a - b; }
}

__device__ __forceinline__ void unpack_bf16x8(const uint4& r, float* v) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// Per-token quantization parameters from the token's extremes of the un-normalised transform.
// s_u is the step in the un-normalised domain; the reported scale is s_u * nrm.
struct TokenQ { float inv; float negz; };

__device__ __forceinline__ TokenQ token_params(float mn, float mx, float amax, int a_bits, int mode, double nrm,
                                               float* scale_out, int32_t* zp_out) {
    const double qmax = (double)((1 << a_bits) - 1);
    double s, z;
    if (mode == LRQ_ACT_ASYM) {
        s = ((double)mx - (double)mn) / qmax;
        if (!(s > 0.0)) s = 1.0 / nrm;            // empty range: unit step in the normalised domain
        z = rint((double)mn / s);
    } else {
        s = (double)amax / (double)((1 << (a_bits - 1)) - 1);
        if (!(s > 0.0)) s = 1.0 / nrm;
        z = -(double)(1 << (a_bits - 1));
    }
    *scale_out = (float)(s * nrm);
    *zp_out = (int32_t)z;
    TokenQ t;
    t.inv = (float)(1.0 / s);
    t.negz = (float)(-z);
    return t;
}

__device__ __forceinline__ int quant1(float u, const TokenQ& t, int qmax) {
    int q = __float2int_rn(fmaf(u, t.inv, t.negz));
    return min(max(q, 0), qmax);
}

// ------------------------------------------------------------------------------------------------
// Generic kernel: one CTA per token, the token's K transformed values live in shared memory.
// Any B = 2^n (8..4096) dividing K, any K that is a multiple of 8.
// SRC_F32: the input is an fp32 matrix that is already rotated (dense path): no transform.
// ------------------------------------------------------------------------------------------------
template <bool SRC_F32>
__global__ void __launch_bounds__(256)
rotq_generic_kernel(const void* __restrict__ Xv, int M, int K, long ldx, int log2B, int a_bits, int mode,
                    uint8_t* __restrict__ codes, float* __restrict__ scale, int32_t* __restrict__ zp) {
    extern __shared__ float row[];
    __shared__ float red_mn[8], red_mx[8], red_am[8];
    __shared__ TokenQ tq;
    const int m = blockIdx.x;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int nchunk = K >> 3;

    if (SRC_F32) {
        const float4* src = reinterpret_cast<const float4*>(static_cast<const float*>(Xv) + (size_t)m * ldx);
        for (int c = tid; c < (K >> 2); c += nthr) reinterpret_cast<float4*>(row)[c] = src[c];
    } else {
        const uint4* src = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(Xv) + (size_t)m * ldx);
        for (int c = tid; c < nchunk; c += nthr) {
            float v[8];
            unpack_bf16x8(src[c], v);
            if (log2B >= 3) bfly8(v);
#pragma unroll
            for (int i = 0; i < 8; ++i) row[c * 8 + i] = v[i];
        }
    }
    __syncthreads();
    if (!SRC_F32) {
        // remaining stages, up to three index bits per pass
        for (int bit = 3; bit < log2B; bit += 3) {
            const int nb = min(3, log2B - bit);           // bits handled in this pass
            const int span = 1 << nb;
            const int ngroups = K >> nb;
            const int lowmask = (1 << bit) - 1;
            for (int g = tid; g < ngroups; g += nthr) {
                // g enumerates indices with the nb bits [bit, bit+nb) removed
                const int base = ((g & ~lowmask) << nb) | (g & lowmask);
                float v[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = (i < span) ? row[base + (i << bit)] : 0.f;
                if (nb == 3) bfly8(v);
                else if (nb == 2) {
                    float a = v[0] + v[1], b = v[0] - v[1], c = v[2] + v[3], d = v[2] - v[3];
                    v[0] = a + c; v[1] = b + d; v[2] = a - c; v[3] = b - d;
                } else { float a = v[0], b = v[1]; v[0] = a + b; v[1] = a - b; }
#pragma unroll
                for (int i = 0; i < 8; ++i) if (i < span) row[base + (i << bit)] = v[i];
            }
            __syncthreads();
        }
    }
    // token extremes
    float mn = INFINITY, mx = -INFINITY, am = 0.f;
    for (int k = tid; k < K; k += nthr) { float u = row[k]; mn = fminf(mn, u); mx = fmaxf(mx, u); am = fmaxf(am, fabsf(u)); }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
    }
    if ((tid & 31) == 0) { red_mn[tid >> 5] = mn; red_mx[tid >> 5] = mx; red_am[tid >> 5] = am; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < (nthr >> 5); ++w) { mn = fminf(mn, red_mn[w]); mx = fmaxf(mx, red_mx[w]); am = fmaxf(am, red_am[w]); }
        const double nrm = SRC_F32 ? 1.0 : 1.0 / sqrt((double)(1 << log2B));
        tq = token_params(mn, mx, am, a_bits, mode, nrm, scale + m, zp + m);
    }
    __syncthreads();
    const TokenQ t = tq;
    const int qmax = (1 << a_bits) - 1;
    if (a_bits == 8) {
        uint2* dst = reinterpret_cast<uint2*>(codes + (size_t)m * K);
        for (int c = tid; c < nchunk; c += nthr) {
            uint32_t w[2] = {0, 0};
#pragma unroll
            for (int i = 0; i < 8; ++i) w[i >> 2] |= (uint32_t)quant1(row[c * 8 + i], t, qmax) << (8 * (i & 3));
            dst[c] = make_uint2(w[0], w[1]);
        }
    } else {
        uint32_t* dst = reinterpret_cast<uint32_t*>(codes + (size_t)m * (K >> 1));
        for (int c = tid; c < nchunk; c += nthr) {
            uint32_t w = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) w |= (uint32_t)quant1(row[c * 8 + i], t, qmax) << (4 * i);
            dst[c] = w;
        }
    }
}

}  // namespace

static lrq_status launch_generic(bool f32, const void* X, int M, int K, long ldx, int log2B, int a_bits, int mode,
                                 uint8_t* codes, float* scale, int32_t* zp, cudaStream_t st) {
    const size_t smem = (size_t)K * sizeof(float);
    if (smem > 200 * 1024) return LRQ_ERR_UNSUPPORTED;
    auto kern = f32 ? rotq_generic_kernel<true> : rotq_generic_kernel<false>;
    if (smem > 40 * 1024)
        LRQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int threads = (K >= 2048) ? 256 : (K >= 1024 ? 128 : 64);
    kern<<<M, threads, smem, st>>>(X, M, K, ldx, log2B, a_bits, mode, codes, scale, zp);
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}

lrq_status lrq_launch_rotq_hadamard(const void* X, int M, int K, long ldx, int B, int a_bits, int mode,
                                    uint8_t* codes, float* scale, int32_t* zp, cudaStream_t st) {
    int log2B = 0;
    while ((1 << log2B) < B) ++log2B;
    return launch_generic(false, X, M, K, ldx, log2B, a_bits, mode, codes, scale, zp, st);
}

lrq_status lrq_launch_quantize_f32(const float* Y, int M, int K, long ldy, int a_bits, int mode,
                                   uint8_t* codes, float* scale, int32_t* zp, cudaStream_t st) {
    return launch_generic(true, Y, M, K, ldy, 0, a_bits, mode, codes, scale, zp, st);
}
