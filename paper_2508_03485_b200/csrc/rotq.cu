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


// ------------------------------------------------------------------------------------------------
// Fast kernel.  A thread owns 32 consecutive elements of one token (four 128-bit loads in flight):
// index bits 0-4 of the transform are butterflies between its own registers, bits 5-9 are
// butterflies with the lane whose index differs in one bit (one shuffle and one fused
// multiply-add per element and stage), bits 10-11 (B = 2048, 4096) go through shared memory.
// A CTA holds T whole tokens (T * K/32 threads, a multiple of 32); the token's extremes are reduced
// through shared memory, then every thread quantizes and packs its own 32 values from registers:
// 32 bytes (8-bit codes) or 16 bytes (4-bit codes) per thread, contiguous across the warp.
// ------------------------------------------------------------------------------------------------
constexpr int EPT = 32;

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

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

template <int LOG2B, int A_BITS>
__global__ void __launch_bounds__(512)
rotq_fast_kernel(const __nv_bfloat16* __restrict__ X, int M, int K, long ldx, int mode, int tok_per_cta,
                 uint8_t* __restrict__ codes, float* __restrict__ scale, int32_t* __restrict__ zp) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tpt = K / EPT;                         // threads per token
    const int tid = threadIdx.x, lane = tid & 31;
    const int tl = tid / tpt, j = tid - tl * tpt;    // token within the CTA, thread within the token
    const int m = blockIdx.x * tok_per_cta + tl;
    const bool live = m < M;

    float v[EPT];
    if (live) {
        const uint4* src = reinterpret_cast<const uint4*>(X + (size_t)m * ldx + (size_t)j * EPT);
        uint4 r[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) r[i] = ldg_stream(src + i);
#pragma unroll
        for (int i = 0; i < 4; ++i) unpack_bf16x8(r[i], v + 8 * i);
    } else {
#pragma unroll
        for (int i = 0; i < EPT; ++i) v[i] = 0.f;
    }
    // index bits 0..4: registers
#pragma unroll
    for (int h = 1; h < EPT && h < (1 << LOG2B); h <<= 1)
#pragma unroll
        for (int i = 0; i < EPT; ++i)
            if (!(i & h)) { const float a = v[i], b = v[i | h]; v[i] = a + b; v[i | h] = a - b; }
    // index bits 5..9: partner lanes
#pragma unroll
    for (int b = 5; b < LOG2B && b < 10; ++b) {
        const int lm = 1 << (b - 5);
        const float sgn = (lane & lm) ? -1.f : 1.f;
#pragma unroll
        for (int i = 0; i < EPT; ++i) {
            const float o = __shfl_xor_sync(0xffffffffu, v[i], lm);
            v[i] = fmaf(v[i], sgn, o);               // low lane: own + other, high lane: other - own
        }
    }
    // index bits 10..11: partner warps, through shared memory (chunk index swizzled by the lane)
    float* red = reinterpret_cast<float*>(smem_raw);                 // [3][nthreads]
    TokenQ* tqs = reinterpret_cast<TokenQ*>(red + 3 * blockDim.x);   // [tok_per_cta]
    if (LOG2B > 10) {
        float4* xb = reinterpret_cast<float4*>(tqs + tok_per_cta + 1);
        xb = reinterpret_cast<float4*>((reinterpret_cast<uintptr_t>(xb) + 15) & ~uintptr_t(15));
#pragma unroll
        for (int b = 10; b < LOG2B; ++b) {
            const int tm = 1 << (b - 5);
            __syncthreads();
#pragma unroll
            for (int c = 0; c < 8; ++c)
                xb[tid * 8 + (c ^ (lane & 7))] = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
            __syncthreads();
            const int pt = tid ^ tm;
            const float sgn = (tid & tm) ? -1.f : 1.f;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 o = xb[pt * 8 + (c ^ (lane & 7))];
                v[4 * c] = fmaf(v[4 * c], sgn, o.x); v[4 * c + 1] = fmaf(v[4 * c + 1], sgn, o.y);
                v[4 * c + 2] = fmaf(v[4 * c + 2], sgn, o.z); v[4 * c + 3] = fmaf(v[4 * c + 3], sgn, o.w);
            }
        }
    }
    // extremes of the thread's values, then of the token
    float mn = v[0], mx = v[0];
#pragma unroll
    for (int i = 1; i < EPT; ++i) { mn = fminf(mn, v[i]); mx = fmaxf(mx, v[i]); }
    __syncthreads();
    red[tid] = mn; red[blockDim.x + tid] = mx;
    __syncthreads();
    const int warp = tid >> 5, nwarp = blockDim.x >> 5;
    for (int t = warp; t < tok_per_cta; t += nwarp) {
        float a = INFINITY, b = -INFINITY;
        for (int i = lane; i < tpt; i += 32) { a = fminf(a, red[t * tpt + i]); b = fmaxf(b, red[blockDim.x + t * tpt + i]); }
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            a = fminf(a, __shfl_xor_sync(0xffffffffu, a, o));
            b = fmaxf(b, __shfl_xor_sync(0xffffffffu, b, o));
        }
        const int mt = blockIdx.x * tok_per_cta + t;
        if (lane == 0 && mt < M)
            tqs[t] = token_params(a, b, fmaxf(fabsf(a), fabsf(b)), A_BITS, mode, 1.0 / sqrt((double)(1 << LOG2B)),
                                  scale + mt, zp + mt);
    }
    __syncthreads();
    if (!live) return;
    const TokenQ t = tqs[tl];
    int q[EPT];
#pragma unroll
    for (int i = 0; i < EPT; ++i) q[i] = __float2int_rn(fmaf(v[i], t.inv, t.negz));
    if (A_BITS == 8) {
        uint4* dst = reinterpret_cast<uint4*>(codes + (size_t)m * K + (size_t)j * EPT);
        uint32_t w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = pack_u8x4(q[4 * i], q[4 * i + 1], q[4 * i + 2], q[4 * i + 3]);
        dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
        dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
    } else {
        uint4* dst = reinterpret_cast<uint4*>(codes + (((size_t)m * K + (size_t)j * EPT) >> 1));
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] = pack_u4x8(q + 8 * i);
        dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
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

template <int LOG2B>
static lrq_status launch_fast(const void* X, int M, int K, long ldx, int a_bits, int mode, uint8_t* codes,
                              float* scale, int32_t* zp, cudaStream_t st) {
    const int tpt = K / EPT;
    // whole tokens per CTA: thread count a multiple of 32, at least 256 when the token is small
    int T = 1;
    while ((T * tpt) % 32) ++T;
    const int T0 = T;
    while (T * tpt < 256 && (T + T0) * tpt <= 512) T += T0;
    const int threads = T * tpt;
    if (threads > 512) return LRQ_ERR_UNSUPPORTED;
    size_t smem = 3 * sizeof(float) * threads + sizeof(TokenQ) * (T + 1) + 16;
    if (LOG2B > 10) smem += (size_t)threads * EPT * sizeof(float);
    auto kern = a_bits == 8 ? rotq_fast_kernel<LOG2B, 8> : rotq_fast_kernel<LOG2B, 4>;
    if (smem > 40 * 1024) LRQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<(M + T - 1) / T, threads, smem, st>>>(static_cast<const __nv_bfloat16*>(X), M, K, ldx, mode, T, codes, scale, zp);
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}

lrq_status lrq_launch_rotq_hadamard(const void* X, int M, int K, long ldx, int B, int a_bits, int mode,
                                    uint8_t* codes, float* scale, int32_t* zp, cudaStream_t st) {
    int log2B = 0;
    while ((1 << log2B) < B) ++log2B;
    // the fast kernel needs whole 32-element thread slices and, for B >= 2048, whole-CTA tokens
    const bool fast_ok = (K % EPT) == 0 && B >= 8 && (ldx % 8) == 0;
    if (fast_ok) {
        lrq_status r = LRQ_ERR_UNSUPPORTED;
        switch (log2B) {
#define LRQ_CASE(L) case L: r = launch_fast<L>(X, M, K, ldx, a_bits, mode, codes, scale, zp, st); break;
            LRQ_CASE(3) LRQ_CASE(4) LRQ_CASE(5) LRQ_CASE(6) LRQ_CASE(7) LRQ_CASE(8) LRQ_CASE(9) LRQ_CASE(10)
            LRQ_CASE(11) LRQ_CASE(12)
#undef LRQ_CASE
            default: break;
        }
        if (r != LRQ_ERR_UNSUPPORTED) return r;
    }
    return launch_generic(false, X, M, K, ldx, log2B, a_bits, mode, codes, scale, zp, st);
}

lrq_status lrq_launch_quantize_f32(const float* Y, int M, int K, long ldy, int a_bits, int mode,
                                   uint8_t* codes, float* scale, int32_t* zp, cudaStream_t st) {
    return launch_generic(true, Y, M, K, ldy, 0, a_bits, mode, codes, scale, zp, st);
}
