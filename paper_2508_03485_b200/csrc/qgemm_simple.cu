// Quantized contraction and epilogue on the CUDA cores (Sec. 4.1, Eq. 10 evaluated exactly).
//
// In-library ablation baseline and the path for shapes the tensor-core kernel does not take.
// A 64x64 output tile per CTA; activation codes and TLQ codes are decoded to fp32 in shared
// memory (codes through the group's level table), every product q*level is exact in fp32 and
// the sum is accumulated in fp32.
//
// A second kernel evaluates the contraction in the integer form the paper gives for hardware (Sec. 4.1, Eq. 10):
// every level is an integer mantissa times a power of two (Eqs. 8-9), so a term is the product of two small
// integers, the activation code and the mantissa, shifted left by the level's exponent:
//   acc[m,n] = 2^(emin_n - 8) * sum_k ((q[m,k] * mant[n,k]) << (e[n,k] - emin_n)),
// with |level| = mant * 2^(e - 8), mant in 128..255, and emin_n the smallest exponent of row n's tables (the
// common factor that keeps every shift non-negative).  The sum is exact (128-bit integer accumulators, which hold
// level sets that span up to 96 octaves; a wider one is recorded as status 32); only the final conversion and the
// epilogue round.  It exists to show the two forms agree, not for speed.
#include "lrq_internal.cuh"
#include <climits>

namespace {

constexpr int TM = 64, TN = 64, TK = 32;

template <typename OutT> __device__ __forceinline__ OutT cast_out(float v);
template <> __device__ __forceinline__ float cast_out<float>(float v) { return v; }
template <> __device__ __forceinline__ __half cast_out<__half>(float v) { return __float2half_rn(v); }
template <> __device__ __forceinline__ __nv_bfloat16 cast_out<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename OutT>
__global__ void __launch_bounds__(256)
qgemm_simple_kernel(const uint8_t* __restrict__ a_codes, const float* __restrict__ a_scale,
                    const int32_t* __restrict__ a_zp, int M, int N, int K, int a_bits, int w_bits, int G, int packed3,
                    const uint8_t* __restrict__ w_codes, const float* __restrict__ levels,
                    const float* __restrict__ wsum, const float* __restrict__ wscale,
                    const float* __restrict__ bias, OutT* __restrict__ Y, long ldy) {
    __shared__ float As[TK][TM + 1];
    __shared__ float Ws[TK][TN + 1];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
    const int tx = tid & 15, ty = tid >> 4;              // 16 x 16 threads, 4 x 4 outputs each
    const int nlev = 1 << w_bits, ngrp = K / G;
    float acc[4][4] = {};

    for (int k0 = 0; k0 < K; k0 += TK) {
        for (int e = tid; e < TM * TK; e += 256) {
            const int r = e / TK, kk = e % TK, m = m0 + r, k = k0 + kk;
            float v = 0.f;
            if (m < M && k < K) {
                if (a_bits == 8) v = (float)a_codes[(size_t)m * K + k];
                else v = (float)((a_codes[((size_t)m * K + k) >> 1] >> (4 * (k & 1))) & 0xF);
            }
            As[kk][r] = v;
        }
        for (int e = tid; e < TN * TK; e += 256) {
            const int r = e / TK, kk = e % TK, n = n0 + r, k = k0 + kk;
            float v = 0.f;
            if (n < N && k < K) {
                int u;
                if (packed3) {                               // eight codes in three bytes: code j at bits 3j..3j+2
                    const uint8_t* g = w_codes + (size_t)n * (K / 8 * 3) + (size_t)(k >> 3) * 3;
                    const uint32_t w24 = (uint32_t)g[0] | ((uint32_t)g[1] << 8) | ((uint32_t)g[2] << 16);
                    u = (w24 >> (3 * (k & 7))) & 7;
                } else {
                    u = (w_codes[((size_t)n * K + k) >> 1] >> (4 * (k & 1))) & 0xF;
                }
                v = levels[((size_t)n * ngrp + k / G) * nlev + u];
            }
            Ws[kk][r] = v;
        }
        __syncthreads();
#pragma unroll 8
        for (int kk = 0; kk < TK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b[i] = Ws[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= M) continue;
        const float s = a_scale[m], z = (float)a_zp[m];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= N) continue;
            float y = s * fmaf(z, wsum[n], acc[i][j]);
            if (wscale) y *= wscale[n];
            if (bias) y += bias[n];
            Y[(size_t)m * ldy + n] = cast_out<OutT>(y);
        }
    }
}

// ---- Eq. 10 literally: integer mantissa products, shifts, integer accumulation ----------------------------------------
constexpr int SM_ROWS = 16;                                   // a CTA computes 16 x 16 outputs, one per thread

template <typename OutT>
__global__ void __launch_bounds__(256)
qgemm_shift_kernel(const uint8_t* __restrict__ a_codes, const float* __restrict__ a_scale,
                   const int32_t* __restrict__ a_zp, int M, int N, int K, int a_bits, int w_bits, int G, int packed3,
                   const uint8_t* __restrict__ w_codes, const float* __restrict__ levels,
                   const float* __restrict__ wsum, const float* __restrict__ wscale,
                   const float* __restrict__ bias, OutT* __restrict__ Y, long ldy, int* status) {
    __shared__ int emin[SM_ROWS];                             // smallest level exponent of each of the tile's weight rows
    __shared__ int Aq[TK][SM_ROWS + 1];                       // activation codes
    __shared__ short Wm[TK][SM_ROWS + 1];                     // signed mantissas
    __shared__ unsigned char Wsh[TK][SM_ROWS + 1];            // shifts
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * SM_ROWS, n0 = blockIdx.x * SM_ROWS;
    const int nlev = 1 << w_bits, ngrp = K / G;
    if (tid < SM_ROWS) {
        const int n = n0 + tid;
        int lo = INT_MAX;
        if (n < N)
            for (int i = 0; i < ngrp * nlev; ++i) {
                int e;
                const float f = frexpf(fabsf(levels[(size_t)n * ngrp * nlev + i]), &e);   // |level| = f * 2^e, f in [0.5, 1)
                if (f > 0.f && e < lo) lo = e;
            }
        emin[tid] = lo == INT_MAX ? 0 : lo;
    }
    __syncthreads();
    __int128 acc = 0;
    for (int k0 = 0; k0 < K; k0 += TK) {
        for (int e = tid; e < SM_ROWS * TK; e += 256) {
            const int r = e / TK, kk = e % TK, m = m0 + r, k = k0 + kk;
            int q = 0;
            if (m < M && k < K)
                q = a_bits == 8 ? a_codes[(size_t)m * K + k] : (a_codes[((size_t)m * K + k) >> 1] >> (4 * (k & 1))) & 0xF;
            Aq[kk][r] = q;
        }
        for (int e = tid; e < SM_ROWS * TK; e += 256) {
            const int r = e / TK, kk = e % TK, n = n0 + r, k = k0 + kk;
            int mant = 0, sh = 0;
            if (n < N && k < K) {
                int u;
                if (packed3) {
                    const uint8_t* g = w_codes + (size_t)n * (K / 8 * 3) + (size_t)(k >> 3) * 3;
                    const uint32_t w24 = (uint32_t)g[0] | ((uint32_t)g[1] << 8) | ((uint32_t)g[2] << 16);
                    u = (w24 >> (3 * (k & 7))) & 7;
                } else {
                    u = (w_codes[((size_t)n * K + k) >> 1] >> (4 * (k & 1))) & 0xF;
                }
                const float lv = levels[((size_t)n * ngrp + k / G) * nlev + u];
                int ex;
                const float f = frexpf(fabsf(lv), &ex);
                mant = (int)(f * 256.f);                      // exact: a level has an 8-bit significand (I = 7)
                if (lv < 0.f) mant = -mant;
                sh = f > 0.f ? ex - emin[r] : 0;
                if (sh > 96) { atomicCAS(status, 0, 32); sh = 96; }   // 16 + 96 + 14 bits is what the accumulator holds
            }
            Wm[kk][r] = (short)mant;
            Wsh[kk][r] = (unsigned char)sh;
        }
        __syncthreads();
        for (int kk = 0; kk < TK; ++kk)
            acc += (__int128)(Aq[kk][ty] * (int)Wm[kk][tx]) << Wsh[kk][tx];     // (mantissa product) << (f - I), Eq. 10
        __syncthreads();
    }
    const int m = m0 + ty, n = n0 + tx;
    if (m < M && n < N) {
        // to floating point through sign and magnitude (the two halves of a negative two's-complement value would cancel)
        const bool neg = acc < 0;
        const unsigned __int128 mag = neg ? (unsigned __int128)(-acc) : (unsigned __int128)acc;
        const double dm = (double)(unsigned long long)(mag >> 64) * 18446744073709551616.0 + (double)(unsigned long long)mag;
        const double a = ldexp(neg ? -dm : dm, emin[tx] - 8);
        float y = a_scale[m] * fmaf((float)a_zp[m], wsum[n], (float)a);
        if (wscale) y *= wscale[n];
        if (bias) y += bias[n];
        Y[(size_t)m * ldy + n] = cast_out<OutT>(y);
    }
}

}  // namespace

lrq_status lrq_launch_qgemm_shift(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale,
                                  const int32_t* a_zp, int M, void* Y, lrq_dtype dt, long ldy, cudaStream_t st) {
    dim3 grid((L->N + SM_ROWS - 1) / SM_ROWS, (M + SM_ROWS - 1) / SM_ROWS), block(256);
    if (grid.y > 65535) return LRQ_ERR_UNSUPPORTED;
#define LRQ_GO(T)                                                                                              \
    qgemm_shift_kernel<T><<<grid, block, 0, st>>>(a_codes, a_scale, a_zp, M, L->N, L->K, L->act.a_bits,        \
                                                  L->w_bits, L->group, L->packed3, L->codes, L->levels, L->wsum, \
                                                  L->wscale, L->bias, static_cast<T*>(Y), ldy, lrq_status_word())
    if (dt == LRQ_F32) LRQ_GO(float);
    else if (dt == LRQ_F16) LRQ_GO(__half);
    else LRQ_GO(__nv_bfloat16);
#undef LRQ_GO
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}

lrq_status lrq_launch_qgemm_simple(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale,
                                   const int32_t* a_zp, int M, void* Y, lrq_dtype dt, long ldy, cudaStream_t st) {
    dim3 grid((L->N + TN - 1) / TN, (M + TM - 1) / TM), block(256);
#define LRQ_GO(T)                                                                                              \
    qgemm_simple_kernel<T><<<grid, block, 0, st>>>(a_codes, a_scale, a_zp, M, L->N, L->K, L->act.a_bits,       \
                                                   L->w_bits, L->group, L->packed3, L->codes, L->levels, L->wsum, \
                                                   L->wscale, L->bias, static_cast<T*>(Y), ldy)
    if (dt == LRQ_F32) LRQ_GO(float);
    else if (dt == LRQ_F16) LRQ_GO(__half);
    else LRQ_GO(__nv_bfloat16);
#undef LRQ_GO
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}
