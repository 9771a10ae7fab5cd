// Outlier-aware rotation y = x . R (Sec. 4.2, Eq. 12, second case) as a dense contraction:
// X bf16 [M,K] times R bf16 [K,K] into an fp32 scratch that the per-token quantizer then reads.
// bf16 x bf16 products are exact in fp32; the sum is accumulated in fp32.
#include "lrq_internal.cuh"

namespace {

constexpr int TM = 64, TN = 64, TK = 32;

__global__ void __launch_bounds__(256)
rotgemm_simple_kernel(const __nv_bfloat16* __restrict__ X, int M, int K, long ldx,
                      const __nv_bfloat16* __restrict__ R, float* __restrict__ Y) {
    __shared__ float Xs[TK][TM + 1];
    __shared__ float Rs[TK][TN + 1];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += TK) {
        for (int e = tid; e < TM * TK; e += 256) {
            const int r = e / TK, kk = e % TK, m = m0 + r, k = k0 + kk;
            Xs[kk][r] = (m < M && k < K) ? __bfloat162float(X[(size_t)m * ldx + k]) : 0.f;
        }
        for (int e = tid; e < TN * TK; e += 256) {
            const int kk = e / TN, c = e % TN, k = k0 + kk, n = n0 + c;
            Rs[kk][c] = (k < K && n < K) ? __bfloat162float(R[(size_t)k * K + n]) : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int kk = 0; kk < TK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = Xs[kk][ty * 4 + i]; b[i] = Rs[kk][tx * 4 + i]; }
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
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n < K) Y[(size_t)m * K + n] = acc[i][j];
        }
    }
}

}  // namespace

lrq_status lrq_launch_rotgemm(const void* X, int M, int K, long ldx, const void* R, float* Y, cudaStream_t st) {
    dim3 grid((K + TN - 1) / TN, (M + TM - 1) / TM), block(256);
    rotgemm_simple_kernel<<<grid, block, 0, st>>>(static_cast<const __nv_bfloat16*>(X), M, K, ldx,
                                                  static_cast<const __nv_bfloat16*>(R), Y);
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}
