// Weight side of the rotation identity (Sec. 3.2, Eq. 2: (X R)(W R)^T = X W^T) with the smoothing of
// Sec. 5.1 folded in: W_rot = W diag(colmul) R, evaluated in fp64 and rounded once to fp32, which is what
// the TLQ quantizer reads.
//
// Offline step.  Hadamard: one CTA per weight row, the row in shared memory as fp64, log2(B) butterfly
// stages with a CTA barrier between them.  Dense: an fp64 matrix product on the CUDA cores, 64 x 64
// output tiles, 4 x 4 accumulators per thread; R is the layer's stored bf16 matrix (exact in fp64), so
// both sides of Eq. 2 use the same R.  Dual transformation (R = R1hat P R2hat, Sec. 4.2): one CTA per row, the
// row in shared memory as fp64, block-diagonal product, gather through the index map, second product.
#include "lrq_internal.cuh"

#include <cuda_bf16.h>

namespace {

__global__ void __launch_bounds__(256)
wrot_hadamard_kernel(const float* __restrict__ W, int N, int K, long ldw, const float* __restrict__ colmul, int log2B,
                     float* __restrict__ out, long ldo) {
    extern __shared__ double row[];                // [K]
    const int n = blockIdx.x, tid = threadIdx.x, nthr = blockDim.x;
    const float* w = W + (size_t)n * ldw;
    for (int k = tid; k < K; k += nthr) row[k] = (double)w[k] * (colmul ? (double)colmul[k] : 1.0);
    __syncthreads();
    const int pairs = K >> 1;
    for (int s = 0; s < log2B; ++s) {
        const int h = 1 << s;
        for (int i = tid; i < pairs; i += nthr) {
            const int lo = ((i >> s) << (s + 1)) | (i & (h - 1));
            const double a = row[lo], b = row[lo + h];
            row[lo] = a + b;
            row[lo + h] = a - b;
        }
        __syncthreads();
    }
    // 1/sqrt(B): a power of two for even log2(B), else a power of two times 1/sqrt(2)
    const double norm = ldexp((log2B & 1) ? 0.70710678118654752440 : 1.0, -(log2B >> 1));
    float* o = out + (size_t)n * ldo;
    for (int k = tid; k < K; k += nthr) o[k] = (float)(row[k] * norm);
}

constexpr int TM = 64, TN = 64, TK = 16;

__global__ void __launch_bounds__(256)
wrot_dense_kernel(const float* __restrict__ W, int N, int K, long ldw, const float* __restrict__ colmul,
                  const __nv_bfloat16* __restrict__ R, float* __restrict__ out, long ldo) {
    __shared__ double sW[TK][TM + 1];              // [k][row]
    __shared__ double sR[TK][TN];                  // [k][col]
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int n0 = blockIdx.y * TM, j0 = blockIdx.x * TN;
    double acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
    for (int k0 = 0; k0 < K; k0 += TK) {
        for (int i = tid; i < TM * TK; i += 256) {
            const int r = i / TK, k = i % TK;
            const int n = n0 + r, kk = k0 + k;
            double v = 0.0;
            if (n < N && kk < K) v = (double)W[(size_t)n * ldw + kk] * (colmul ? (double)colmul[kk] : 1.0);
            sW[k][r] = v;
        }
        for (int i = tid; i < TK * TN; i += 256) {
            const int k = i / TN, c = i % TN;
            const int kk = k0 + k, j = j0 + c;
            sR[k][c] = (kk < K && j < K) ? (double)__bfloat162float(R[(size_t)kk * K + j]) : 0.0;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < TK; ++k) {
            double a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = sW[k][ty * 4 + i]; b[i] = sR[k][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int n = n0 + ty * 4 + i;
        if (n >= N) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = j0 + tx * 4 + j;
            if (c < K) out[(size_t)n * ldo + c] = (float)acc[i][j];
        }
    }
}

// out[n] = ((w[n] * colmul) . blockdiag(R1)) gathered through perm, then . blockdiag(R2); blocks of Bd x Bd, row-major
__global__ void __launch_bounds__(256)
wrot_dual_kernel(const float* __restrict__ W, int N, int K, long ldw, const float* __restrict__ colmul, int Bd,
                 const __nv_bfloat16* __restrict__ R1, const int32_t* __restrict__ perm, const __nv_bfloat16* __restrict__ R2,
                 float* __restrict__ out, long ldo) {
    extern __shared__ double rows2[];              // a[K], b[K]
    double* a = rows2;
    double* b = rows2 + K;
    const int n = blockIdx.x, tid = threadIdx.x;
    const float* w = W + (size_t)n * ldw;
    for (int k = tid; k < K; k += 256) a[k] = (double)w[k] * (colmul ? (double)colmul[k] : 1.0);
    __syncthreads();
    for (int c = tid; c < K; c += 256) {           // b = a . blockdiag(R1)
        const int j = c / Bd, i = c - j * Bd;
        const __nv_bfloat16* r = R1 + (size_t)j * Bd * Bd + i;
        const double* x = a + j * Bd;
        double acc = 0.0;
        for (int l = 0; l < Bd; ++l) acc = fma(x[l], (double)__bfloat162float(r[(size_t)l * Bd]), acc);
        b[c] = acc;
    }
    __syncthreads();
    for (int c = tid; c < K; c += 256) {           // a = b . P
        const int p = perm[c];
        a[c] = (uint32_t)p < (uint32_t)K ? b[p] : b[0];
    }
    __syncthreads();
    float* o = out + (size_t)n * ldo;
    for (int c = tid; c < K; c += 256) {           // out = a . blockdiag(R2)
        const int j = c / Bd, i = c - j * Bd;
        const __nv_bfloat16* r = R2 + (size_t)j * Bd * Bd + i;
        const double* x = a + j * Bd;
        double acc = 0.0;
        for (int l = 0; l < Bd; ++l) acc = fma(x[l], (double)__bfloat162float(r[(size_t)l * Bd]), acc);
        o[c] = (float)acc;
    }
}

__global__ void wrot_scale_kernel(const float* __restrict__ W, int N, int K, long ldw, const float* __restrict__ colmul,
                                  float* __restrict__ out, long ldo) {
    const size_t total = (size_t)N * K;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t n = i / K, k = i % K;
        out[n * ldo + k] = (float)((double)W[n * ldw + k] * (colmul ? (double)colmul[k] : 1.0));
    }
}

}  // namespace

lrq_status lrq_launch_rotate_weights(const float* W, int N, int K, long ldw, const float* colmul, int kind,
                                     int had_block, const void* R, float* out, long ldo, cudaStream_t st) {
    if (kind == LRQ_ROT_HADAMARD) {
        int log2B = 0;
        while ((1 << log2B) < had_block) ++log2B;
        const size_t smem = (size_t)K * sizeof(double);
        if (smem > 200 * 1024) return LRQ_ERR_UNSUPPORTED;
        if (smem > 40 * 1024)
            LRQ_CUDA_TRY(cudaFuncSetAttribute(wrot_hadamard_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        wrot_hadamard_kernel<<<N, 256, smem, st>>>(W, N, K, ldw, colmul, log2B, out, ldo);
    } else if (kind == LRQ_ROT_DENSE) {
        const dim3 grid((K + TN - 1) / TN, (N + TM - 1) / TM);
        wrot_dense_kernel<<<grid, 256, 0, st>>>(W, N, K, ldw, colmul, static_cast<const __nv_bfloat16*>(R), out, ldo);
    } else {
        const size_t total = (size_t)N * K;
        const int blocks = (int)((total + 255) / 256 < 4096 ? (total + 255) / 256 : 4096);
        wrot_scale_kernel<<<blocks, 256, 0, st>>>(W, N, K, ldw, colmul, out, ldo);
    }
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}

lrq_status lrq_launch_rotate_weights_dual(const float* W, int N, int K, long ldw, const float* colmul, int Bd, const void* R1,
                                          const int32_t* perm, const void* R2, float* out, long ldo, cudaStream_t st) {
    const size_t smem = (size_t)K * 2 * sizeof(double);
    if (smem > 200 * 1024) return LRQ_ERR_UNSUPPORTED;
    if (smem > 40 * 1024)
        LRQ_CUDA_TRY(cudaFuncSetAttribute(wrot_dual_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    wrot_dual_kernel<<<N, 256, smem, st>>>(W, N, K, ldw, colmul, Bd, static_cast<const __nv_bfloat16*>(R1), perm,
                                           static_cast<const __nv_bfloat16*>(R2), out, ldo);
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}
