// The channel reordering between the two block-diagonal rotations of the dual transformation (Sec. 4.2:
// y = x . R1hat . P . R2hat, P a staggered permutation given as the index map (u P)_i = u[perm[i]]).
//
// u = x . R1hat arrives in fp32 from the first tensor-core product.  The second product takes bf16 operands, and a
// single rounding of u to bf16 would cost 16 of its 24 significant bits; instead every gathered element is split
// into three bf16 terms h1 + h2 + h3 (h1 = bf16(u), h2 = bf16(u - h1), h3 = bf16(u - h1 - h2); the two
// subtractions are exact in fp32), which together carry u to within 2^-25 of its magnitude.  The terms are written as three
// column panels [M, 3K] that the block-diagonal product sums into one fp32 accumulator, each product of a term
// with a bf16 entry of R2hat being exact.
//
// One CTA per token at a time: the fp32 row is staged in shared memory with coalesced 128-bit loads, gathered from
// there through perm (read once per CTA into shared memory as well), and the panels are written two elements per thread.
#include "lrq_internal.cuh"

#include <cuda_bf16.h>
#include <mutex>

namespace {

__device__ __forceinline__ uint32_t bf16_pair(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__global__ void __launch_bounds__(256)
dual_gather_split_kernel(const float* __restrict__ U, int M, int K, const int32_t* __restrict__ perm,
                         uint32_t* __restrict__ V3, int* status) {
    extern __shared__ __align__(16) unsigned char smem_dual[];
    float* row = reinterpret_cast<float*>(smem_dual);                 // [K]
    int32_t* sp = reinterpret_cast<int32_t*>(smem_dual) + K;          // [K]
    const int tid = threadIdx.x;
    bool bad = false;
    for (int i = tid; i < K; i += 256) {                              // perm does not depend on the previous kernel
        int32_t p = perm[i];
        if ((uint32_t)p >= (uint32_t)K) { p = 0; bad = true; }
        sp[i] = p;
    }
    if (bad) atomicCAS(status, 0, 31);
    lrq_pdl_trigger();
    lrq_pdl_wait();                                                   // U is the previous kernel's output
    const int K4 = K >> 2, K2 = K >> 1;
    for (int m = blockIdx.x; m < M; m += gridDim.x) {
        __syncthreads();                                              // previous token's gathers are done (and sp is filled)
        const float4* src = reinterpret_cast<const float4*>(U + (size_t)m * K);
        for (int i = tid; i < K4; i += 256) reinterpret_cast<float4*>(row)[i] = __ldcs(src + i);
        __syncthreads();
        uint32_t* dst = V3 + (size_t)m * (size_t)(3 * K2);            // three panels of K bf16 = K/2 words each
        for (int i = tid; i < K2; i += 256) {
            const float a = row[sp[2 * i]], b = row[sp[2 * i + 1]];
            const uint32_t h1 = bf16_pair(a, b);
            const float a1 = a - __uint_as_float(h1 << 16), b1 = b - __uint_as_float(h1 & 0xffff0000u);
            const uint32_t h2 = bf16_pair(a1, b1);
            const float a2 = a1 - __uint_as_float(h2 << 16), b2 = b1 - __uint_as_float(h2 & 0xffff0000u);
            const uint32_t h3 = bf16_pair(a2, b2);
            dst[i] = h1;
            dst[K2 + i] = h2;
            dst[2 * K2 + i] = h3;
        }
    }
}

}  // namespace

// V3 bf16 [M, 3K]: panel p holds the p-th bf16 term of U[m, perm[i]].  K a multiple of 4, at most 12288.
lrq_status lrq_launch_dual_gather_split(const float* U, int M, int K, const int32_t* perm, void* V3, cudaStream_t st) {
    if ((K % 4) || K > 12288 || !lrq_aligned(U, 16) || !lrq_aligned(V3, 4)) return LRQ_ERR_INVALID_ARG;
    const size_t smem = (size_t)K * 8;
    int dev = 0, sms = 0;
    if (lrq_current_device(&dev, &sms) != LRQ_OK) return LRQ_ERR_CUDA;
    if (smem > 48 * 1024) {
        static std::mutex mu;
        static bool configured[LRQ_MAX_DEVICES] = {};
        std::lock_guard<std::mutex> lock(mu);
        if (!configured[dev]) {
            LRQ_CUDA_TRY(cudaFuncSetAttribute(dual_gather_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 12288 * 8));
            configured[dev] = true;
        }
    }
    const int per_sm = smem <= 24 * 1024 ? 8 : smem <= 48 * 1024 ? 4 : 2;
    const int grid = M < sms * per_sm ? M : sms * per_sm;
    LRQ_CUDA_TRY(lrq_launch_pdl(dual_gather_split_kernel, dim3(grid), dim3(256), smem, st, U, M, K, perm,
                                static_cast<uint32_t*>(V3), lrq_status_word()));
    return LRQ_OK;
}
