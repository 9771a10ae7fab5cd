// Twin-log weight quantization with search-based clipping (Sec. 4.1, Eqs. 4-9).
//
// Offline step.  One CTA per output row walks the row's groups; log2|w| of the group is kept in
// shared memory (fp64) and every candidate clipping factor of both sides is evaluated by all
// threads together: per element one division, one rounding and one squared difference against
// the candidate's small level table.  All decisions (codes, chosen factor) are taken in fp64.
#include "lrq_internal.cuh"

namespace {

constexpr int kMaxGrid = 64;
struct ClipGrid { double a[kMaxGrid]; double b[kMaxGrid]; int na, nb; };

__device__ __forceinline__ double level_value(double e, int I) {
    // Eqs. 8-9: 2^e ~ II * 2^(f-I) with f = floor(e), II = rint(2^(e-f) * 2^I)
    const double f = floor(e);
    const double II = rint(exp2(e - f) * (double)(1 << I));
    return ldexp(II, (int)f - I);
}

template <typename T, typename Op>
__device__ __forceinline__ T block_reduce(T v, Op op, T* scratch) {
    // deterministic tree: warp shuffles, then warp 0 folds the per-warp values in order
#pragma unroll
    for (int o = 16; o; o >>= 1) v = op(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    T r = scratch[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) r = op(r, scratch[w]);
    return r;
}

struct Side {
    double s, z;        // chosen step and zero-point
    double factor;      // chosen clipping factor
};

__global__ void __launch_bounds__(256)
tlq_quantize_kernel(const float* __restrict__ W, int N, int K, int G, int bits, int I, ClipGrid grid,
                    uint8_t* __restrict__ codes, float* __restrict__ levels, double* __restrict__ meta,
                    float* __restrict__ wsum) {
    extern __shared__ double lg[];                 // [G] log2|w|
    __shared__ double red[8];
    __shared__ double cand_lev[2][10];             // candidate level tables of the two sides
    __shared__ double cand_sz[2][2];
    __shared__ int cand_ok[2];
    __shared__ Side best[2];
    __shared__ double best_err[2];
    __shared__ int found[2];

    const int n = blockIdx.x, tid = threadIdx.x, nthr = blockDim.x;
    const int half = 1 << (bits - 1), nlev = 1 << bits, ngrp = K / G;
    const int nq[2] = {half - 1, half};
    double row_sum = 0.0;                          // accumulated by thread 0 only

    for (int g = 0; g < ngrp; ++g) {
        const float* w = W + (size_t)n * K + (size_t)g * G;
        double lmax[2] = {-INFINITY, -INFINITY}, lmin[2] = {INFINITY, INFINITY};
        int cnt[2] = {0, 0};
        for (int k = tid; k < G; k += nthr) {
            const float v = w[k];
            double l = 0.0;
            if (v != 0.f) {
                l = log2((double)fabsf(v));
                const int sd = v < 0.f;
                lmax[sd] = fmax(lmax[sd], l); lmin[sd] = fmin(lmin[sd], l); cnt[sd]++;
            }
            lg[k] = l;
        }
        for (int sd = 0; sd < 2; ++sd) {
            lmax[sd] = block_reduce(lmax[sd], [](double a, double b) { return fmax(a, b); }, red);
            lmin[sd] = block_reduce(lmin[sd], [](double a, double b) { return fmin(a, b); }, red);
            cnt[sd] = (int)block_reduce((double)cnt[sd], [](double a, double b) { return a + b; }, red);
        }
        if (tid < 2) { best_err[tid] = INFINITY; found[tid] = 0; }
        __syncthreads();

        const int ncand = max(grid.na, grid.nb);
        for (int c = 0; c < ncand; ++c) {
            // candidate parameters and level tables
            if (tid < 2) {
                const int sd = tid;
                const int ng = sd ? grid.nb : grid.na;
                int ok = 0;
                if (c < ng && cnt[sd] > 0 && nq[sd] > 0) {
                    const double top = (sd ? grid.b[c] : grid.a[c]) * lmax[sd], bot = lmin[sd];
                    if (top > bot) {
                        const double s = (top - bot) / (double)nq[sd];
                        cand_sz[sd][0] = s; cand_sz[sd][1] = rint(bot / s);
                        ok = 1;
                    }
                }
                cand_ok[sd] = ok;
            }
            __syncthreads();
            if (tid < 20) {
                const int sd = tid / 10, q = tid % 10;
                if (cand_ok[sd] && q <= nq[sd]) cand_lev[sd][q] = level_value(cand_sz[sd][0] * ((double)q + cand_sz[sd][1]), I);
            }
            __syncthreads();
            double err[2] = {0.0, 0.0};
            for (int k = tid; k < G; k += nthr) {
                const float v = w[k];
                if (v == 0.f) continue;
                const int sd = v < 0.f;
                if (!cand_ok[sd]) continue;
                const double s = cand_sz[sd][0], z = cand_sz[sd][1];
                const int q = (int)fmin(fmax(rint(lg[k] / s) - z, 0.0), (double)nq[sd]);
                const double d = (double)fabsf(v) - cand_lev[sd][q];
                err[sd] += d * d;
            }
            for (int sd = 0; sd < 2; ++sd) err[sd] = block_reduce(err[sd], [](double a, double b) { return a + b; }, red);
            if (tid < 2 && cand_ok[tid] && err[tid] < best_err[tid]) {
                best_err[tid] = err[tid];
                best[tid].s = cand_sz[tid][0]; best[tid].z = cand_sz[tid][1];
                best[tid].factor = tid ? grid.b[c] : grid.a[c];
                found[tid] = 1;
            }
            __syncthreads();
        }
        if (tid < 2 && !found[tid]) {               // no usable range: unit step anchored at the smallest element
            best[tid].s = 1.0; best[tid].z = cnt[tid] ? rint(lmin[tid]) : 0.0; best[tid].factor = 1.0;
        }
        __syncthreads();
        // final level table of the group: entry u = c + half
        __shared__ double T[16];
        if (tid < nlev) {
            const int cc = tid - half;
            double v;
            if (cc > 0) v = cnt[0] ? level_value(best[0].s * ((double)cc + best[0].z), I) : 0.0;
            else if (cc < 0) v = cnt[1] ? -level_value(best[1].s * ((double)(-cc) + best[1].z), I) : 0.0;
            else v = cnt[0] ? level_value(best[0].s * best[0].z, I) : 0.0;
            T[tid] = v;
            levels[((size_t)n * ngrp + g) * nlev + tid] = (float)v;
        }
        if (tid == 0 && meta) {
            double* mt = meta + ((size_t)n * ngrp + g) * 6;
            mt[0] = best[0].s; mt[1] = best[0].z; mt[2] = best[1].s; mt[3] = best[1].z;
            mt[4] = best[0].factor; mt[5] = best[1].factor;
        }
        __syncthreads();
        // codes, two per byte; per-thread partial of the de-quantized sum
        double part = 0.0;
        uint8_t* cdst = codes + ((size_t)n * K + (size_t)g * G) / 2;
        for (int j = tid; j < G / 2; j += nthr) {
            uint32_t byte = 0;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int k = 2 * j + e;
                const float v = w[k];
                int cc = 0;
                if (v > 0.f) cc = (int)fmin(fmax(rint(lg[k] / best[0].s) - best[0].z, 0.0), (double)nq[0]);
                else if (v < 0.f) cc = -(int)fmin(fmax(rint(lg[k] / best[1].s) - best[1].z, 0.0), (double)nq[1]);
                const int u = cc + half;
                part += T[u];
                byte |= (uint32_t)u << (4 * e);
            }
            cdst[j] = (uint8_t)byte;
        }
        part = block_reduce(part, [](double a, double b) { return a + b; }, red);
        row_sum += part;
        __syncthreads();
    }
    if (tid == 0) wsum[n] = (float)row_sum;
}

}  // namespace

extern "C" lrq_status lrq_tlq_quantize_weights(const float* W_rot, int N, int K, const lrq_tlq_params* p,
                                               uint8_t* codes, float* levels, double* meta, float* wsum,
                                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
    (void)workspace; (void)workspace_bytes;
    if (!W_rot || !p || !codes || !levels || !wsum || N <= 0 || K <= 0) return LRQ_ERR_INVALID_ARG;
    if (!p->alpha || !p->beta) return LRQ_ERR_INVALID_ARG;
    if (!lrq_aligned(W_rot, 16) || !lrq_aligned(codes, 4) || !lrq_aligned(levels, 4)) return LRQ_ERR_INVALID_ARG;
    const int G = p->group_size > 0 ? p->group_size : K;
    if (p->w_bits < 2 || p->w_bits > 4) return LRQ_ERR_UNSUPPORTED;
    if (p->integerize_I < 1 || p->integerize_I > 7) return LRQ_ERR_UNSUPPORTED;
    if (p->n_alpha < 1 || p->n_alpha > kMaxGrid || p->n_beta < 1 || p->n_beta > kMaxGrid) return LRQ_ERR_UNSUPPORTED;
    if (K % G || G % 8 || (K & 1)) return LRQ_ERR_UNSUPPORTED;
    if ((size_t)G * sizeof(double) > 160 * 1024) return LRQ_ERR_UNSUPPORTED;
    ClipGrid grid;
    grid.na = p->n_alpha; grid.nb = p->n_beta;
    for (int i = 0; i < kMaxGrid; ++i) {
        grid.a[i] = i < grid.na ? p->alpha[i] : 0.0;
        grid.b[i] = i < grid.nb ? p->beta[i] : 0.0;
    }
    const size_t smem = (size_t)G * sizeof(double);
    if (smem > 40 * 1024)
        LRQ_CUDA_TRY(cudaFuncSetAttribute(tlq_quantize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int threads = G >= 1024 ? 256 : 128;
    tlq_quantize_kernel<<<N, threads, smem, (cudaStream_t)cuda_stream>>>(W_rot, N, K, G, p->w_bits, p->integerize_I,
                                                                         grid, codes, levels, meta, wsum);
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}
