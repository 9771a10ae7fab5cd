// Twin-log weight quantization with search-based clipping (Sec. 4.1, Eqs. 4-9).
//
// Offline step.  One CTA of two warps per output row walks the row's groups.  The search of Eq. 6 is a
// comparison of sums of squared errors, and near-ties between two clipping factors do occur (two factors that
// give the same codes and differ only in the lowest level): which one wins then depends on how the fp64 sum
// was rounded.  The sum is therefore taken exactly as its definition reads - over the side's elements in
// increasing k, one add after another, products and sums rounded separately - and the parallelism is across
// candidates instead of across elements: warp 0 scores the positive side, warp 1 the negative side, each lane
// one clipping factor of the caller's grid, all lanes walking over the same elements (a lane computes log2|w|
// for one element of a 32-element chunk; the chunk is then handed round by shuffles).  Every decision (codes,
// chosen factor) is taken in fp64 with explicitly rounded operations, so no multiply-add is ever fused.
#include "lrq_internal.cuh"
#include <climits>

namespace {

constexpr int kMaxGrid = 64;
constexpr int kThreads = 64;
struct ClipGrid { double a[kMaxGrid]; double b[kMaxGrid]; int na, nb; };

__device__ __forceinline__ double level_value(double e, int I) {
    // Eqs. 8-9: 2^e ~ II * 2^(f-I) with f = floor(e), II = rint(2^(e-f) * 2^I)
    const double f = floor(e);
    const double II = rint(exp2(__dsub_rn(e, f)) * (double)(1 << I));      // the factor is a power of two: exact
    return ldexp(II, (int)f - I);
}

// code of Eq. 5 on one side: clamp(rint(l / s) - z, 0, nq)
__device__ __forceinline__ int side_code(double l, double s, double z, int nq) {
    return (int)fmin(fmax(__dsub_rn(rint(__ddiv_rn(l, s)), z), 0.0), (double)nq);
}

__device__ __forceinline__ double shfl_double(double v, int src) {
    return __hiloint2double(__shfl_sync(0xffffffffu, __double2hiint(v), src), __shfl_sync(0xffffffffu, __double2loint(v), src));
}

struct Side { double s, z, factor; };

__global__ void __launch_bounds__(kThreads)
tlq_quantize_kernel(const float* __restrict__ W, int N, int K, int G, int bits, int I, ClipGrid grid, int pack3,
                    uint8_t* __restrict__ codes, float* __restrict__ levels, double* __restrict__ meta,
                    float* __restrict__ wsum) {
    __shared__ double cand_lev[2][9][32];          // level table of each lane's candidate, per side
    __shared__ double ext[2][2][2];                // [warp][side][max, min] of log2|w|
    __shared__ int ext_cnt[2][2];
    __shared__ Side best[2];
    __shared__ double T[16];
    __shared__ double red[2];

    const int n = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int half = 1 << (bits - 1), nlev = 1 << bits, ngrp = K / G;
    double row_sum = 0.0;                          // meaningful in thread 0

    for (int g = 0; g < ngrp; ++g) {
        const float* w = W + (size_t)n * K + (size_t)g * G;
        // ---- extremes of log2|w| per side (order does not matter for max / min)
        double lmax[2] = {-INFINITY, -INFINITY}, lmin[2] = {INFINITY, INFINITY};
        int cnt[2] = {0, 0};
        for (int k = tid; k < G; k += kThreads) {
            const float v = w[k];
            if (v != 0.f) {
                const double l = log2((double)fabsf(v));
                const int sd = v < 0.f;
                lmax[sd] = fmax(lmax[sd], l); lmin[sd] = fmin(lmin[sd], l); cnt[sd]++;
            }
        }
#pragma unroll
        for (int sd = 0; sd < 2; ++sd) {
#pragma unroll
            for (int o = 16; o; o >>= 1) {
                lmax[sd] = fmax(lmax[sd], shfl_double(lmax[sd], lane ^ o));
                lmin[sd] = fmin(lmin[sd], shfl_double(lmin[sd], lane ^ o));
                cnt[sd] += __shfl_xor_sync(0xffffffffu, cnt[sd], o);
            }
            if (lane == 0) { ext[warp][sd][0] = lmax[sd]; ext[warp][sd][1] = lmin[sd]; ext_cnt[warp][sd] = cnt[sd]; }
        }
        __syncthreads();
        // ---- search of the clipping factor: warp `sd` owns side sd, lane c the c-th factor of that side's grid
        const int sd = warp;
        const int nq = sd ? half : half - 1;       // highest code of the side = denominator of Eq. 6
        const double smax = fmax(ext[0][sd][0], ext[1][sd][0]), smin = fmin(ext[0][sd][1], ext[1][sd][1]);
        const int scnt = ext_cnt[0][sd] + ext_cnt[1][sd];
        const int ng = sd ? grid.nb : grid.na;
        double best_err = INFINITY, best_s = 1.0, best_z = 0.0, best_f = 1.0;
        bool found = false;
        for (int c0 = 0; c0 < ng; c0 += 32) {
            const int c = c0 + lane;
            bool ok = false;
            double s = 1.0, z = 0.0, fac = 1.0;
            if (c < ng && scnt > 0 && nq > 0) {
                fac = sd ? grid.b[c] : grid.a[c];
                const double top = __dmul_rn(fac, smax), bot = smin;
                if (top > bot) {
                    s = __ddiv_rn(__dsub_rn(top, bot), (double)nq);
                    z = rint(__ddiv_rn(bot, s));
                    ok = true;
                }
            }
            __syncwarp();
            for (int q = 0; q <= nq; ++q)
                cand_lev[sd][q][lane] = ok ? level_value(__dmul_rn(s, __dadd_rn((double)q, z)), I) : 0.0;
            __syncwarp();
            // the side's elements in increasing k, one chunk of 32 at a time
            double err = 0.0;
            for (int k0 = 0; k0 < G; k0 += 32) {
                const int k = k0 + lane;
                const float v = k < G ? w[k] : 0.f;
                const bool mine = sd ? (v < 0.f) : (v > 0.f);
                const double a = (double)fabsf(v);
                const double l = mine ? log2(a) : 0.0;
                unsigned m = __ballot_sync(0xffffffffu, mine);
                while (m) {
                    const int j = __ffs(m) - 1;
                    m &= m - 1;
                    const double lj = shfl_double(l, j), aj = shfl_double(a, j);
                    if (ok) {
                        const double d = __dsub_rn(aj, cand_lev[sd][side_code(lj, s, z, nq)][lane]);
                        err = __dadd_rn(err, __dmul_rn(d, d));
                    }
                }
            }
            // first minimum in grid order: the smallest error, the lowest index among equals
            double e = ok ? err : INFINITY;
            int idx = ok ? c : INT_MAX;
#pragma unroll
            for (int o = 16; o; o >>= 1) {
                const double e2 = shfl_double(e, lane ^ o);
                const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
                if (e2 < e || (e2 == e && i2 < idx)) { e = e2; idx = i2; }
            }
            if (idx != INT_MAX && e < best_err) {  // a later pass replaces the best only when strictly smaller
                const int src = idx - c0;
                best_err = e;
                best_s = shfl_double(s, src); best_z = shfl_double(z, src); best_f = shfl_double(fac, src);
                found = true;
            }
        }
        if (!found) {                               // no usable range: unit step anchored at the smallest element
            best_s = 1.0; best_z = scnt ? rint(smin) : 0.0; best_f = 1.0;
        }
        if (lane == 0) { best[sd].s = best_s; best[sd].z = best_z; best[sd].factor = best_f; }
        __syncthreads();
        // ---- final level table of the group: entry u = c + half
        const int pcnt = ext_cnt[0][0] + ext_cnt[1][0], ncnt = ext_cnt[0][1] + ext_cnt[1][1];
        if (tid < nlev) {
            const int cc = tid - half;
            double v;
            if (cc > 0) v = pcnt ? level_value(__dmul_rn(best[0].s, __dadd_rn((double)cc, best[0].z)), I) : 0.0;
            else if (cc < 0) v = ncnt ? -level_value(__dmul_rn(best[1].s, __dadd_rn((double)(-cc), best[1].z)), I) : 0.0;
            else v = pcnt ? level_value(__dmul_rn(best[0].s, best[0].z), I) : 0.0;
            T[tid] = v;
            levels[((size_t)n * ngrp + g) * nlev + tid] = (float)v;
        }
        if (tid == 0 && meta) {
            double* mt = meta + ((size_t)n * ngrp + g) * 6;
            mt[0] = best[0].s; mt[1] = best[0].z; mt[2] = best[1].s; mt[3] = best[1].z;
            mt[4] = best[0].factor; mt[5] = best[1].factor;
        }
        __syncthreads();
        // ---- codes, eight at a time (one 32-bit word of nibbles, or three bytes of packed 3-bit codes)
        double part = 0.0;
        for (int j = tid; j < G / 8; j += kThreads) {
            uint32_t word = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float v = w[8 * j + e];
                int cc = 0;
                if (v > 0.f) cc = side_code(log2((double)v), best[0].s, best[0].z, half - 1);
                else if (v < 0.f) cc = -side_code(log2((double)-v), best[1].s, best[1].z, half);
                const int u = cc + half;
                part += T[u];
                word |= (uint32_t)u << ((pack3 ? 3 : 4) * e);
            }
            if (pack3) {
                uint8_t* dst = codes + ((size_t)n * K + (size_t)g * G) / 8 * 3 + (size_t)3 * j;
                dst[0] = (uint8_t)word; dst[1] = (uint8_t)(word >> 8); dst[2] = (uint8_t)(word >> 16);
            } else {
                *reinterpret_cast<uint32_t*>(codes + ((size_t)n * K + (size_t)g * G) / 2 + (size_t)4 * j) = word;
            }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) part += shfl_double(part, lane ^ o);
        if (lane == 0) red[warp] = part;
        __syncthreads();
        if (tid == 0) row_sum += red[0] + red[1];
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
    if (p->code_layout != LRQ_CODES_NIBBLE && p->code_layout != LRQ_CODES_PACKED3) return LRQ_ERR_INVALID_ARG;
    if (p->code_layout == LRQ_CODES_PACKED3 && p->w_bits != 3) return LRQ_ERR_UNSUPPORTED;
    ClipGrid grid;
    grid.na = p->n_alpha; grid.nb = p->n_beta;
    for (int i = 0; i < kMaxGrid; ++i) {
        grid.a[i] = i < grid.na ? p->alpha[i] : 0.0;
        grid.b[i] = i < grid.nb ? p->beta[i] : 0.0;
    }
    tlq_quantize_kernel<<<N, kThreads, 0, (cudaStream_t)cuda_stream>>>(W_rot, N, K, G, p->w_bits, p->integerize_I, grid,
                                                                      p->code_layout == LRQ_CODES_PACKED3 ? 1 : 0, codes,
                                                                      levels, meta, wsum);
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}
