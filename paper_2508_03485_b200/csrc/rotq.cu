// Rotation + per-token activation quantization (Sec. 4.2 Eq. 12, first case; Sec. 3.1 Eq. 1).
//
// HBM-bound step: each activation is read once (bf16) and written once as a 4- or 8-bit code.
// This file holds the register-resident kernels: a thread keeps 8 consecutive channels of a token (16 with
// 256-bit loads), runs the first butterfly stages of the block-diagonal Walsh-Hadamard transform on them in
// fp32, the next stages by warp shuffles, and for blocks above 256 the rest through one shared-memory
// transpose; the per-token range is reduced with redux.sync and one named barrier, and the kernel is
// persistent with the next token group's loads in flight.  Blocks of 8..128 with K a multiple of 128 go to the
// TMA-fed kernel of rotq_blk.cu first; a generic shared-memory kernel covers whatever neither takes.
// The 1/sqrt(B) normalisation is never applied to the elements: it is folded into the per-token scale, since
// rint(y/s) is invariant under a common factor of y and s.  The fp32 quantizer after a dense rotation and the
// fluctuation metric of Eq. 11 live here as well.
#include "lrq_internal.cuh"
#include "f32x2.cuh"
#include "rotq_common.cuh"
#include <climits>
#include <mutex>
#include <vector>

namespace {
using namespace lrq_rq;

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
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
rotq_generic_kernel(const void* __restrict__ Xv, int M, int K, long ldx, int log2B, int a_bits, int mode,
                    const float* __restrict__ prescale,
                    uint8_t* __restrict__ codes, float* __restrict__ scale, int32_t* __restrict__ zp) {
    extern __shared__ float row[];
    __shared__ float red_mn[8], red_mx[8], red_am[8];
    __shared__ TokenQ tq;
    const int m = blockIdx.x;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int nchunk = K >> 3;
    lrq_pdl_trigger();
    lrq_pdl_wait();

    {
        const uint4* src = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(Xv) + (size_t)m * ldx);
        for (int c = tid; c < nchunk; c += nthr) {
            float v[8];
            unpack_bf16x8(src[c], v);
            if (prescale) {                                   // smoothing multipliers (Sec. 5.1), before the rotation
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] *= __ldg(prescale + c * 8 + i);
            }
            if (log2B >= 3) bfly8(v);
#pragma unroll
            for (int i = 0; i < 8; ++i) row[c * 8 + i] = v[i];
        }
    }
    __syncthreads();
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
        const double nrm = 1.0 / sqrt((double)(1 << log2B));
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
// Fast kernel.  A thread owns 32 consecutive elements of one token (four 128-bit loads in flight,
// the next token group's loads issued before the current group's arithmetic): index bits 0-4 of the
// transform are butterflies between its own registers, bits 5-8 (B up to 512) are butterflies with the
// lane whose index differs in one bit (two shuffles and one packed fused multiply-add per element pair
// and stage); larger blocks take rotq_big_kernel below.  All fp32 arithmetic on element
// pairs uses the packed two-wide instructions (add/sub/fma.f32x2): one issue slot per two elements.
// A CTA holds T whole tokens (T * K/32 threads, a multiple of 32) and walks over token groups with
// a grid stride; the token's extremes are reduced through shared memory, then every thread
// quantizes and packs its own 32 values from registers: 32 bytes (8-bit codes) or 16 bytes (4-bit
// codes) per thread, contiguous across the warp.
// ------------------------------------------------------------------------------------------------
constexpr int EPT = 32;
using namespace lrq_f2;

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// A thread's 64 input bytes.  WIDE: two 256-bit loads, so that every lane reads whole 32-byte sectors (with
// 128-bit loads at a 64-byte lane stride each sector would be requested twice); needs 32-byte aligned rows.
template <bool WIDE>
__device__ __forceinline__ void load_raw(const __nv_bfloat16* p, uint4* raw) {
    if (WIDE) {
#pragma unroll
        for (int i = 0; i < 2; ++i)
            asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(raw[2 * i].x), "=r"(raw[2 * i].y), "=r"(raw[2 * i].z), "=r"(raw[2 * i].w),
                           "=r"(raw[2 * i + 1].x), "=r"(raw[2 * i + 1].y), "=r"(raw[2 * i + 1].z), "=r"(raw[2 * i + 1].w)
                         : "l"(p + 16 * i));
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) raw[i] = ldg_stream(reinterpret_cast<const uint4*>(p) + i);
    }
}

template <int LOG2B, int A_BITS, int MAX_THREADS, int MIN_CTAS, bool WIDE>
__global__ void __launch_bounds__(MAX_THREADS, MIN_CTAS)
rotq_fast_kernel(const __nv_bfloat16* __restrict__ X, int M, int K, long ldx, int mode, int tok_per_cta, int num_groups,
                 const float* __restrict__ prescale,
                 uint8_t* __restrict__ codes, float* __restrict__ scale, int32_t* __restrict__ zp) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int NP = EPT / 2;                      // element pairs per thread
    const int tpt = K / EPT;                         // threads per token
    const int tid = threadIdx.x, lane = tid & 31;
    const int tl = tid / tpt, j = tid - tl * tpt;    // token within the CTA, thread within the token
    int* ext = reinterpret_cast<int*>(smem_raw);     // [3][tok_per_cta][2] token extremes (ordered ints), rotating
    // lanes of this warp that belong to the same token, and the lowest of them
    const unsigned seg_mask = __match_any_sync(0xffffffffu, tl);
    const int seg_lane = __ffs(seg_mask) - 1;
    const bool seg_leader = lane == seg_lane;
    for (int i = tid; i < 3 * 2 * tok_per_cta; i += blockDim.x) ext[i] = (i & 1) ? INT_MIN : INT_MAX;
    __syncthreads();
    lrq_pdl_trigger();
    lrq_pdl_wait();                      // X may be the previous kernel's output; the code buffer may still be read by it

    uint4 raw[4];
    {
        const int m = blockIdx.x * tok_per_cta + tl;
        if (m < M) {
            load_raw<WIDE>(X + (size_t)m * ldx + (size_t)j * EPT, raw);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) raw[i] = make_uint4(0, 0, 0, 0);
        }
    }
    int it = 0;
    for (int g = blockIdx.x; g < num_groups; g += gridDim.x, ++it) {
        const int m = g * tok_per_cta + tl;
        const bool live = m < M;
        // bf16 -> fp32, two elements per word
        f32x2 P[NP];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
            for (int c = 0; c < 4; ++c)
                P[4 * i + c] = pack2(__uint_as_float(w[c] << 16), __uint_as_float(w[c] & 0xffff0000u));
        }
        if (prescale) {                                       // smoothing multipliers (Sec. 5.1), before the rotation
            const float4* ps = reinterpret_cast<const float4*>(prescale + (size_t)j * EPT);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float4 f = __ldg(ps + i);
                P[2 * i] = mul2(P[2 * i], pack2(f.x, f.y)); P[2 * i + 1] = mul2(P[2 * i + 1], pack2(f.z, f.w));
            }
        }
        // the next group's loads fly while this group is transformed
        {
            const int mn = (g + (int)gridDim.x) * tok_per_cta + tl;
            if (g + (int)gridDim.x < num_groups && mn < M) {
                load_raw<WIDE>(X + (size_t)mn * ldx + (size_t)j * EPT, raw);
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) raw[i] = make_uint4(0, 0, 0, 0);
            }
        }
        // index bit 0: the two halves of a pair
#pragma unroll
        for (int i = 0; i < NP; ++i) { float a, b; unpack2(P[i], a, b); P[i] = pack2(a + b, a - b); }
        // index bits 1..4: between pairs
#pragma unroll
        for (int h = 1; h < NP && (2 * h) < (1 << LOG2B); h <<= 1)
#pragma unroll
            for (int i = 0; i < NP; ++i)
                if (!(i & h)) { const f32x2 a = P[i], b = P[i | h]; P[i] = add2(a, b); P[i | h] = sub2(a, b); }
        // index bits 5..8: partner lanes
#pragma unroll
        for (int b = 5; b < LOG2B; ++b) {
            const int lm = 1 << (b - 5);
            const float sg = (lane & lm) ? -1.f : 1.f;
            const f32x2 S = pack2(sg, sg);
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                float x, y;
                unpack2(P[i], x, y);
                const float ox = __shfl_xor_sync(0xffffffffu, x, lm), oy = __shfl_xor_sync(0xffffffffu, y, lm);
                P[i] = fma2(P[i], S, pack2(ox, oy));     // low lane: own + other, high lane: other - own
            }
        }
        // extremes of the thread's values, of the token's lanes in this warp (one redux each on order-preserving
        // integer images), then of the token: one shared-memory atomic per warp and token, one CTA barrier
        float mn, mx;
        unpack2(P[0], mn, mx);
        { const float t0 = fminf(mn, mx); mx = fmaxf(mn, mx); mn = t0; }
#pragma unroll
        for (int i = 1; i < NP; ++i) { float x, y; unpack2(P[i], x, y); mn = min3(mn, x, y); mx = max3(mx, x, y); }
        int* slot = ext + (it % 3) * 2 * tok_per_cta + 2 * tl;
        {
            const int imn = __reduce_min_sync(seg_mask, lrq_ordered_int(mn)), imx = __reduce_max_sync(seg_mask, lrq_ordered_int(mx));
            if (seg_leader) { atomicMin(slot, imn); atomicMax(slot + 1, imx); }
        }
        __syncthreads();
        // every warp works out its token's step and zero-point itself (one lane, fp64): no second barrier
        TokenQ t;
        {
            float sc = 0.f; int z = 0;
            t.inv = 0.f; t.negz = 0.f;
            if (seg_leader) {
                const float a = lrq_ordered_float(slot[0]), b = lrq_ordered_float(slot[1]);
                t = token_params_fast(a, b, A_BITS, mode, 1.0 / sqrt((double)(1 << LOG2B)), &sc, &z);
                if (j == 0 && live) { scale[m] = sc; zp[m] = z; }
            }
            t.inv = __shfl_sync(seg_mask, t.inv, seg_lane);
            t.negz = __shfl_sync(seg_mask, t.negz, seg_lane);
        }
        // the slots used two groups from now are reset here: their last readers passed the barrier above, and
        // their next writers come after the next barrier
        if (tid < 2 * tok_per_cta) ext[((it + 2) % 3) * 2 * tok_per_cta + tid] = (tid & 1) ? INT_MIN : INT_MAX;
        if (live) {
            const f32x2 INV = pack2(t.inv, t.inv), NEGZ = pack2(t.negz, t.negz);
            int q[EPT];
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                float x, y;
                unpack2(fma2(P[i], INV, NEGZ), x, y);
                q[2 * i] = __float2int_rn(x); q[2 * i + 1] = __float2int_rn(y);
            }
            if (A_BITS == 8) {
                uint4* dst = reinterpret_cast<uint4*>(codes + (size_t)m * K + (size_t)j * EPT);
                uint32_t w[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) w[i] = pack_u8x4(q[4 * i], q[4 * i + 1], q[4 * i + 2], q[4 * i + 3]);
                if (WIDE) {
                    asm volatile("st.global.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                                 :: "l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                                 : "memory");
                } else {
                    dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                    dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
                }
            } else {
                uint4* dst = reinterpret_cast<uint4*>(codes + (((size_t)m * K + (size_t)j * EPT) >> 1));
                uint32_t w[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) w[i] = pack_u4x8(q + 8 * i);
                dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Large blocks (B = 1024, 2048, 4096).  With five or more index bits above a thread's own 32 elements,
// butterflies between lanes move every value through the shuffle network once per stage (20 bytes per element
// for bits 5-9, 8 more per shared-memory stage above).  This kernel instead re-distributes the data twice
// through shared memory and keeps every butterfly between a thread's own registers:
//   A  a warp transposes its 32 x 32 elements (index = 32 * row + col: each thread writes its row, reads its
//      column), after which index bits 5-9 are register butterflies;
//   B  the U = B/1024 warps of a transform block write their columns back and every thread reads four runs of
//      eight consecutive elements, one run per value of the block's top two index bits: bits 10-11 become
//      register butterflies too, and the runs are what the packer needs (4 or 8 code bytes each).
// Shared-memory traffic is 16 bytes per element in all.  Layouts: A is 32 rows of 128 bytes whose 16-byte
// chunks are swizzled by the row (rows written with 128-bit stores, columns read word by word, both
// conflict-free); B stores element y of the block at (y / 8) * 4 + y % 4 of one of two half-buffers chosen by
// bit 2 of y, the second half shifted by 16 banks, so that the word-wise writes and the 128-bit reads are
// conflict-free as well.  A warp's rows and its B words occupy the same two 2 KB pieces, so only the B reads
// cross warps: one barrier before them; the barrier of the extremes separates them from the next group.
// ------------------------------------------------------------------------------------------------
template <int LOG2B, int A_BITS, int MAX_THREADS, int MIN_CTAS, bool WIDE>
__global__ void __launch_bounds__(MAX_THREADS, MIN_CTAS)
rotq_big_kernel(const __nv_bfloat16* __restrict__ X, int M, int K, long ldx, int mode, int tok_per_cta, int num_groups,
                const float* __restrict__ prescale,
                uint8_t* __restrict__ codes, float* __restrict__ scale, int32_t* __restrict__ zp) {
    static_assert(LOG2B >= 10 && LOG2B <= 12, "block sizes 1024..4096");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int NP = EPT / 2;
    constexpr int U = 1 << (LOG2B - 10);             // warps per transform block
    constexpr int HALF_OFF = U * 512 + 16;           // floats from the first half-buffer to the second
    constexpr int UNIT_FLOATS = U * 1024 + 32;
    const int tpt = K / EPT;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tl = tid / tpt, j = tid - tl * tpt;
    int* ext = reinterpret_cast<int*>(smem_raw);
    float* buf = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(ext + 3 * 2 * tok_per_cta) + 127) & ~uintptr_t(127));
    const int wu = warp % U;                         // warp within the transform block
    // shared-memory byte addresses: the block's buffer, this warp's two 2 KB pieces (second = first + HALF_OFF floats)
    const uint32_t ub = (uint32_t)__cvta_generic_to_shared(buf + (warp / U) * UNIT_FLOATS);
    const uint32_t piece0 = ub + wu * 2048;
    // A: own row (written; chunk c at slot c ^ (lane & 7)), own column (read; word lane ^ 4 * (row & 7) of a row)
    const uint32_t rowa = piece0 + (lane < 16 ? lane * 128 : HALF_OFF * 4 + (lane - 16) * 128);
    const uint32_t l7s = (lane & 7) << 4;
    const uint32_t cola = piece0 + lane * 4;
    // B: own words (written), own runs (read)
    const uint32_t wra = piece0 + (((lane >> 2) & 1) ? HALF_OFF * 4 : 0) + ((lane >> 3) * 4 + (lane & 3)) * 4;
    const int tau = wu * 32 + lane;                  // thread within the block
    const uint32_t rda = ub + tau * 16;
    const int unit_in_token = j / (U * 32);

    const unsigned seg_mask = __match_any_sync(0xffffffffu, tl);
    const int seg_lane = __ffs(seg_mask) - 1;
    const bool seg_leader = lane == seg_lane;
    for (int i = tid; i < 3 * 2 * tok_per_cta; i += blockDim.x) ext[i] = (i & 1) ? INT_MIN : INT_MAX;
    __syncthreads();
    lrq_pdl_trigger();
    lrq_pdl_wait();                      // X may be the previous kernel's output; the code buffer may still be read by it

    uint4 raw[4];
    {
        const int m = blockIdx.x * tok_per_cta + tl;
        if (m < M) {
            load_raw<WIDE>(X + (size_t)m * ldx + (size_t)j * EPT, raw);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) raw[i] = make_uint4(0, 0, 0, 0);
        }
    }
    int it = 0;
    for (int g = blockIdx.x; g < num_groups; g += gridDim.x, ++it) {
        const int m = g * tok_per_cta + tl;
        const bool live = m < M;
        f32x2 P[NP];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
            for (int c = 0; c < 4; ++c)
                P[4 * i + c] = pack2(__uint_as_float(w[c] << 16), __uint_as_float(w[c] & 0xffff0000u));
        }
        if (prescale) {
            const float4* ps = reinterpret_cast<const float4*>(prescale + (size_t)j * EPT);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float4 f = __ldg(ps + i);
                P[2 * i] = mul2(P[2 * i], pack2(f.x, f.y)); P[2 * i + 1] = mul2(P[2 * i + 1], pack2(f.z, f.w));
            }
        }
        {
            const int mn = (g + (int)gridDim.x) * tok_per_cta + tl;
            if (g + (int)gridDim.x < num_groups && mn < M) {
                load_raw<WIDE>(X + (size_t)mn * ldx + (size_t)j * EPT, raw);
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) raw[i] = make_uint4(0, 0, 0, 0);
            }
        }
        // index bits 0..4 and, after the transposition, 5..9: the same register butterflies twice
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
            for (int i = 0; i < NP; ++i) { float a, b; unpack2(P[i], a, b); P[i] = pack2(a + b, a - b); }
#pragma unroll
            for (int h = 1; h < NP; h <<= 1)
#pragma unroll
                for (int i = 0; i < NP; ++i)
                    if (!(i & h)) { const f32x2 a = P[i], b = P[i | h]; P[i] = add2(a, b); P[i | h] = sub2(a, b); }
            if (pass == 0) {
                // A: rows out (chunk c of row `lane` at slot c ^ (lane & 7)), columns in
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    asm volatile("st.shared.v2.b64 [%0], {%1, %2};" :: "r"(rowa + (l7s ^ (c << 4))), "l"(P[2 * c]), "l"(P[2 * c + 1]) : "memory");
                __syncwarp();
#pragma unroll
                for (int i = 0; i < NP; ++i) {
                    // rows 2i and 2i+1 of the warp's 32 x 32 elements, word `lane` of each (swizzled by the row)
                    const int r = 2 * i;
                    const uint32_t rb = (r < 16 ? r * 128 : HALF_OFF * 4 + (r - 16) * 128);
                    float a, b;
                    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(a) : "r"((cola ^ ((r & 7) << 4)) + rb) : "memory");
                    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(b) : "r"((cola ^ (((r + 1) & 7) << 4)) + rb + 128) : "memory");
                    P[i] = pack2(a, b);
                }
                __syncwarp();                         // every lane has read its column before the words below land
            }
        }
        // B: the thread's column (element 32 * i + lane of the warp's 1024) out word by word, four runs of eight in
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            float a, b;
            unpack2(P[i], a, b);
            asm volatile("st.shared.f32 [%0], %1;" :: "r"(wra + (2 * i) * 64), "f"(a) : "memory");
            asm volatile("st.shared.f32 [%0], %1;" :: "r"(wra + (2 * i + 1) * 64), "f"(b) : "memory");
        }
        // the block's U warps meet on their own named barrier (ids 1..: barrier 0 is the CTA's)
        if (U == 1) __syncwarp(); else asm volatile("bar.sync %0, %1;" :: "r"(1 + warp / U), "n"(U * 32) : "memory");
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(P[4 * r]), "=l"(P[4 * r + 1]) : "r"(rda + r * (U * 512)) : "memory");
            asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(P[4 * r + 2]), "=l"(P[4 * r + 3]) : "r"(rda + r * (U * 512) + HALF_OFF * 4) : "memory");
        }
        // index bits 10..11: between the runs
#pragma unroll
        for (int h = (LOG2B == 12 ? 4 : 8); h < NP && LOG2B > 10; h <<= 1)
#pragma unroll
            for (int i = 0; i < NP; ++i)
                if (!(i & h)) { const f32x2 a = P[i], b = P[i | h]; P[i] = add2(a, b); P[i | h] = sub2(a, b); }

        float mn, mx;
        unpack2(P[0], mn, mx);
        { const float t0 = fminf(mn, mx); mx = fmaxf(mn, mx); mn = t0; }
#pragma unroll
        for (int i = 1; i < NP; ++i) { float x, y; unpack2(P[i], x, y); mn = min3(mn, x, y); mx = max3(mx, x, y); }
        int* slot = ext + (it % 3) * 2 * tok_per_cta + 2 * tl;
        {
            const int imn = __reduce_min_sync(seg_mask, lrq_ordered_int(mn)), imx = __reduce_max_sync(seg_mask, lrq_ordered_int(mx));
            if (seg_leader) { atomicMin(slot, imn); atomicMax(slot + 1, imx); }
        }
        __syncthreads();
        TokenQ t;
        {
            float sc = 0.f; int z = 0;
            t.inv = 0.f; t.negz = 0.f;
            if (seg_leader) {
                const float a = lrq_ordered_float(slot[0]), b = lrq_ordered_float(slot[1]);
                t = token_params_fast(a, b, A_BITS, mode, 1.0 / sqrt((double)(1 << LOG2B)), &sc, &z);
                if (j == 0 && live) { scale[m] = sc; zp[m] = z; }
            }
            t.inv = __shfl_sync(seg_mask, t.inv, seg_lane);
            t.negz = __shfl_sync(seg_mask, t.negz, seg_lane);
        }
        if (tid < 2 * tok_per_cta) ext[((it + 2) % 3) * 2 * tok_per_cta + tid] = (tid & 1) ? INT_MIN : INT_MAX;
        if (live) {
            const f32x2 INV = pack2(t.inv, t.inv), NEGZ = pack2(t.negz, t.negz);
            // run r holds elements r * (B / 4) + 8 * tau .. + 7 of the thread's transform block
            const size_t e0 = (size_t)m * K + (size_t)unit_in_token * (U * 1024) + (size_t)tau * 8;
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                int q[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float x, y;
                    unpack2(fma2(P[4 * r + i], INV, NEGZ), x, y);
                    q[2 * i] = __float2int_rn(x); q[2 * i + 1] = __float2int_rn(y);
                }
                const size_t e = e0 + (size_t)r * (U * 256);
                if (A_BITS == 8) {
                    *reinterpret_cast<uint2*>(codes + e) = make_uint2(pack_u8x4(q[0], q[1], q[2], q[3]), pack_u8x4(q[4], q[5], q[6], q[7]));
                } else {
                    *reinterpret_cast<uint32_t*>(codes + (e >> 1)) = pack_u4x8(q);
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Quantizer of already rotated fp32 rows whose extremes are known (dense path: the rotation GEMM's epilogue
// found them).  One warp per token, grid-stride; lane 0 works out the step and zero-point, then the warp
// streams the row: 32 bytes in (one 256-bit load), 8 or 4 code bytes out per lane and step.
// ext_min / ext_max alias scale / zp: the warp reads its row's extremes before it writes the results.
// ------------------------------------------------------------------------------------------------
template <int A_BITS>
__global__ void __launch_bounds__(256)
quant_rows_f32_kernel(const float* __restrict__ Y, int M, int K, int mode, uint8_t* __restrict__ codes,
                      float* scale, int32_t* zp) {
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    lrq_pdl_trigger();
    lrq_pdl_wait();                      // the rows and their extremes are the rotation kernel's output
    for (int m = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; m < M; m += warps) {
        TokenQ t;
        t.inv = 0.f; t.negz = 0.f;
        if (lane == 0) {
            const float mn = lrq_ordered_float(reinterpret_cast<const int*>(scale)[m]);
            const float mx = lrq_ordered_float(reinterpret_cast<const int*>(zp)[m]);
            float sc; int32_t z;
            t = token_params_fast(mn, mx, A_BITS, mode, 1.0, &sc, &z);
            scale[m] = sc; zp[m] = z;
        }
        t.inv = __shfl_sync(0xffffffffu, t.inv, 0);
        t.negz = __shfl_sync(0xffffffffu, t.negz, 0);
        const f32x2 INV = pack2(t.inv, t.inv), NEGZ = pack2(t.negz, t.negz);
        const float* row = Y + (size_t)m * K;
        for (int c = lane; c < (K >> 3); c += 32) {
            uint32_t r[8];
            asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                         : "l"(row + 8 * c));
            int q[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float x, y;
                unpack2(fma2(pack2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1])), INV, NEGZ), x, y);
                q[2 * i] = __float2int_rn(x); q[2 * i + 1] = __float2int_rn(y);
            }
            if (A_BITS == 8)
                *reinterpret_cast<uint2*>(codes + (size_t)m * K + 8 * c) = make_uint2(pack_u8x4(q[0], q[1], q[2], q[3]), pack_u8x4(q[4], q[5], q[6], q[7]));
            else
                *reinterpret_cast<uint32_t*>(codes + (((size_t)m * K) >> 1) + 4 * c) = pack_u4x8(q);
        }
    }
}

}  // namespace

lrq_status lrq_launch_quantize_f32_ext(const float* Y, int M, int K, int a_bits, int mode, uint8_t* codes,
                                       float* scale, int32_t* zp, cudaStream_t st) {
    if (!lrq_aligned(Y, 32)) return LRQ_ERR_INVALID_ARG;          // rows are K*4 bytes with K % 8 == 0: 32-byte aligned chunks
    int sms = 0;
    if (lrq_current_device(nullptr, &sms) != LRQ_OK) return LRQ_ERR_CUDA;
    const int blocks_needed = (M + 7) / 8;                        // 8 warps per CTA, one token per warp and step
    const int grid = blocks_needed < sms * 8 ? blocks_needed : sms * 8;
    if (a_bits == 8) LRQ_CUDA_TRY(lrq_launch_pdl(quant_rows_f32_kernel<8>, dim3(grid), dim3(256), 0, st, Y, M, K, mode, codes, scale, zp));
    else LRQ_CUDA_TRY(lrq_launch_pdl(quant_rows_f32_kernel<4>, dim3(grid), dim3(256), 0, st, Y, M, K, mode, codes, scale, zp));
    return LRQ_OK;
}

// ------------------------------------------------------------------------------------------------
// Fluctuation metric of a layer's activations (Sec. 4.2, Eq. 11): J = ||X||_F / sqrt(M K), and the rotation
// kind the threshold rule of Eq. 12 picks.  HBM-bound: 2 bytes per element, read once with 256-bit loads.
// Squares of bf16 values are exact in fp32; a thread sums its 16 squares in fp32 (relative error below
// 16 * 2^-24), everything above that in fp64.
// ------------------------------------------------------------------------------------------------
namespace {
__global__ void __launch_bounds__(256)
sumsq_kernel(const __nv_bfloat16* __restrict__ X, int M, int K, long ldx, double* __restrict__ acc) {
    const int cpr = K >> 4;                                  // 32-byte chunks per row
    double part = 0.0;
    // a warp walks over rows (grid stride), its lanes over the row's chunks, four loads in flight per lane
    const int lane = threadIdx.x & 31;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    for (int m = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; m < M; m += nwarps) {
        const __nv_bfloat16* row = X + (size_t)m * ldx;
        for (int c0 = lane; c0 < cpr; c0 += 128) {
            uint32_t r[4][8];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int c = c0 + 32 * u;
                if (c < cpr)
                    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                                 : "=r"(r[u][0]), "=r"(r[u][1]), "=r"(r[u][2]), "=r"(r[u][3]), "=r"(r[u][4]), "=r"(r[u][5]),
                                   "=r"(r[u][6]), "=r"(r[u][7]) : "l"(row + 16 * c));
                else {
#pragma unroll
                    for (int k = 0; k < 8; ++k) r[u][k] = 0;
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float s = 0.f;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float lo = __uint_as_float(r[u][k] << 16), hi = __uint_as_float(r[u][k] & 0xffff0000u);
                    s = fmaf(lo, lo, s); s = fmaf(hi, hi, s);
                }
                part += (double)s;
            }
        }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    __shared__ double wsum[8];
    if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = part;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += wsum[w];
        atomicAdd(acc, t);
    }
}
__global__ void ars_finish_kernel(const double* __restrict__ acc, double count, double thr, float* __restrict__ J,
                                  int* __restrict__ kind) {
    const double j = sqrt(*acc) / sqrt(count);
    *J = (float)j;
    *kind = j < thr ? (int)LRQ_ROT_HADAMARD : (int)LRQ_ROT_DENSE;
}
}  // namespace

lrq_status lrq_launch_ars_metric(const void* X, int M, int K, long ldx, double thr, float* J, int* kind, double* acc,
                                 cudaStream_t st) {
    int sms = 0;
    if (lrq_current_device(nullptr, &sms) != LRQ_OK) return LRQ_ERR_CUDA;
    LRQ_CUDA_TRY(cudaMemsetAsync(acc, 0, sizeof(double), st));
    long blocks = ((long)M + 7) / 8;                         // 8 warps per CTA, one row per warp and step
    if (blocks > (long)sms * 8) blocks = (long)sms * 8;
    sumsq_kernel<<<(int)blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(X), M, K, ldx, acc);
    LRQ_CUDA_TRY(cudaGetLastError());
    ars_finish_kernel<<<1, 1, 0, st>>>(acc, (double)M * (double)K, thr, J, kind);
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}

// CTAs of `kern` (with this CTA size and dynamic shared memory) that one SM keeps resident.  The answer, and the
// shared-memory opt-in it needs (a per-device function attribute), are worked out once per (kernel, device, shape)
// under a lock and remembered: the launch path itself then makes no runtime query.
static lrq_status resident_ctas(const void* kern, int dev, int threads, size_t smem, int* per_sm) {
    struct Entry { const void* kern; int dev, threads; size_t smem; int per_sm; };
    static std::mutex mu;
    static std::vector<Entry> cache;
    std::lock_guard<std::mutex> lock(mu);
    for (const Entry& e : cache)
        if (e.kern == kern && e.dev == dev && e.threads == threads && e.smem == smem) { *per_sm = e.per_sm; return LRQ_OK; }
    if (smem > 40 * 1024) LRQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int n = 0;
    LRQ_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, threads, smem));
    if (n < 1) return LRQ_ERR_UNSUPPORTED;
    cache.push_back({kern, dev, threads, smem, n});
    *per_sm = n;
    return LRQ_OK;
}

static lrq_status launch_generic(const void* X, int M, int K, long ldx, int log2B, int a_bits, int mode, const float* prescale,
                                 uint8_t* codes, float* scale, int32_t* zp, cudaStream_t st) {
    const size_t smem = (size_t)K * sizeof(float);
    if (smem > 200 * 1024) return LRQ_ERR_UNSUPPORTED;
    int dev = 0, per_sm = 0;
    if (lrq_current_device(&dev, nullptr) != LRQ_OK) return LRQ_ERR_CUDA;
    const int threads = (K >= 2048) ? 256 : (K >= 1024 ? 128 : 64);
    lrq_status rs = resident_ctas(reinterpret_cast<const void*>(rotq_generic_kernel), dev, threads, smem, &per_sm);   // sets the shared-memory opt-in
    if (rs != LRQ_OK) return rs;
    LRQ_CUDA_TRY(lrq_launch_pdl(rotq_generic_kernel, dim3(M), dim3(threads), smem, st, X, M, K, ldx, log2B, a_bits, mode, prescale, codes,
                                scale, zp));
    return LRQ_OK;
}

template <int LOG2B, bool BIG, int A_BITS, int NT, int NB, bool WIDE>
struct RotqPick {
    static constexpr auto kern = rotq_fast_kernel<LOG2B, A_BITS, NT, NB, WIDE>;
};
template <int LOG2B, int A_BITS, int NT, int NB, bool WIDE>
struct RotqPick<LOG2B, true, A_BITS, NT, NB, WIDE> {
    static constexpr auto kern = rotq_big_kernel<LOG2B, A_BITS, NT, NB, WIDE>;
};

template <int LOG2B, bool BIG = false>
static lrq_status launch_fast(const void* X, int M, int K, long ldx, int a_bits, int mode, const float* prescale, uint8_t* codes,
                              float* scale, int32_t* zp, cudaStream_t st) {
    const int tpt = K / EPT;
    // whole tokens per CTA: thread count a multiple of 32, at least 256 when the token is small
    int T = 1;
    while ((T * tpt) % 32) ++T;
    const int T0 = T;
    while (T * tpt < 256 && (T + T0) * tpt <= 512) T += T0;
    const int threads = T * tpt;
    if (threads > 512) return LRQ_ERR_UNSUPPORTED;
    size_t smem = 3 * 2 * sizeof(int) * T + (BIG ? 128 : 16);
    if (BIG) {                                       // one buffer of B + 32 floats per transform block held by the CTA
        const int B = 1 << LOG2B;
        smem += (size_t)(threads * EPT / B) * (size_t)(B + 32) * sizeof(float);
    }
    // register budget by CTA size: three CTAs of up to 288 threads, two of up to 384, else one
    typedef void (*Kern)(const __nv_bfloat16*, int, int, long, int, int, int, const float*, uint8_t*, float*, int32_t*);
    // 256-bit accesses when every thread's 64 input bytes and 32 code bytes start on 32-byte boundaries
    const bool wide = lrq_aligned(X, 32) && (ldx % 16) == 0 && lrq_aligned(codes, 32);
    Kern kern;
#define LRQ_PICK(NT, NB) (wide ? (a_bits == 8 ? RotqPick<LOG2B, BIG, 8, NT, NB, true>::kern : RotqPick<LOG2B, BIG, 4, NT, NB, true>::kern) \
                               : (a_bits == 8 ? RotqPick<LOG2B, BIG, 8, NT, NB, false>::kern : RotqPick<LOG2B, BIG, 4, NT, NB, false>::kern))
    if (threads <= 288) kern = LRQ_PICK(288, 3);
    else if (threads <= 384) kern = LRQ_PICK(384, 2);
    else kern = LRQ_PICK(512, 1);
#undef LRQ_PICK
    // persistent grid: as many CTAs as stay resident, each walking over token groups with a grid stride
    int dev = 0, sms = 0, per_sm = 0;
    if (lrq_current_device(&dev, &sms) != LRQ_OK) return LRQ_ERR_CUDA;
    lrq_status rs = resident_ctas(reinterpret_cast<const void*>(kern), dev, threads, smem, &per_sm);
    if (rs != LRQ_OK) return rs;
    const int groups = (M + T - 1) / T;
    const int grid = groups < sms * per_sm ? groups : sms * per_sm;
    LRQ_CUDA_TRY(lrq_launch_pdl(kern, dim3(grid), dim3(threads), smem, st, static_cast<const __nv_bfloat16*>(X), M, K, ldx, mode, T,
                                groups, prescale, codes, scale, zp));
    return LRQ_OK;
}

lrq_status lrq_launch_rotq_hadamard(const void* X, int M, int K, long ldx, int B, int a_bits, int mode, const float* prescale,
                                    uint8_t* codes, float* scale, int32_t* zp, cudaStream_t st) {
    // blocks of up to 128 channels: whole blocks per thread, TMA-fed (rotq_blk.cu), when the shape allows
    {
        const lrq_status r = lrq_launch_rotq_blk(X, M, K, ldx, B, a_bits, mode, prescale, codes, scale, zp, st);
        if (r != LRQ_ERR_UNSUPPORTED) return r;
    }
    int log2B = 0;
    while ((1 << log2B) < B) ++log2B;
    // the fast kernel needs whole 32-element thread slices and, for B >= 2048, whole-CTA tokens
    const bool fast_ok = (K % EPT) == 0 && B >= 8 && (ldx % 8) == 0;
    if (fast_ok) {
        lrq_status r = LRQ_ERR_UNSUPPORTED;
        switch (log2B) {
#define LRQ_CASE(L) case L: r = launch_fast<L>(X, M, K, ldx, a_bits, mode, prescale, codes, scale, zp, st); break;
            LRQ_CASE(3) LRQ_CASE(4) LRQ_CASE(5) LRQ_CASE(6) LRQ_CASE(7) LRQ_CASE(8) LRQ_CASE(9)
#undef LRQ_CASE
#define LRQ_CASE(L) case L: r = launch_fast<L, true>(X, M, K, ldx, a_bits, mode, prescale, codes, scale, zp, st); break;
            LRQ_CASE(10) LRQ_CASE(11) LRQ_CASE(12)
#undef LRQ_CASE
            default: break;
        }
        if (r != LRQ_ERR_UNSUPPORTED) return r;
    }
    return launch_generic(X, M, K, ldx, log2B, a_bits, mode, prescale, codes, scale, zp, st);
}
