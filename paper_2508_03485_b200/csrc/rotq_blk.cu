// Rotation + per-token activation quantization (Sec. 4.2 Eq. 12, first case; Sec. 3.1 Eq. 1): the kernel for
// Hadamard blocks of up to 128 channels, the block size of the DiT workloads.
//
// HBM-bound by intent: each activation is read once (bf16) and written once as a 4- or 8-bit code.  What the
// kernel has to hide is not bandwidth but latency: a token's range is known only after every thread that holds a
// part of it has finished its butterflies, so each step ends in a reduction, a barrier and a short dependent
// chain.  The kernel therefore runs one CTA per SM made of several independent sub-groups (a few warps each, their
// own shared-memory stages, mbarriers and named barrier) that take steps from a common counter on demand; while one
// sub-group sits in its reduction the others keep the arithmetic pipes busy.
//   * A thread owns 64 consecutive channels of one token.  Index bits 0-5 of the transform are butterflies between
//     its own registers (packed two-wide fp32 adds).  For B = 128 the two threads of a block are neighbouring lanes:
//     the odd one runs its bit-5 stage with the outputs swapped (a fused multiply-add with -1), so that both keep
//     registers 0-31 and hand registers 32-63 to the partner with one shuffle each; bit 6 is then a register
//     butterfly again.  The odd thread's differences come out negated, which its reciprocal step absorbs.
//   * Tokens arrive through TMA: one 3-D bulk-tensor copy brings a step's tokens into shared memory as 128-byte
//     lines, 128-byte swizzled, two steps ahead of the arithmetic; a thread fetches its line with eight 128-bit
//     shared loads, conflict-free.  No load instruction touches global memory, no register holds prefetched data.
//   * Per-token range: each thread folds its 64 values, one redux per warp segment, whose first lane publishes the
//     part's extremes in shared memory; after the sub-group's barrier every warp reads the (at most four) parts of
//     its token and derives the step and zero-point itself (one lane; fp32 with error-free corrections, fp64 only
//     when min/s comes close to a rounding boundary).
//   * Quantization: one packed FMA (y / s - z), round to nearest even, saturating pack (the clamp of Eq. 1).
// The 1/sqrt(B) normalisation is never applied to elements: rint(y/s) is invariant under a common factor of y
// and s, so it is folded into the reported scale.
#include "lrq_internal.cuh"
#include "f32x2.cuh"
#include "rotq_common.cuh"
#include "tc_ptx.cuh"
#include "tma_host.cuh"
#include <climits>
#include <mutex>

namespace {
using namespace lrq_f2;
using namespace lrq_rq;
using namespace lrq_tc;

constexpr int EPT = 64;                  // elements per thread
constexpr int NP = EPT / 2;              // element pairs per thread
constexpr int NSTAGE = 2;                // token steps in flight per sub-group
constexpr int MAX_WARPS = 20;            // warps per CTA (one CTA per SM; 102 registers per thread)
constexpr int MAX_NSUB = 10;

struct SubCtl {
    uint64_t full[NSTAGE];               // stage filled by TMA (or marked "no more work")
    uint64_t empty[NSTAGE];              // stage read by all warps of the sub-group
    int group[NSTAGE];                   // step held by the stage, -1: none left
};
struct BlkCtl {
    SubCtl sub[MAX_NSUB];
    int next;                            // next unclaimed step of this CTA (steps are dealt to the sub-groups on demand)
    volatile int abort_flag;
};

__device__ __forceinline__ void lds128(uint32_t addr, uint4& v) {
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
}
__device__ __forceinline__ int lds32(uint32_t addr) {
    int v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_f2(uint32_t addr, float a, float b) {
    asm volatile("st.shared.v2.f32 [%0], {%1, %2};" :: "r"(addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void lds_f2(uint32_t addr, float& a, float& b) {
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(a), "=f"(b) : "r"(addr) : "memory");
}
__device__ __forceinline__ f32x2 shfl_xor2(f32x2 v, int m) {
    float a, b;
    unpack2(v, a, b);
    return pack2(__shfl_xor_sync(0xffffffffu, a, m), __shfl_xor_sync(0xffffffffu, b, m));
}

// Step and zero-point of a token (Eq. 1) from its extremes, in fp32 with error-free corrections, for the common
// case; the fp64 routine takes over when the token's range is degenerate or when min/s comes within 2e-3 of a
// rounding boundary, so that the zero-point is always the one exact arithmetic gives.  The reciprocal step is
// refined from the hardware approximation against the exact range (max - min as an unevaluated sum hi + lo), which
// leaves it within an ulp of the correctly rounded value: the same accuracy as rounding the fp64 result.
// scale_mul = nrm / qsteps rounded to fp32.
template <int A_BITS>
__device__ __forceinline__ TokenQ token_params_f32(float mn, float mx, int mode, float scale_mul, double nrm,
                                                   float* scale_out, int32_t* zp_out) {
    const bool asym = mode == LRQ_ACT_ASYM;
    const float qs = asym ? (float)((1 << A_BITS) - 1) : (float)((1 << (A_BITS - 1)) - 1);
    float hi, lo;
    if (asym) {
        hi = mx - mn;                                          // TwoSum(mx, -mn): hi + lo is the exact range
        const float bv = hi - mx;
        lo = (mx - (hi - bv)) + (-mn - bv);
    } else {
        hi = fmaxf(fabsf(mn), fabsf(mx)); lo = 0.f;
    }
    if (hi > 1e-30f && hi < 1e30f) {
        float r;
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(hi));
        float inv = qs * r;
        float e = fmaf(-hi, inv, qs);
        e = fmaf(-lo, inv, e);
        inv = fmaf(e, r, inv);
        const float p = mn * inv, zr = rintf(p);
        if (!asym || fabsf(fabsf(p - zr) - 0.5f) > 2e-3f) {
            const float z = asym ? zr : -(float)(1 << (A_BITS - 1));
            *scale_out = hi * scale_mul;
            *zp_out = (int32_t)z;
            TokenQ t;
            t.inv = inv; t.negz = -z;
            return t;
        }
    }
    return token_params_fast(mn, mx, A_BITS, mode, nrm, scale_out, zp_out);
}

// 32 consecutive values (16 pairs) -> codes; A8: 32 bytes (two 128-bit stores), A4: 16 bytes (one)
template <int A_BITS>
__device__ __forceinline__ void quantize_store_32(const f32x2* P, f32x2 INV, f32x2 NEGZ, uint8_t* dst) {
    int q[32];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        float x, y;
        unpack2(fma2(P[i], INV, NEGZ), x, y);
        q[2 * i] = __float2int_rn(x); q[2 * i + 1] = __float2int_rn(y);
    }
    if (A_BITS == 8) {
        uint32_t w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = pack_u8x4(q[4 * i], q[4 * i + 1], q[4 * i + 2], q[4 * i + 3]);
        reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
        reinterpret_cast<uint4*>(dst)[1] = make_uint4(w[4], w[5], w[6], w[7]);
    } else {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] = pack_u4x8(q + 8 * i);
        reinterpret_cast<uint4*>(dst)[0] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

template <int LOG2B, int A_BITS>
__global__ void __launch_bounds__(MAX_WARPS * 32, 1)
rotq_blk_kernel(const __grid_constant__ CUtensorMap tmX, int M, int K, int mode, int tok_per_step, int num_steps,
                int sub_warps, uint32_t stage_bytes, float scale_mul, const float* __restrict__ prescale,
                uint8_t* __restrict__ codes, float* __restrict__ scale, int32_t* __restrict__ zp, int* status) {
    static_assert(LOG2B >= 3 && LOG2B <= 7, "blocks of 8..128 channels");
    constexpr bool PAIRED = LOG2B == 7;              // a block spans two neighbouring threads
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    const int sub_threads = sub_warps * 32;
    const int nsub = blockDim.x / sub_threads;
    BlkCtl* ctl = reinterpret_cast<BlkCtl*>(base + (size_t)nsub * NSTAGE * stage_bytes);
    const int ext_tok = tok_per_step + 1;            // one more slot: the idle thread slots of a sub-group fold into it

    const int tpt = K / EPT;                         // threads per token = 128-byte lines per token
    const int tid = threadIdx.x, lane = tid & 31;
    const int sg = tid / sub_threads, ts = tid - sg * sub_threads;
    const bool active = ts < tok_per_step * tpt;
    const int tl = active ? ts / tpt : tok_per_step; // token within the step (idle slots: the extra one)
    const int jh = active ? ts - tl * tpt : 0;       // thread within the token: channels 64 jh .. 64 jh + 63
    const unsigned seg_mask = __match_any_sync(0xffffffffu, tl);
    const int seg_lane = __ffs(seg_mask) - 1;
    const bool seg_leader = lane == seg_lane;
    SubCtl* sc = &ctl->sub[sg];
    // extremes of the token parts: [2 (step parity)][ext_tok][sub_warps] pairs (min, max), one per warp that holds a
    // part of the token; written before the sub-group's barrier, read after it, never reset
    const uint32_t ext0 = smem_u32(reinterpret_cast<float*>(ctl + 1)) + (uint32_t)(sg * 2 * ext_tok * sub_warps) * 8u;
    const int wsub = ts >> 5;                        // warp within the sub-group
    const int w_first = active ? (tl * tpt) >> 5 : wsub, w_last = active ? (tl * tpt + tpt - 1) >> 5 : wsub;
    const uint32_t group_addr = smem_u32(&sc->group[0]), abort_addr = smem_u32(const_cast<int*>(&ctl->abort_flag));
    const uint32_t tx_bytes = (uint32_t)tok_per_step * (uint32_t)K * 2u;
    const uint32_t stage0 = smem_u32(base) + (uint32_t)(sg * NSTAGE) * stage_bytes;

    if (ts == 0) {
        for (int s = 0; s < NSTAGE; ++s) { mbar_init(smem_u32(&sc->full[s]), 1); mbar_init(smem_u32(&sc->empty[s]), sub_warps); }
        if (tid == 0) { ctl->abort_flag = 0; ctl->next = 0; tma_prefetch_desc(&tmX); }
        mbar_init_fence();
    }
    __syncthreads();
    lrq_pdl_trigger();
    lrq_pdl_wait();                      // X may be the previous kernel's output; the code buffer may still be read by it

    // this thread's 128-byte line of a stage is line L = ts; its chunk c sits at c ^ (L & 7), i.e. at byte
    // (L * 128 + ((L & 7) << 4)) ^ (c << 4): consecutive lanes read consecutive lines, eight distinct chunk slots
    const uint32_t L = active ? (uint32_t)ts : 0u;
    const uint32_t line_off = L * 128u + ((L & 7u) << 4);

    // The sub-group's first thread deals the CTA's steps out: it claims the next one from the shared counter and
    // either starts its copy into stage s or, when none is left, completes the stage's barrier with the mark -1.
    auto refill = [&](int s) {
        int i;
        asm volatile("atom.shared.add.u32 %0, [%1], 1;" : "=r"(i) : "r"(smem_u32(&ctl->next)) : "memory");
        const long long step = (long long)blockIdx.x + (long long)i * gridDim.x;
        if (step < num_steps) {
            sc->group[s] = (int)step;
            mbar_arrive_expect_tx(smem_u32(&sc->full[s]), tx_bytes);
            tma_load_3d(stage0 + s * stage_bytes, &tmX, 0, 0, (int)step * tok_per_step, smem_u32(&sc->full[s]));
        } else {
            sc->group[s] = -1;
            mbar_arrive(smem_u32(&sc->full[s]));
        }
    };
    if (ts == 0) {
#pragma unroll
        for (int s = 0; s < NSTAGE; ++s) refill(s);
    }

    const int odd = PAIRED ? (jh & 1) : 0;           // second thread of a 128-channel block
    const float sgn = odd ? -1.f : 1.f;
    const double nrm = 1.0 / sqrt((double)(1 << LOG2B));
    int it = 0;
    bool aborted = false;
    for (;; ++it) {
        const int s = it % NSTAGE;
        const uint32_t ph = (uint32_t)(it / NSTAGE) & 1u;
        const bool ok = mbar_wait<32>(smem_u32(&sc->full[s]), ph, &ctl->abort_flag, status, 21);
        const int g = ok ? lds32(group_addr + 4u * s) : 0;
        if (ok && g < 0) break;                       // the same for the whole sub-group: no step left
        const int m = g * tok_per_step + tl;
        const bool live = active && m < M;
        f32x2 P[NP];
        {
            const uint32_t a0 = stage0 + s * stage_bytes + line_off;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint4 r;
                lds128(a0 ^ (uint32_t)(c << 4), r);
                const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    P[4 * c + i] = pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u));
            }
        }
        // the stage is handed back once every lane of the warp holds its values in registers
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sc->empty[s]));
        if (prescale) {                                       // smoothing multipliers (Sec. 5.1), before the rotation
            const float4* ps = reinterpret_cast<const float4*>(prescale + (size_t)jh * EPT);
#pragma unroll
            for (int i = 0; i < NP / 2; ++i) {
                const float4 f = __ldg(ps + i);
                P[2 * i] = mul2(P[2 * i], pack2(f.x, f.y)); P[2 * i + 1] = mul2(P[2 * i + 1], pack2(f.z, f.w));
            }
        }
        // index bit 0: the two halves of a pair; bits 1-4: between pairs
#pragma unroll
        for (int i = 0; i < NP; ++i) { float a, b; unpack2(P[i], a, b); P[i] = pack2(a + b, a - b); }
#pragma unroll
        for (int h = 1; h < 16 && (2 * h) < (1 << LOG2B); h <<= 1)
#pragma unroll
            for (int i = 0; i < NP; ++i)
                if (!(i & h)) { const f32x2 a = P[i], b = P[i | h]; P[i] = add2(a, b); P[i | h] = sub2(a, b); }
        if (LOG2B == 6) {
#pragma unroll
            for (int i = 0; i < 16; ++i) { const f32x2 a = P[i], b = P[i | 16]; P[i] = add2(a, b); P[i | 16] = sub2(a, b); }
        }
        if (PAIRED) {
            // bit 5 with the outputs of the odd thread swapped: registers 0-15 then hold what the thread keeps (its
            // half of the block's low or high 64), registers 16-31 what the partner needs
            const f32x2 S = pack2(sgn, sgn), NS = pack2(-sgn, -sgn);
#pragma unroll
            for (int i = 0; i < 16; ++i) { const f32x2 a = P[i], b = P[i | 16]; P[i] = fma2(b, S, a); P[i | 16] = fma2(b, NS, a); }
            // bit 6: own (kept) with the partner's; the odd thread's differences come out negated
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const f32x2 o = P[i], r = shfl_xor2(P[i | 16], 1);
                P[i] = add2(o, r); P[i | 16] = sub2(o, r);
            }
        }
        // extremes: independent chains over the thread's values, one redux per warp segment, one shared atomic
        float mn, mx;
        {
            float mn4[4], mx4[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float x, y;
                unpack2(P[q], x, y);
                mn4[q] = fminf(x, y); mx4[q] = fmaxf(x, y);
            }
#pragma unroll
            for (int i = 4; i < 16; ++i) {
                float x, y;
                unpack2(P[i], x, y);
                mn4[i & 3] = min3(mn4[i & 3], x, y); mx4[i & 3] = max3(mx4[i & 3], x, y);
            }
            float mnd[4], mxd[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float x, y;
                unpack2(P[16 + q], x, y);
                mnd[q] = fminf(x, y); mxd[q] = fmaxf(x, y);
            }
#pragma unroll
            for (int i = 20; i < 32; ++i) {
                float x, y;
                unpack2(P[i], x, y);
                mnd[i & 3] = min3(mnd[i & 3], x, y); mxd[i & 3] = max3(mxd[i & 3], x, y);
            }
            const float a = fminf(min3(mn4[0], mn4[1], mn4[2]), mn4[3]), b = fmaxf(max3(mx4[0], mx4[1], mx4[2]), mx4[3]);
            float c = fminf(min3(mnd[0], mnd[1], mnd[2]), mnd[3]), d = fmaxf(max3(mxd[0], mxd[1], mxd[2]), mxd[3]);
            if (odd) { const float t0 = -d; d = -c; c = t0; }          // true values of the odd thread's upper half
            mn = fminf(a, c); mx = fmaxf(b, d);
        }
        // one redux per warp segment; the segment's first lane publishes the part's extremes
        const uint32_t tok_ext = ext0 + (uint32_t)(((it & 1) * ext_tok + tl) * sub_warps) * 8u;
        {
            const int imn = __reduce_min_sync(seg_mask, lrq_ordered_int(mn)), imx = __reduce_max_sync(seg_mask, lrq_ordered_int(mx));
            if (seg_leader) sts_f2(tok_ext + 8u * wsub, lrq_ordered_float(imn), lrq_ordered_float(imx));
        }
        // the sub-group's warps meet on their own named barrier (ids 1..: barrier 0 is the CTA's)
        asm volatile("bar.sync %0, %1;" :: "r"(1 + sg), "r"(sub_threads) : "memory");
        if (lds32(abort_addr)) { aborted = true; break; }
        // every warp has handed stage s back (its arrival precedes the barrier above): claim a step for it
        if (ts == 0) {
            mbar_wait<0>(smem_u32(&sc->empty[s]), ph, &ctl->abort_flag, status, 22);
            refill(s);
        }
        // every warp works out its token's step and zero-point itself (one lane): no second barrier
        TokenQ t;
        {
            float scv = 0.f; int z = 0;
            t.inv = 0.f; t.negz = 0.f;
            if (seg_leader && active) {
                float a, b;
                lds_f2(tok_ext + 8u * w_first, a, b);
                for (int w = w_first + 1; w <= w_last; ++w) {
                    float a2, b2;
                    lds_f2(tok_ext + 8u * w, a2, b2);
                    a = fminf(a, a2); b = fmaxf(b, b2);
                }
                t = token_params_f32<A_BITS>(a, b, mode, scale_mul, nrm, &scv, &z);
                if (jh == 0 && live) { scale[m] = scv; zp[m] = z; }
            }
            t.inv = __shfl_sync(seg_mask, t.inv, seg_lane);
            t.negz = __shfl_sync(seg_mask, t.negz, seg_lane);
        }
        if (live) {
            const f32x2 INV = pack2(t.inv, t.inv), NEGZ = pack2(t.negz, t.negz);
            const f32x2 INVD = pack2(t.inv * sgn, t.inv * sgn);
            // PAIRED: registers 0-15 are channels 32 odd .. + 31 of the block, registers 16-31 the same 64 further up
            const size_t e0 = (size_t)m * K + (PAIRED ? (size_t)(jh >> 1) * 128 + (size_t)odd * 32 : (size_t)jh * EPT);
            const size_t e1 = e0 + (PAIRED ? 64 : 32);
            quantize_store_32<A_BITS>(P, INV, NEGZ, codes + (A_BITS == 8 ? e0 : e0 >> 1));
            quantize_store_32<A_BITS>(P + 16, INVD, NEGZ, codes + (A_BITS == 8 ? e1 : e1 >> 1));
        }
    }
    if (aborted && ts == 0) {
        // copies already issued still write this CTA's shared memory: let them land (bounded) before the CTA ends
        for (int back = 0; back < NSTAGE; ++back) {
            const int i2 = it + back;                                 // steps whose copy may be in flight
            const uint32_t bar = smem_u32(&sc->full[i2 % NSTAGE]);
            const long long t0 = clock64();
            while (!mbar_try_wait(bar, (uint32_t)(i2 / NSTAGE) & 1u) && clock64() - t0 < kWaitCycles / 8) {}
        }
    }
    __syncthreads();                     // no sub-group leaves while another may still use the shared control block
}

typedef lrq_status (*BlkLaunch)(const CUtensorMap&, int, int, int, int, int, int, int, uint32_t, float, const float*, uint8_t*, float*,
                                int32_t*, int, size_t, cudaStream_t);

template <int LOG2B, int A_BITS>
lrq_status launch_blk(const CUtensorMap& tm, int M, int K, int mode, int T, int steps, int sub_warps, int nsub, uint32_t stage_bytes,
                      float scale_mul, const float* prescale, uint8_t* codes, float* scale, int32_t* zp, int sms, size_t smem,
                      cudaStream_t st) {
    auto kern = rotq_blk_kernel<LOG2B, A_BITS>;
    // the shared-memory opt-in is a per-device function attribute: set once per device and kernel variant
    static std::mutex mu;
    static bool configured[LRQ_MAX_DEVICES] = {};
    int dev = 0;
    if (lrq_current_device(&dev, nullptr) != LRQ_OK) return LRQ_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!configured[dev]) {
            LRQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 210 * 1024));
            configured[dev] = true;
        }
    }
    // one CTA per SM; each deals its steps (blockIdx, blockIdx + grid, ...) out to its sub-groups on demand
    const int per_cta = (steps + nsub - 1) / nsub;
    const int grid = per_cta < sms ? per_cta : sms;
    LRQ_CUDA_TRY(lrq_launch_pdl(kern, dim3(grid), dim3(nsub * sub_warps * 32), smem, st, tm, M, K, mode, T, steps, sub_warps, stage_bytes,
                                scale_mul, prescale, codes, scale, zp, lrq_status_word()));
    return LRQ_OK;
}

}  // namespace

// Returns LRQ_ERR_UNSUPPORTED for shapes this kernel does not take (the caller then uses the other kernels).
lrq_status lrq_launch_rotq_blk(const void* X, int M, int K, long ldx, int B, int a_bits, int mode, const float* prescale,
                               uint8_t* codes, float* scale, int32_t* zp, cudaStream_t st) {
    if (K % 128 || B < 8 || B > 128 || (ldx % 8) || !lrq_aligned(X, 16) || !lrq_aligned(codes, 16)) return LRQ_ERR_UNSUPPORTED;
    const int tpt = K / EPT;
    if (K / 64 > 256) return LRQ_ERR_UNSUPPORTED;
    int log2B = 0;
    while ((1 << log2B) < B) ++log2B;
    // Shape of the CTA.  A sub-group is sub_warps warps holding T whole tokens (a token is K/64 threads, rarely a
    // whole number of warps, so some thread slots idle); nsub of them fill the CTA's warps.  Preferred: the most
    // active threads per SM; among equals the smaller sub-group, i.e. the more independent ones (measured at
    // K = 4608: four sub-groups of five warps take 104 us, two of nine warps 111 us, for the same active threads).
    int sub_warps = 0, nsub = 0, T = 0;
    long best_threads = 0;
    for (int sw = 1; sw <= MAX_WARPS / 2; ++sw) {
        int t = sw * 32 / tpt;
        if (t < 1) continue;
        if (t > 256) t = 256;
        if (t > M) t = M;
        int ns = MAX_WARPS / sw;
        if (ns > MAX_NSUB) ns = MAX_NSUB;                       // named barriers 1..15 and the control block
        const size_t need = (size_t)ns * NSTAGE * lrq_round_up((size_t)t * K * 2, 1024);
        if (need > 190 * 1024) continue;
        const long threads = (long)t * tpt * ns;
        if (threads > best_threads) { best_threads = threads; sub_warps = sw; nsub = ns; T = t; }
    }
    if (!sub_warps) return LRQ_ERR_UNSUPPORTED;
    const uint32_t stage_bytes = (uint32_t)lrq_round_up((size_t)T * K * 2, 1024);
    const size_t smem = 1024 + (size_t)nsub * NSTAGE * stage_bytes + sizeof(BlkCtl) + (size_t)nsub * 2 * (T + 1) * sub_warps * 8 + 16;
    int sms = 0;
    if (lrq_current_device(nullptr, &sms) != LRQ_OK) return LRQ_ERR_CUDA;
    CUtensorMap tm;
    if (!lrq_tma::make_map_rows_bf16(&tm, X, (uint64_t)M, (uint64_t)K, (uint64_t)ldx, (uint32_t)T)) return LRQ_ERR_UNSUPPORTED;
    const int steps = (M + T - 1) / T;
    const double qsteps = mode == LRQ_ACT_ASYM ? (double)((1 << a_bits) - 1) : (double)((1 << (a_bits - 1)) - 1);
    const float scale_mul = (float)(1.0 / (sqrt((double)B) * qsteps));
    BlkLaunch fn = nullptr;
    switch (log2B * 2 + (a_bits == 8)) {
#define LRQ_CASE(L) case L * 2: fn = launch_blk<L, 4>; break; case L * 2 + 1: fn = launch_blk<L, 8>; break;
        LRQ_CASE(3) LRQ_CASE(4) LRQ_CASE(5) LRQ_CASE(6) LRQ_CASE(7)
#undef LRQ_CASE
        default: return LRQ_ERR_UNSUPPORTED;
    }
    return fn(tm, M, K, mode, T, steps, sub_warps, nsub, stage_bytes, scale_mul, prescale, codes, scale, zp, sms, smem, st);
}
