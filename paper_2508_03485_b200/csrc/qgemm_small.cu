// Quantized contraction + epilogue for small token counts (Sec. 4.1, Eq. 10), where the layer is bound by
// streaming the weight codes once and by latency, not by tensor throughput: the kernel for M up to a few hundred
// tokens, and the one that reads TLQ's 3-bit codes in their true packing (eight codes in three bytes).
//
//   acc[m,n] = sum_k q[m,k] * T[n, k/G, u[n,k]]          exact bf16 products, fp32 accumulation in TMEM
//   Y[m,n]   = s_m * (acc + z_m * wsum_n) * wscale_n + bias_n
//
// The large-tile kernel (qgemm_tc.cu) gives a 256-token batch four tiles, so four CTA pairs work while 70 idle.
// Here a CTA owns 128 tokens x 32 output channels, so that a 1024 x 1024 layer at M = 256 spreads over 64 SMs and
// each weight row is fetched by at most M/128 CTAs.  The kernel is a chain of K/64 dependent steps, so what counts
// is the latency of one step: nine warps, so that a step's decode is spread thin, and every operand of the
// prologue and epilogue (level tables, per-token and per-channel terms) is requested before the first step.
//   warps 0-7   fetch the packed codes of both operands for the next k-block straight into registers (plain
//               coalesced loads, a few blocks ahead of the arithmetic), expand half a token row of activation codes each
//               and decode one 8-code group of weight codes through the row's level table (byte permutes
//               on two byte planes, as in the large-tile kernel) into bf16 stages in the K-major 128-byte-swizzled
//               UMMA layout; after the last k-block they read the accumulator (tcgen05.ld), scale and store
//   warp 8      allocates TMEM, stages the per-channel epilogue terms; one lane issues tcgen05.mma (M = 128, N = 32,
//               K = 16) and commits
// Packed 3-bit codes: a group of eight codes is three bytes at any byte offset; it is fetched as the 32-bit
// window starting there (two aligned words and a funnel shift) and its 3-bit fields are spread to nibbles with three
// mask-and-shift steps, after which it is the same word the nibble layout stores.
// The A operand is centred as in the large-tile kernel (q - 128, q - 8) and the epilogue's zero-point term absorbs
// the offset.  Every wait is bounded and reports through the status word.
#include "lrq_internal.cuh"
#include "tc_ptx.cuh"
#include "f32x2.cuh"
#include <mutex>

namespace {
using namespace lrq_tc;
using namespace lrq_f2;

constexpr int BM = 128, BN = 32, BK = 64;
constexpr int NSTG = 3;
constexpr int A_STAGE = BM * BK * 2;             // 16 KB
constexpr int B_STAGE = BN * BK * 2;             // 4 KB
constexpr int WORKERS = 256, NUM_THREADS = WORKERS + 32;
constexpr int TMEM_COLS = 32;

struct __align__(16) Ctl {
    uint64_t full[NSTG];          // stage written by the four worker warps
    uint64_t empty[NSTG];         // stage consumed by the MMAs (tcgen05.commit)
    uint64_t acc_full;            // accumulator complete
    uint32_t tmem_base;
    volatile int abort_flag;
    float col[3][BN];             // wsum, wscale, bias of the tile's columns (fetched while the main loop runs)
};
constexpr size_t SMEM_BYTES = 1024 + (size_t)NSTG * (A_STAGE + B_STAGE) + sizeof(Ctl);

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ uint32_t add_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4)); }
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// 8-bit codes: four per word -> bf16 of (q - 128): 0x4300 | (q & 0x7f) is 128 + (q & 0x7f); adding -256 (bit 7 clear)
// or -128 (bit 7 set) gives q - 128 exactly.
__device__ __forceinline__ void expand_a8(uint32_t w, uint32_t& o01, uint32_t& o23) {
    const uint32_t p01 = prmt(w, 0u, 0x4140u), p23 = prmt(w, 0u, 0x4342u);
    o01 = add_bf16x2((p01 & 0x007F007Fu) | 0x43004300u, (p01 & 0x00800080u) ^ 0xC380C380u);
    o23 = add_bf16x2((p23 & 0x007F007Fu) | 0x43004300u, (p23 & 0x00800080u) ^ 0xC380C380u);
}
// 4-bit codes: eight per word -> bf16 of (q - 8), emitted in the order k = 0,2, 4,6, 1,3, 5,7 (one permute per pair);
// the weight decode of 4-bit-activation layers emits the same order, and a sum does not care about the order of k
__device__ __forceinline__ void expand_a4(uint32_t w, uint32_t* o) {
    const uint32_t lo = w & 0x0F0F0F0Fu, hi = (w >> 4) & 0x0F0F0F0Fu;
    o[0] = add_bf16x2(prmt(lo, 0x43434343u, 0x4140u), 0xC308C308u);
    o[1] = add_bf16x2(prmt(lo, 0x43434343u, 0x4342u), 0xC308C308u);
    o[2] = add_bf16x2(prmt(hi, 0x43434343u, 0x4140u), 0xC308C308u);
    o[3] = add_bf16x2(prmt(hi, 0x43434343u, 0x4342u), 0xC308C308u);
}

// level table of one (row, group) as two byte planes (low / high byte of each bf16 entry)
struct Lut { uint32_t lo[4], hi[4]; };
template <int W_BITS>
__device__ __forceinline__ void load_lut(Lut& L, const float* __restrict__ tab) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (j < (1 << W_BITS) / 4) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(tab) + j);
            const uint32_t t01 = prmt(__float_as_uint(v.x), __float_as_uint(v.y), 0x7632u);
            const uint32_t t23 = prmt(__float_as_uint(v.z), __float_as_uint(v.w), 0x7632u);
            L.lo[j] = prmt(t01, t23, 0x6420u);
            L.hi[j] = prmt(t01, t23, 0x7531u);
        } else {
            L.lo[j] = 0; L.hi[j] = 0;
        }
    }
}
// eight codes as nibbles (one word) -> four registers of two bf16 each, in k order or in the 4-bit activation order
template <int W_BITS, bool A4_ORDER>
__device__ __forceinline__ void decode_w(uint32_t w, const Lut& L, uint32_t* o) {
    constexpr uint32_t S0 = A4_ORDER ? 0x6240u : 0x5140u, S1 = A4_ORDER ? 0x7351u : 0x7362u;
    const uint32_t selA = w & 0x77777777u, selB = selA >> 16;
    uint32_t loA, hiA, loB, hiB;
    if (W_BITS == 4) {
        const uint32_t x0 = w << 4;
        const uint32_t mA = prmt(x0, w, 0xD9C8u), mB = prmt(x0, w, 0xFBEAu);    // 0xFF where the code's top bit is set
        loA = (prmt(L.lo[0], L.lo[1], selA) & ~mA) | (prmt(L.lo[2], L.lo[3], selA) & mA);
        hiA = (prmt(L.hi[0], L.hi[1], selA) & ~mA) | (prmt(L.hi[2], L.hi[3], selA) & mA);
        loB = (prmt(L.lo[0], L.lo[1], selB) & ~mB) | (prmt(L.lo[2], L.lo[3], selB) & mB);
        hiB = (prmt(L.hi[0], L.hi[1], selB) & ~mB) | (prmt(L.hi[2], L.hi[3], selB) & mB);
    } else {
        loA = prmt(L.lo[0], L.lo[1], selA); hiA = prmt(L.hi[0], L.hi[1], selA);
        loB = prmt(L.lo[0], L.lo[1], selB); hiB = prmt(L.hi[0], L.hi[1], selB);
    }
    if (A4_ORDER) { o[0] = prmt(loA, hiA, S0); o[1] = prmt(loB, hiB, S0); o[2] = prmt(loA, hiA, S1); o[3] = prmt(loB, hiB, S1); }
    else { o[0] = prmt(loA, hiA, S0); o[1] = prmt(loA, hiA, S1); o[2] = prmt(loB, hiB, S0); o[3] = prmt(loB, hiB, S1); }
}
// eight 3-bit codes in the low 24 bits -> eight nibbles
__device__ __forceinline__ uint32_t spread3(uint32_t x) {
    x = (x & 0x00000FFFu) | ((x & 0x00FFF000u) << 4);        // two groups of four codes, one per 16-bit half
    x = (x & 0x003F003Fu) | ((x & 0x0FC00FC0u) << 2);        // four groups of two codes, one per byte
    return (x & 0x07070707u) | ((x & 0x38383838u) << 1);     // one code per nibble
}

struct Params {
    const uint8_t* a_codes; const float* a_scale; const int32_t* a_zp;
    const uint8_t* w_codes; const float* levels; const float* wsum; const float* wscale; const float* bias;
    void* Y; long ldy; int M, N, K, G, y_dtype; int* status;
};

template <int A_BITS, int W_BITS, bool PACKED3>
__global__ void __launch_bounds__(NUM_THREADS, 1)
qgemm_small_kernel(const Params p) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    unsigned char* sA = base;
    unsigned char* sB = base + NSTG * A_STAGE;
    Ctl* ctl = reinterpret_cast<Ctl*>(sB + NSTG * B_STAGE);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN, m0 = blockIdx.y * BM;
    const int kblocks = p.K / BK;
    constexpr int NLEV = 1 << W_BITS;
    constexpr uint32_t IDESC = umma_idesc_bf16(BM, BN, false, false);

    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTG; ++s) { mbar_init(smem_u32(&ctl->full[s]), WORKERS / 32); mbar_init(smem_u32(&ctl->empty[s]), 1); }
        mbar_init(smem_u32(&ctl->acc_full), 1);
        ctl->abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == WORKERS / 32) tmem_alloc(smem_u32(&ctl->tmem_base), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    lrq_pdl_trigger();
    if (threadIdx.x == 32) {
        // The tile's weight codes and level tables do not depend on the previous kernel: ask for them in L2 now, while
        // that kernel is still running, so that the main loop's first fetches do not start from DRAM.
        const size_t w_pitch = PACKED3 ? (size_t)p.K * 3 / 8 : (size_t)p.K / 2;
        const int rows = min(BN, p.N - n0);
        const uint8_t* wc0 = p.w_codes + (size_t)n0 * w_pitch;
        const size_t wbytes = (size_t)rows * w_pitch;
        if (((reinterpret_cast<uintptr_t>(wc0) | wbytes) & 15) == 0)
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" :: "l"(wc0), "r"((uint32_t)wbytes) : "memory");
        const float* lv0 = p.levels + (size_t)n0 * (p.K / p.G) * NLEV;
        const size_t lbytes = (size_t)rows * (p.K / p.G) * NLEV * sizeof(float);
        if (((reinterpret_cast<uintptr_t>(lv0) | lbytes) & 15) == 0)
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" :: "l"(lv0), "r"((uint32_t)lbytes) : "memory");
    }
    lrq_pdl_wait();                      // the activation codes are the previous kernel's output

    if (warp < WORKERS / 32) {
        // ------------------------------ workers: fetch, expand / decode, then the epilogue ------------------------------
        const int t = threadIdx.x;                         // 0..255
        const int ar = t & 127, ah = t >> 7;               // A: token row of the tile, which half of its 64 codes
        const int m = min(m0 + ar, p.M - 1);               // rows past M fetch a valid row; never stored
        constexpr int A_HALF = BK * A_BITS / 16;           // 32 or 16 code bytes per thread and k-block
        const uint8_t* arow = p.a_codes + (size_t)m * ((size_t)p.K * A_BITS / 8) + ah * A_HALF;
        // B: one group of eight codes per thread: (row, group) = (t >> 3, t & 7)
        const int wr = t >> 3, wc = t & 7;
        const int ngrp = p.K / p.G, kb_per_grp = p.G / BK;
        const size_t w_pitch = PACKED3 ? (size_t)p.K * 3 / 8 : (size_t)p.K / 2;
        const uint8_t* w_end = p.w_codes + (size_t)p.N * w_pitch;
        const int n = min(n0 + wr, p.N - 1);               // rows past N decode a valid row; never stored
        const uint8_t* wrow = p.w_codes + (size_t)n * w_pitch + (PACKED3 ? 3 * wc : 4 * wc);
        const float* tab = p.levels + (size_t)n * ngrp * NLEV;
        Lut L;
        load_lut<W_BITS>(L, tab);                           // the first table, requested before anything else
        int next_switch = kb_per_grp;                       // k-block at which the next group's table starts
        // per-token terms of the epilogue: rows of this thread's TMEM lane quadrant
        const int er = (warp & 3) * 32 + lane, em = m0 + er;
        const float sm = em < p.M ? __ldg(p.a_scale + em) : 0.f;
        const float zm = em < p.M ? (float)__ldg(p.a_zp + em) + (A_BITS == 8 ? 128.f : 8.f) : 0.f;
        uint32_t offA[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) offA[c] = swz(ar, 4 * ah + c);
        const uint32_t offB = swz(wr, wc);
        auto fetch_w = [&](int kb) -> uint32_t {
            if (!PACKED3) return __ldg(reinterpret_cast<const uint32_t*>(wrow + (size_t)kb * (BK / 2)));
            // three bytes at any offset: the 32-bit window that starts there, from the two aligned words around it
            const uint8_t* a = wrow + (size_t)kb * (BK * 3 / 8);
            const uintptr_t ai = reinterpret_cast<uintptr_t>(a);
            const uint32_t* w0 = reinterpret_cast<const uint32_t*>(ai & ~uintptr_t(3));
            const uint32_t lo = __ldg(w0);
            const uint32_t hi = (reinterpret_cast<const uint8_t*>(w0 + 2) <= w_end) ? __ldg(w0 + 1) : 0u;   // never past the code matrix
            return __funnelshift_r(lo, hi, 8 * (uint32_t)(ai & 3)) & 0x00FFFFFFu;
        };
        // Register ring: the codes of the next DEPTH k-blocks are in flight while one is decoded.  With a cold L2 a
        // fetch takes about a microsecond and a k-block a fifth of that, so one block of look-ahead would leave the
        // kernel waiting on DRAM latency at every step.
        constexpr int DEPTH = 4;
        uint4 araw[DEPTH][A_HALF / 16];
        uint32_t wraw[DEPTH];
        auto fetch = [&](int slot, int kb) {
#pragma unroll
            for (int i = 0; i < A_HALF / 16; ++i) araw[slot][i] = __ldg(reinterpret_cast<const uint4*>(arow + (size_t)kb * (2 * A_HALF)) + i);
            wraw[slot] = fetch_w(kb);
        };
#pragma unroll
        for (int d = 0; d < DEPTH; ++d)
            if (d < kblocks) fetch(d, d);
        bool ok = true;
        for (int kb0 = 0; kb0 < kblocks && ok; kb0 += DEPTH) {
#pragma unroll
            for (int d = 0; d < DEPTH; ++d) {
                const int kb = kb0 + d;
                if (kb >= kblocks) break;
                const int s = kb % NSTG;
                uint4 a_now[A_HALF / 16];
#pragma unroll
                for (int i = 0; i < A_HALF / 16; ++i) a_now[i] = araw[d][i];
                const uint32_t w_now = wraw[d];
                if (kb + DEPTH < kblocks) fetch(d, kb + DEPTH);
                if (kb >= next_switch) {                       // grouped tables: the next group's
                    load_lut<W_BITS>(L, tab + (size_t)(kb / kb_per_grp) * NLEV);
                    next_switch += kb_per_grp;
                }
                ok = mbar_wait_warp<0>(smem_u32(&ctl->empty[s]), ((kb / NSTG) & 1) ^ 1, &ctl->abort_flag, p.status, 31);
                if (!ok) break;
                const uint32_t dA = smem_u32(sA + s * A_STAGE), dB = smem_u32(sB + s * B_STAGE);
                if (A_BITS == 4) {
                    const uint32_t w[4] = {a_now[0].x, a_now[0].y, a_now[0].z, a_now[0].w};
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t o[4];
                        expand_a4(w[c], o);
                        sts128(dA + offA[c], o[0], o[1], o[2], o[3]);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {             // eight codes = two words per 16-byte chunk
                        const uint4 v = a_now[(c >> 1) % (A_HALF / 16)];
                        const uint32_t w0 = (c & 1) ? v.z : v.x, w1 = (c & 1) ? v.w : v.y;
                        uint32_t o[4];
                        expand_a8(w0, o[0], o[1]);
                        expand_a8(w1, o[2], o[3]);
                        sts128(dA + offA[c], o[0], o[1], o[2], o[3]);
                    }
                }
                {
                    uint32_t o[4];
                    decode_w<W_BITS, A_BITS == 4>(PACKED3 ? spread3(w_now) : w_now, L, o);
                    sts128(dB + offB, o[0], o[1], o[2], o[3]);
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->full[s]));
            }
        }
        // ------------------------------ epilogue: one token row per thread, 16 of the 32 columns ------------------------------
        asm volatile("bar.sync 1, %0;" :: "n"(NUM_THREADS) : "memory");       // the per-channel terms are in shared memory
        if (ok) ok = mbar_wait_warp<0>(smem_u32(&ctl->acc_full), 0, &ctl->abort_flag, p.status, 33);
        tc_fence_after();
        if (ok) {
            const int c0 = (warp >> 2) * 16;                  // warps 0-3: columns 0-15, warps 4-7: columns 16-31
            uint32_t acc[16];
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                : "=r"(acc[0]), "=r"(acc[1]), "=r"(acc[2]), "=r"(acc[3]), "=r"(acc[4]), "=r"(acc[5]), "=r"(acc[6]), "=r"(acc[7]),
                  "=r"(acc[8]), "=r"(acc[9]), "=r"(acc[10]), "=r"(acc[11]), "=r"(acc[12]), "=r"(acc[13]), "=r"(acc[14]), "=r"(acc[15])
                : "r"(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)c0) : "memory");
            tc_wait_ld();
            if (em < p.M) {
                float y[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    float v = sm * fmaf(zm, ctl->col[0][c0 + j], __uint_as_float(acc[j]));
                    if (p.wscale) v *= ctl->col[1][c0 + j];
                    if (p.bias) v += ctl->col[2][c0 + j];
                    y[j] = v;
                }
                const int nb = n0 + c0;
                if (p.y_dtype == LRQ_F32) {
                    float* dst = static_cast<float*>(p.Y) + (size_t)em * p.ldy + nb;
                    if (nb + 16 <= p.N) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) reinterpret_cast<float4*>(dst)[j] = make_float4(y[4 * j], y[4 * j + 1], y[4 * j + 2], y[4 * j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) if (nb + j < p.N) dst[j] = y[j];
                    }
                } else {
                    uint16_t* dst = static_cast<uint16_t*>(p.Y) + (size_t)em * p.ldy + nb;
                    uint32_t h[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (p.y_dtype == LRQ_BF16) { __nv_bfloat162 v = __floats2bfloat162_rn(y[2 * j], y[2 * j + 1]); h[j] = *reinterpret_cast<uint32_t*>(&v); }
                        else { __half2 v = __floats2half2_rn(y[2 * j], y[2 * j + 1]); h[j] = *reinterpret_cast<uint32_t*>(&v); }
                    }
                    if (nb + 16 <= p.N) {
                        reinterpret_cast<uint4*>(dst)[0] = make_uint4(h[0], h[1], h[2], h[3]);
                        reinterpret_cast<uint4*>(dst)[1] = make_uint4(h[4], h[5], h[6], h[7]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) if (nb + j < p.N) dst[j] = (uint16_t)(h[j >> 1] >> (16 * (j & 1)));
                    }
                }
            }
        }
    } else {
        // ------------------------------ per-channel epilogue terms, then the MMA issuer ------------------------------
        {
            const int n = n0 + lane;
            const bool okc = n < p.N;
            ctl->col[0][lane] = okc ? __ldg(p.wsum + n) : 0.f;
            ctl->col[1][lane] = (okc && p.wscale) ? __ldg(p.wscale + n) : 1.f;
            ctl->col[2][lane] = (okc && p.bias) ? __ldg(p.bias + n) : 0.f;
            // published to the workers, who take the same named barrier (id 1) before their epilogue
            asm volatile("bar.arrive 1, %0;" :: "n"(NUM_THREADS) : "memory");
        }
        bool ok = true;
        if (lane == 0) {
        for (int kb = 0; kb < kblocks && ok; ++kb) {
            const int s = kb % NSTG;
            ok = mbar_wait<0>(smem_u32(&ctl->full[s]), (kb / NSTG) & 1, &ctl->abort_flag, p.status, 32);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_addr = smem_u32(sA + s * A_STAGE), b_addr = smem_u32(sB + s * B_STAGE);
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)
                tc_mma_f16(tmem_base, umma_desc_sw128(a_addr + k * 32, 16, 1024), umma_desc_sw128(b_addr + k * 32, 16, 1024), IDESC,
                           (kb | k) ? 1u : 0u);
            tc_commit(smem_u32(&ctl->empty[s]));
        }
        if (ok) tc_commit(smem_u32(&ctl->acc_full));
        }
        __syncwarp();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == WORKERS / 32) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <int A_BITS, int W_BITS, bool PACKED3>
lrq_status launch(const Params& p, cudaStream_t st) {
    auto kern = qgemm_small_kernel<A_BITS, W_BITS, PACKED3>;
    static std::mutex mu;
    static bool configured[LRQ_MAX_DEVICES] = {};
    int dev = 0;
    if (lrq_current_device(&dev, nullptr) != LRQ_OK) return LRQ_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!configured[dev]) {
            LRQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
            configured[dev] = true;
        }
    }
    const dim3 grid((p.N + BN - 1) / BN, (p.M + BM - 1) / BM);
    LRQ_CUDA_TRY(lrq_launch_pdl(kern, grid, dim3(NUM_THREADS), SMEM_BYTES, st, p));
    return LRQ_OK;
}

}  // namespace

bool lrq_qgemm_small_takes(const lrq_layer* L) {
    if (L->K % BK || L->group % BK) return false;
    if (L->w_bits < 3 || L->w_bits > 4) return false;
    if (L->packed3 && L->w_bits != 3) return false;
    return lrq_aligned(L->levels, 16) && lrq_aligned(L->codes, 4);
}

lrq_status lrq_launch_qgemm_small(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale, const int32_t* a_zp, int M,
                                  void* Y, lrq_dtype dt, long ldy, cudaStream_t st) {
    if (!lrq_qgemm_small_takes(L) || !lrq_aligned(a_codes, 16)) return LRQ_ERR_UNSUPPORTED;
    const size_t es = dt == LRQ_F32 ? 4 : 2;
    if (!lrq_aligned(Y, 16) || ((size_t)ldy * es) % 16) return LRQ_ERR_UNSUPPORTED;
    Params p;
    p.a_codes = a_codes; p.a_scale = a_scale; p.a_zp = a_zp;
    p.w_codes = L->codes; p.levels = L->levels; p.wsum = L->wsum; p.wscale = L->wscale; p.bias = L->bias;
    p.Y = Y; p.ldy = ldy; p.M = M; p.N = L->N; p.K = L->K; p.G = L->group; p.y_dtype = (int)dt;
    p.status = lrq_status_word();
    const int ab = L->act.a_bits;
    if (L->packed3) return ab == 8 ? launch<8, 3, true>(p, st) : launch<4, 3, true>(p, st);
    if (L->w_bits == 3) return ab == 8 ? launch<8, 3, false>(p, st) : launch<4, 3, false>(p, st);
    return ab == 8 ? launch<8, 4, false>(p, st) : launch<4, 4, false>(p, st);
}
