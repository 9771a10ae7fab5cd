// Quantized contraction + epilogue on the 5th-generation tensor cores (Sec. 4.1, Eq. 10).
//
//   acc[m,n] = sum_k q[m,k] * T[n, k/G, u[n,k]]          exact bf16 products, fp32 accumulation in TMEM
//   Y[m,n]   = s_m * (acc + z_m * wsum_n) * wscale_n + bias_n
//
// Every level II * 2^(f-7) of Eqs. 8-9 has an 8-bit significand and every activation code is an
// integer below 256, so both operands are exactly bf16 numbers; products are exact and only the
// fp32 accumulation order differs from the fp64 definition.
//
// One persistent CTA per SM walks over 128 x 256 output tiles.  Warp roles:
//   warps 0-3   expand activation codes of the tile's 128 tokens into the bf16 A stage
//   warps 4-11  decode TLQ codes of the tile's 256 output channels through the row's level table
//               (held in registers as two byte planes, looked up with byte permutes) into the B stage
//   warps 12-15 epilogue: tcgen05.ld the finished accumulator, scale, store
//   warp  16    allocates TMEM and issues tcgen05.mma (one elected lane)
// The A/B stages use the canonical K-major 128-byte-swizzled layout that the UMMA shared-memory
// descriptor expects; they are written with ordinary shared stores, published to the async proxy
// with fence.proxy.async and handed over through mbarriers.  The accumulator is double-buffered in
// TMEM (2 x 256 columns) so that the epilogue of one tile overlaps the main loop of the next.
// Every wait is bounded: when one expires the CTA records a code in the status word, stops waiting
// and runs to its end (TMEM is always freed).
//
// To keep the expansion cheap the A operand carries a constant offset that the epilogue removes:
// 8-bit codes are fed as q - 128, 4-bit codes as q - 8 (the zero-point term absorbs it); centring
// also keeps the accumulator free of a large common-mode term.
#include "lrq_internal.cuh"

namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int STAGES = 4;
constexpr int A_STAGE_BYTES = BM * BK * 2;   // 16 KB
constexpr int B_STAGE_BYTES = BN * BK * 2;   // 32 KB
constexpr int NUM_A_WARPS = 4, NUM_B_WARPS = 8, NUM_EPI_WARPS = 4;
constexpr int EPI_WARP0 = NUM_A_WARPS + NUM_B_WARPS;          // 12 (a multiple of 4: TMEM lane quadrants line up)
constexpr int MMA_WARP = EPI_WARP0 + NUM_EPI_WARPS;           // 16
constexpr int NUM_THREADS = (MMA_WARP + 1) * 32;              // 544
constexpr int TMEM_COLS = 512;
constexpr uint32_t WAIT_LIMIT = 1u << 22;

struct __align__(8) SharedCtl {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
    float col[2][3][BN];          // per TMEM buffer: wsum, wscale, bias of the tile's columns
};

constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + sizeof(SharedCtl);

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and raises the CTA's abort flag) if the phase never completed.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, SharedCtl* ctl, int* status, int code) {
    for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (ctl->abort_flag) return false;
    }
    ctl->abort_flag = 1;
    if (status) atomicCAS(status, 0, code);
    return false;
}

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// UMMA shared-memory descriptor: K-major operand, 128-byte swizzle, rows of 64 bf16 (128 B), groups of
// 8 rows 1024 B apart.  Bits: [0,14) address>>4, [16,30) leading offset>>4 (unused for this layout),
// [32,46) stride offset>>4, [46,48) descriptor version 1, [61,64) layout type 2 (128B swizzle).
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulator (bits 4-5 = 1), A and B bf16 (bits 7-9, 10-12 = 1),
// both K-major (bits 15, 16 = 0), N>>3 at bits 17-22, M>>4 at bits 24-28.
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

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

// Byte offset of 16-byte chunk `c` (0..7) of row `r` in a K-major 128B-swizzled stage.
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4)); }

// ---- activation codes -> bf16 ---------------------------------------------------------------------
// 8-bit: four codes per word -> bf16 of (q - 128).  0x4300|x7 is 128 + x7; adding -256 (bit 7 clear)
// or -128 (bit 7 set) gives q - 128 exactly.
__device__ __forceinline__ void expand_a8(uint32_t w, uint32_t& o01, uint32_t& o23) {
    const uint32_t p01 = prmt(w, 0u, 0x4140u), p23 = prmt(w, 0u, 0x4342u);
    o01 = add_bf16x2((p01 & 0x007F007Fu) | 0x43004300u, (p01 & 0x00800080u) ^ 0xC380C380u);
    o23 = add_bf16x2((p23 & 0x007F007Fu) | 0x43004300u, (p23 & 0x00800080u) ^ 0xC380C380u);
}
// 4-bit: eight codes per word -> bf16 of (q - 8): 0x4300 | q is 128 + q, and 128 + q - 136 is exact.
__device__ __forceinline__ void expand_a4(uint32_t w, uint32_t* o) {
    const uint32_t lo = w & 0x0F0F0F0Fu, hi = (w >> 4) & 0x0F0F0F0Fu;      // even / odd codes, one per byte
    // bytes below 16 have a clear top bit: selector 8|k yields 0x00
    o[0] = add_bf16x2(prmt(lo, hi, 0x8480u) | 0x43004300u, 0xC308C308u);
    o[1] = add_bf16x2(prmt(lo, hi, 0x8581u) | 0x43004300u, 0xC308C308u);
    o[2] = add_bf16x2(prmt(lo, hi, 0x8682u) | 0x43004300u, 0xC308C308u);
    o[3] = add_bf16x2(prmt(lo, hi, 0x8783u) | 0x43004300u, 0xC308C308u);
}

// ---- TLQ codes -> bf16 through the row's level table ------------------------------------------------
// The table is kept as two byte planes (low and high byte of each bf16 entry), 16 entries = 4 + 4 registers.
struct Lut { uint32_t lo[4], hi[4]; };

template <int W_BITS>
__device__ __forceinline__ void load_lut(Lut& L, const float* __restrict__ tab) {
    constexpr int NL = 1 << W_BITS;
    uint32_t e[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) e[i] = 0;
#pragma unroll
    for (int i = 0; i < NL / 4; ++i) {
        const float4 v = *reinterpret_cast<const float4*>(tab + 4 * i);
        e[4 * i] = __float_as_uint(v.x) >> 16; e[4 * i + 1] = __float_as_uint(v.y) >> 16;   // levels are exact bf16 numbers
        e[4 * i + 2] = __float_as_uint(v.z) >> 16; e[4 * i + 3] = __float_as_uint(v.w) >> 16;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        L.lo[j] = (e[4 * j] & 0xFF) | ((e[4 * j + 1] & 0xFF) << 8) | ((e[4 * j + 2] & 0xFF) << 16) | ((e[4 * j + 3] & 0xFF) << 24);
        L.hi[j] = (e[4 * j] >> 8) | ((e[4 * j + 1] >> 8) << 8) | ((e[4 * j + 2] >> 8) << 16) | ((e[4 * j + 3] >> 8) << 24);
    }
}

// eight codes (one word) -> four registers of two bf16 each, in k order
template <int W_BITS>
__device__ __forceinline__ void decode_w(uint32_t w, const Lut& L, uint32_t* o) {
    if (W_BITS == 4) {
        const uint32_t selA = w & 0x77777777u, selB = selA >> 16;
        const uint32_t x0 = w << 4;
        const uint32_t mA = prmt(x0, w, 0xD9C8u), mB = prmt(x0, w, 0xFBEAu);    // 0xFF where the code's top bit is set
        const uint32_t loA = (prmt(L.lo[0], L.lo[1], selA) & ~mA) | (prmt(L.lo[2], L.lo[3], selA) & mA);
        const uint32_t hiA = (prmt(L.hi[0], L.hi[1], selA) & ~mA) | (prmt(L.hi[2], L.hi[3], selA) & mA);
        const uint32_t loB = (prmt(L.lo[0], L.lo[1], selB) & ~mB) | (prmt(L.lo[2], L.lo[3], selB) & mB);
        const uint32_t hiB = (prmt(L.hi[0], L.hi[1], selB) & ~mB) | (prmt(L.hi[2], L.hi[3], selB) & mB);
        o[0] = prmt(loA, hiA, 0x5140u); o[1] = prmt(loA, hiA, 0x7362u);
        o[2] = prmt(loB, hiB, 0x5140u); o[3] = prmt(loB, hiB, 0x7362u);
    } else {                                   // at most 8 table entries: one permute per plane
        const uint32_t selA = w & 0x77777777u, selB = selA >> 16;
        const uint32_t loA = prmt(L.lo[0], L.lo[1], selA), hiA = prmt(L.hi[0], L.hi[1], selA);
        const uint32_t loB = prmt(L.lo[0], L.lo[1], selB), hiB = prmt(L.hi[0], L.hi[1], selB);
        o[0] = prmt(loA, hiA, 0x5140u); o[1] = prmt(loA, hiA, 0x7362u);
        o[2] = prmt(loB, hiB, 0x5140u); o[3] = prmt(loB, hiB, 0x7362u);
    }
}

__device__ __forceinline__ void sts128(unsigned char* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    *reinterpret_cast<uint4*>(p) = make_uint4(a, b, c, d);
}

struct Params {
    const uint8_t* a_codes; const float* a_scale; const int32_t* a_zp;
    const uint8_t* w_codes; const float* levels; const float* wsum; const float* wscale; const float* bias;
    void* Y; long ldy; int M, N, K, G, y_dtype; int* status;
};

template <int A_BITS, int W_BITS>
__global__ void __launch_bounds__(NUM_THREADS, 1)
qgemm_tc_kernel(const Params p) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    unsigned char* sA = base;                                   // STAGES x 16 KB
    unsigned char* sB = base + STAGES * A_STAGE_BYTES;          // STAGES x 32 KB
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(sB + STAGES * B_STAGE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (p.M + BM - 1) / BM, tiles_n = (p.N + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int kblocks = p.K / BK;
    constexpr int NLEV = 1 << W_BITS;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), NUM_A_WARPS + NUM_B_WARPS);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[b]), NUM_EPI_WARPS);
        }
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == MMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp < NUM_A_WARPS) {
        // =============================== A producers: one token row per thread ===============================
        const int r = threadIdx.x;                                // 0..127
        constexpr int ROW_BYTES = BK * A_BITS / 8;                // 64 (8-bit) or 32 (4-bit) code bytes per k-block
        constexpr int NV = ROW_BYTES / 16;
        uint32_t it = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
            const int m0 = (tile % tiles_m) * BM;
            const int m = min(m0 + r, p.M - 1);                   // rows past M read a valid row; never stored
            const uint4* src = reinterpret_cast<const uint4*>(p.a_codes + (size_t)m * ((size_t)p.K * A_BITS / 8));
            uint4 cur[NV];
#pragma unroll
            for (int i = 0; i < NV; ++i) cur[i] = __ldg(src + i);
            for (int kb = 0; kb < kblocks; ++kb, ++it) {
                uint4 nxt[NV];
                if (kb + 1 < kblocks) {
#pragma unroll
                    for (int i = 0; i < NV; ++i) nxt[i] = __ldg(src + (size_t)(kb + 1) * NV + i);
                }
                const int s = it % STAGES;
                if (!mbar_wait(smem_u32(&ctl->empty[s]), ((it / STAGES) & 1) ^ 1, ctl, p.status, 1)) break;
                unsigned char* dst = sA + s * A_STAGE_BYTES;
                if (A_BITS == 8) {
#pragma unroll
                    for (int i = 0; i < NV; ++i) {                // 16 codes -> two 16-byte chunks
                        uint32_t o[8];
                        expand_a8(cur[i].x, o[0], o[1]); expand_a8(cur[i].y, o[2], o[3]);
                        expand_a8(cur[i].z, o[4], o[5]); expand_a8(cur[i].w, o[6], o[7]);
                        sts128(dst + swz(r, 2 * i), o[0], o[1], o[2], o[3]);
                        sts128(dst + swz(r, 2 * i + 1), o[4], o[5], o[6], o[7]);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < NV; ++i) {                // 32 codes -> four chunks
                        uint32_t o[4];
                        expand_a4(cur[i].x, o); sts128(dst + swz(r, 4 * i), o[0], o[1], o[2], o[3]);
                        expand_a4(cur[i].y, o); sts128(dst + swz(r, 4 * i + 1), o[0], o[1], o[2], o[3]);
                        expand_a4(cur[i].z, o); sts128(dst + swz(r, 4 * i + 2), o[0], o[1], o[2], o[3]);
                        expand_a4(cur[i].w, o); sts128(dst + swz(r, 4 * i + 3), o[0], o[1], o[2], o[3]);
                    }
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->full[s]));
#pragma unroll
                for (int i = 0; i < NV; ++i) cur[i] = nxt[i];
            }
            if (ctl->abort_flag) break;
        }
    } else if (warp < EPI_WARP0) {
        // =============================== B producers: one output channel per thread ==========================
        const int r = threadIdx.x - NUM_A_WARPS * 32;             // 0..255
        const int ngrp = p.K / p.G, kb_per_grp = p.G / BK;
        uint32_t it = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
            const int n0 = (tile / tiles_m) * BN;
            const int n = min(n0 + r, p.N - 1);
            const uint4* src = reinterpret_cast<const uint4*>(p.w_codes + (size_t)n * (p.K / 2));
            const float* tab = p.levels + (size_t)n * ngrp * NLEV;
            Lut L;
            uint4 cur[2];
            cur[0] = __ldg(src); cur[1] = __ldg(src + 1);
            for (int kb = 0; kb < kblocks; ++kb, ++it) {
                uint4 nxt[2];
                if (kb + 1 < kblocks) { nxt[0] = __ldg(src + 2 * (kb + 1)); nxt[1] = __ldg(src + 2 * (kb + 1) + 1); }
                if (kb % kb_per_grp == 0) load_lut<W_BITS>(L, tab + (size_t)(kb / kb_per_grp) * NLEV);
                const int s = it % STAGES;
                if (!mbar_wait(smem_u32(&ctl->empty[s]), ((it / STAGES) & 1) ^ 1, ctl, p.status, 2)) break;
                unsigned char* dst = sB + s * B_STAGE_BYTES;
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    uint32_t o[4];
                    decode_w<W_BITS>(cur[i].x, L, o); sts128(dst + swz(r, 4 * i), o[0], o[1], o[2], o[3]);
                    decode_w<W_BITS>(cur[i].y, L, o); sts128(dst + swz(r, 4 * i + 1), o[0], o[1], o[2], o[3]);
                    decode_w<W_BITS>(cur[i].z, L, o); sts128(dst + swz(r, 4 * i + 2), o[0], o[1], o[2], o[3]);
                    decode_w<W_BITS>(cur[i].w, L, o); sts128(dst + swz(r, 4 * i + 3), o[0], o[1], o[2], o[3]);
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->full[s]));
                cur[0] = nxt[0]; cur[1] = nxt[1];
            }
            if (ctl->abort_flag) break;
        }
    } else if (warp < MMA_WARP) {
        // =============================== epilogue: TMEM -> registers -> global ===============================
        const int ew = warp - EPI_WARP0;                           // TMEM lane quadrant
        const int et = threadIdx.x - EPI_WARP0 * 32;               // 0..127 = accumulator row
        const float zoff = (A_BITS == 8) ? 128.f : 8.f;      // the A operand is fed as q - 128 / q - 8
        uint32_t t = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++t) {
            const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
            const int buf = t & 1;
            // stage the tile's per-column terms (wsum, wscale, bias) in shared memory
            float (*col)[BN] = ctl->col[buf];
            for (int c = et; c < BN; c += NUM_EPI_WARPS * 32) {
                const int n = n0 + c;
                const bool ok = n < p.N;
                col[0][c] = ok ? __ldg(p.wsum + n) : 0.f;
                col[1][c] = (ok && p.wscale) ? __ldg(p.wscale + n) : 1.f;
                col[2][c] = (ok && p.bias) ? __ldg(p.bias + n) : 0.f;
            }
            asm volatile("bar.sync 1, %0;" ::"n"(NUM_EPI_WARPS * 32) : "memory");
            const int m = m0 + et;
            const bool row_ok = m < p.M;
            const float sm = row_ok ? __ldg(p.a_scale + m) : 0.f;
            const float zm = row_ok ? (float)__ldg(p.a_zp + m) + zoff : 0.f;
            const bool okw = mbar_wait(smem_u32(&ctl->tmem_full[buf]), (t >> 1) & 1, ctl, p.status, 3);
            tc_fence_after();
            if (okw) {
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    if (n0 + c0 >= p.N) break;                     // warp-uniform
                    uint32_t acc[32];
                    tc_ld32(tmem_base + ((uint32_t)(ew * 32) << 16) + (uint32_t)(buf * BN + c0), acc);
                    tc_wait_ld();
                    if (row_ok) {
                        float y[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            y[j] = fmaf(sm * fmaf(zm, col[0][c0 + j], __uint_as_float(acc[j])), col[1][c0 + j], col[2][c0 + j]);
                        const int nvalid = min(32, p.N - (n0 + c0));
                        if (p.y_dtype == LRQ_F32) {
                            float* dst = static_cast<float*>(p.Y) + (size_t)m * p.ldy + n0 + c0;
                            if (nvalid == 32) {
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    reinterpret_cast<float4*>(dst)[j] = make_float4(y[4 * j], y[4 * j + 1], y[4 * j + 2], y[4 * j + 3]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j) if (j < nvalid) dst[j] = y[j];
                            }
                        } else {
                            uint32_t h[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                if (p.y_dtype == LRQ_BF16) {
                                    __nv_bfloat162 v = __floats2bfloat162_rn(y[2 * j], y[2 * j + 1]);
                                    h[j] = *reinterpret_cast<uint32_t*>(&v);
                                } else {
                                    __half2 v = __floats2half2_rn(y[2 * j], y[2 * j + 1]);
                                    h[j] = *reinterpret_cast<uint32_t*>(&v);
                                }
                            }
                            uint16_t* dst = static_cast<uint16_t*>(p.Y) + (size_t)m * p.ldy + n0 + c0;
                            if (nvalid == 32) {
#pragma unroll
                                for (int j = 0; j < 4; ++j)
                                    reinterpret_cast<uint4*>(dst)[j] = make_uint4(h[4 * j], h[4 * j + 1], h[4 * j + 2], h[4 * j + 3]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j) if (j < nvalid) dst[j] = (uint16_t)(h[j >> 1] >> (16 * (j & 1)));
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[buf]));
            if (ctl->abort_flag) break;
        }
    } else {
        // =============================== MMA issuer ==========================================================
        if (lane == 0) {
            uint32_t it = 0, t = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++t) {
                const int buf = t & 1;
                ok = mbar_wait(smem_u32(&ctl->tmem_empty[buf]), ((t >> 1) & 1) ^ 1, ctl, p.status, 4);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % STAGES;
                    ok = mbar_wait(smem_u32(&ctl->full[s]), (it / STAGES) & 1, ctl, p.status, 5);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(sA + s * A_STAGE_BYTES), b_addr = smem_u32(sB + s * B_STAGE_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        tc_mma_bf16(d_tmem, make_desc(a_addr + k * 32), make_desc(b_addr + k * 32), IDESC, (kb | k) ? 1u : 0u);
                    tc_commit(smem_u32(&ctl->empty[s]));            // stage reusable once these MMAs have read it
                }
                if (ok) tc_commit(smem_u32(&ctl->tmem_full[buf]));  // accumulator complete
            }
        }
        __syncwarp();
    }

    // teardown: every role has left its loop; nothing is waiting any more
    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

template <int A_BITS, int W_BITS>
lrq_status launch(const Params& p, int grid, cudaStream_t st) {
    auto kern = qgemm_tc_kernel<A_BITS, W_BITS>;
    static bool configured = false;
    if (!configured) {
        LRQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
        configured = true;
    }
    kern<<<grid, NUM_THREADS, SMEM_BYTES, st>>>(p);
    LRQ_CUDA_TRY(cudaGetLastError());
    return LRQ_OK;
}

}  // namespace

lrq_status lrq_launch_qgemm_tc(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale,
                               const int32_t* a_zp, int M, void* Y, lrq_dtype dt, long ldy, cudaStream_t st) {
    // shapes this kernel takes: whole 64-wide k-blocks that never straddle a TLQ group; 16-byte code rows
    if (L->K % BK || L->group % BK) return LRQ_ERR_UNSUPPORTED;
    if (L->w_bits < 3 || L->w_bits > 4) return LRQ_ERR_UNSUPPORTED;   // 2-bit tables take the CUDA-core kernel
    if (!lrq_aligned(L->levels, 16) || !lrq_aligned(L->codes, 16)) return LRQ_ERR_UNSUPPORTED;
    const size_t es = dt == LRQ_F32 ? 4 : 2;
    if (!lrq_aligned(Y, 16) || ((size_t)ldy * es) % 16) return LRQ_ERR_UNSUPPORTED;
    int dev = 0, sms = 0;
    LRQ_CUDA_TRY(cudaGetDevice(&dev));
    LRQ_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    Params p;
    p.a_codes = a_codes; p.a_scale = a_scale; p.a_zp = a_zp;
    p.w_codes = L->codes; p.levels = L->levels; p.wsum = L->wsum; p.wscale = L->wscale; p.bias = L->bias;
    p.Y = Y; p.ldy = ldy; p.M = M; p.N = L->N; p.K = L->K; p.G = L->group; p.y_dtype = (int)dt;
    p.status = lrq_status_word();
    const int tiles = ((M + BM - 1) / BM) * ((L->N + BN - 1) / BN);
    const int grid = tiles < sms ? tiles : sms;
    const int ab = L->act.a_bits;
    if (ab == 8 && L->w_bits == 4) return launch<8, 4>(p, grid, st);
    if (ab == 8) return launch<8, 3>(p, grid, st);
    if (ab == 4 && L->w_bits == 4) return launch<4, 4>(p, grid, st);
    return launch<4, 3>(p, grid, st);
}
