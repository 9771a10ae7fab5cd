// Quantized contraction + epilogue on the 5th-generation tensor cores (Sec. 4.1, Eq. 10).
//
//   acc[m,n] = sum_k q[m,k] * T[n, k/G, u[n,k]]          exact bf16 products, fp32 accumulation in TMEM
//   Y[m,n]   = s_m * (acc + z_m * wsum_n) * wscale_n + bias_n
//
// Every level II * 2^(f-7) of Eqs. 8-9 has an 8-bit significand and every activation code is an
// integer below 256, so both operands are exactly bf16 numbers; products are exact and only the
// fp32 accumulation order differs from the fp64 definition.
//
// The decode of both operands runs on the integer ALUs and is what bounds the kernel, so the tile is
// shaped to decode each element as rarely as possible: a pair of CTAs (a cluster of two, cta_group::2)
// owns a 256 x 256 output tile.  Each CTA decodes its own 128 token rows of A and only its own 128 of
// the 256 weight rows of B; the tensor core reads the other half from the peer's shared memory.
// Per CTA (18 warps):
//   warp 0       one lane streams the packed code tiles (128 rows x 64 codes of each operand per k-block)
//                into shared memory with TMA, CSTAGES deep
//   warp 1       allocates TMEM; in the even CTA one lane issues tcgen05.mma (M = 256, N = 256, K = 16)
//   warps 2-9    decode TLQ weight codes through the row's level table (held in registers as two byte
//                planes, looked up with byte permutes) into the bf16 B stage
//   warps 10-13  expand activation codes into the bf16 A stage
//                (the decode warps work as two groups on alternate k-blocks: fewer, longer steps per warp,
//                and one group's barrier latencies hide behind the other's arithmetic)
//   warps 14-17  epilogue: tcgen05.ld the finished accumulator, scale, store
// The bf16 stages use the canonical K-major 128-byte-swizzled UMMA layout; they are written with
// ordinary shared stores, published to the async proxy with fence.proxy.async and handed to the MMA
// thread of the even CTA through an mbarrier there (the odd CTA's warps arrive on it remotely, with
// CTA-scope release: their data already sits, proxy-fenced, in their own shared memory by then).  Stage release and
// accumulator completion come back to both CTAs through multicast tcgen05.commit.  The accumulator is
// double-buffered in TMEM (2 x 256 columns) so that the epilogue of one tile overlaps the main loop of
// the next.  Every wait is bounded: when one expires the CTA records a code in the status word, stops
// waiting, lets its TMA loads land, and both CTAs meet at the final cluster barrier (TMEM is always freed).
//
// The A operand carries a constant offset that the epilogue removes: 8-bit codes are fed as q - 128,
// 4-bit codes as q - 8 (the zero-point term absorbs it); centring keeps the expansion cheap and the
// accumulator free of a large common-mode term.
#include "lrq_internal.cuh"
#include "tc_ptx.cuh"
#include "f32x2.cuh"
#include "tma_host.cuh"
#include <mutex>

namespace {
using namespace lrq_tc;

constexpr int BM_CTA = 128;                  // token rows per CTA; the pair's tile has 256
constexpr int BN = 256;                      // output channels per tile (template BN_T: 256, or 128 for small problems)
constexpr int BN_CTA = 128;                  // weight rows decoded per CTA
constexpr int BK = 64;
constexpr int STAGES = 4;                    // bf16 operand stages
constexpr int CSTAGES = 6;                   // packed-code stages: the TMA runs this many k-blocks ahead of the decode (with 32768
                                             // tokens the code tiles come from a busy L2 / DRAM: 2 stages 614, 4 stages 972, 6 stages 1038 TFLOP/s)
constexpr int A_STAGE_BYTES = BM_CTA * BK * 2;      // 16 KB
constexpr int B_STAGE_BYTES = BN_CTA * BK * 2;      // 16 KB
constexpr int AC_STAGE_BYTES = BM_CTA * BK;         // room for 8-bit codes (4-bit codes use half)
constexpr int WC_STAGE_BYTES = BN_CTA * BK / 2;     // 4 KB
constexpr int TMA_WARP = 0, MMA_WARP = 1, B_WARP0 = 2, NUM_B_WARPS = 8, A_WARP0 = 10, NUM_A_WARPS = 4;
constexpr int EPI_WARP0 = 14, NUM_EPI_WARPS = 4;
constexpr int GROUP_WARPS = (NUM_A_WARPS + NUM_B_WARPS) / 2;   // decode warps that fill one stage (two groups alternate)
constexpr int NUM_THREADS = (EPI_WARP0 + NUM_EPI_WARPS) * 32;      // 576
constexpr int TMEM_COLS = 512;

struct __align__(16) SharedCtl {
    uint64_t cfull[CSTAGES];      // code stage filled by TMA                       (local)
    uint64_t cempty[CSTAGES];     // code stage read by the group that decodes it   (local)
    uint64_t full[STAGES];        // bf16 stage written by the decode warps of both CTAs (used in the even CTA)
    uint64_t empty[STAGES];       // bf16 stage consumed by the MMAs                (each CTA, multicast commit)
    uint64_t tmem_full[2];        // accumulator complete                           (each CTA, multicast commit)
    uint64_t tmem_empty[2];       // accumulator drained by both CTAs' epilogues    (used in the even CTA)
    uint32_t tmem_base;
    volatile int abort_flag;
    alignas(16) float col[2][3][BN];   // per TMEM buffer: wsum, wscale, bias of the tile's columns (read as float4)
};

constexpr int EPI_TILE_BYTES = 32 * 32 * 4;         // one epilogue warp's 32 x 32 fp32 chunk, staged for a TMA store
constexpr int EPI_TILES = 1;                        // staging tiles per epilogue warp (a second one bought nothing; its 16 KB went to the code stages)
constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) +
                              (size_t)NUM_EPI_WARPS * EPI_TILES * EPI_TILE_BYTES +
                              (size_t)CSTAGES * (AC_STAGE_BYTES + WC_STAGE_BYTES) + sizeof(SharedCtl);
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");


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
// Constants of the expansions, held in registers: an instruction encodes at most one immediate, so a
// three-input logic operation or a byte permute with two constant operands would otherwise be split in two.
struct ExpandConst {
    uint32_t k7f, k43, k80, kc3, k4343;
    __device__ ExpandConst() {
        asm volatile("mov.u32 %0, 0x007F007F;" : "=r"(k7f));
        asm volatile("mov.u32 %0, 0x43004300;" : "=r"(k43));
        asm volatile("mov.u32 %0, 0x00800080;" : "=r"(k80));
        asm volatile("mov.u32 %0, 0xC380C380;" : "=r"(kc3));
        asm volatile("mov.u32 %0, 0x43434343;" : "=r"(k4343));
    }
};
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {     // (a & b) | c
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t and_xor(uint32_t a, uint32_t b, uint32_t c) {    // (a & b) ^ c
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// 8-bit: four codes per word -> bf16 of (q - 128).  0x4300|x7 is 128 + x7; adding -256 (bit 7 clear)
// or -128 (bit 7 set) gives q - 128 exactly.
__device__ __forceinline__ void expand_a8(uint32_t w, const ExpandConst& k, uint32_t& o01, uint32_t& o23) {
    const uint32_t p01 = prmt(w, 0u, 0x4140u), p23 = prmt(w, 0u, 0x4342u);
    o01 = add_bf16x2(and_or(p01, k.k7f, k.k43), and_xor(p01, k.k80, k.kc3));
    o23 = add_bf16x2(and_or(p23, k.k7f, k.k43), and_xor(p23, k.k80, k.kc3));
}
// 4-bit: eight codes per word -> bf16 of (q - 8): 0x4300 | q is 128 + q, and 128 + q - 136 is exact.
// The eight elements come out in the order k = 0,2, 4,6, 1,3, 5,7 within the word (one byte permute per
// pair instead of a permute and an OR); the weight decode of 4-bit-activation layers emits the same order,
// and a contraction does not care in which order k is summed as long as both operands agree.
__device__ __forceinline__ void expand_a4(uint32_t w, const ExpandConst& k, uint32_t* o) {
    const uint32_t lo = w & 0x0F0F0F0Fu, hi = (w >> 4) & 0x0F0F0F0Fu;      // even / odd codes, one per byte
    o[0] = add_bf16x2(prmt(lo, k.k4343, 0x4140u), 0xC308C308u);            // codes 0, 2
    o[1] = add_bf16x2(prmt(lo, k.k4343, 0x4342u), 0xC308C308u);            // codes 4, 6
    o[2] = add_bf16x2(prmt(hi, k.k4343, 0x4140u), 0xC308C308u);            // codes 1, 3
    o[3] = add_bf16x2(prmt(hi, k.k4343, 0x4342u), 0xC308C308u);            // codes 5, 7
}

// ---- TLQ codes -> bf16 through the row's level table ------------------------------------------------
// The table is kept as two byte planes (low and high byte of each bf16 entry), 16 entries = 4 + 4 registers.
struct Lut { uint32_t lo[4], hi[4]; };

// Levels are exact bf16 numbers stored as fp32: the upper two bytes of each word are the entry.
template <int W_BITS>
__device__ __forceinline__ void build_lut(Lut& L, const float4* raw) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (j < (1 << W_BITS) / 4) {
            const uint32_t t01 = prmt(__float_as_uint(raw[j].x), __float_as_uint(raw[j].y), 0x7632u);
            const uint32_t t23 = prmt(__float_as_uint(raw[j].z), __float_as_uint(raw[j].w), 0x7632u);
            L.lo[j] = prmt(t01, t23, 0x6420u);
            L.hi[j] = prmt(t01, t23, 0x7531u);
        } else {
            L.lo[j] = 0; L.hi[j] = 0;
        }
    }
}

// eight codes (one word) -> four registers of two bf16 each: in k order, or (A4_ORDER) in the order
// 0,2, 4,6, 1,3, 5,7 that the 4-bit activation expansion produces
template <int W_BITS, bool A4_ORDER>
__device__ __forceinline__ void decode_w(uint32_t w, const Lut& L, uint32_t* o) {
    // loA/hiA hold codes 0-3, loB/hiB codes 4-7 (one byte each); output register = two (lo, hi) byte pairs
    constexpr uint32_t S0 = A4_ORDER ? 0x6240u : 0x5140u, S1 = A4_ORDER ? 0x7351u : 0x7362u;
    if (W_BITS == 4) {
        const uint32_t selA = w & 0x77777777u, selB = selA >> 16;
        const uint32_t x0 = w << 4;
        const uint32_t mA = prmt(x0, w, 0xD9C8u), mB = prmt(x0, w, 0xFBEAu);    // 0xFF where the code's top bit is set
        const uint32_t loA = (prmt(L.lo[0], L.lo[1], selA) & ~mA) | (prmt(L.lo[2], L.lo[3], selA) & mA);
        const uint32_t hiA = (prmt(L.hi[0], L.hi[1], selA) & ~mA) | (prmt(L.hi[2], L.hi[3], selA) & mA);
        const uint32_t loB = (prmt(L.lo[0], L.lo[1], selB) & ~mB) | (prmt(L.lo[2], L.lo[3], selB) & mB);
        const uint32_t hiB = (prmt(L.hi[0], L.hi[1], selB) & ~mB) | (prmt(L.hi[2], L.hi[3], selB) & mB);
        if (A4_ORDER) { o[0] = prmt(loA, hiA, S0); o[1] = prmt(loB, hiB, S0); o[2] = prmt(loA, hiA, S1); o[3] = prmt(loB, hiB, S1); }
        else { o[0] = prmt(loA, hiA, S0); o[1] = prmt(loA, hiA, S1); o[2] = prmt(loB, hiB, S0); o[3] = prmt(loB, hiB, S1); }
    } else {                                   // at most 8 table entries: one permute per plane
        const uint32_t selA = w & 0x77777777u, selB = selA >> 16;
        const uint32_t loA = prmt(L.lo[0], L.lo[1], selA), hiA = prmt(L.hi[0], L.hi[1], selA);
        const uint32_t loB = prmt(L.lo[0], L.lo[1], selB), hiB = prmt(L.hi[0], L.hi[1], selB);
        if (A4_ORDER) { o[0] = prmt(loA, hiA, S0); o[1] = prmt(loB, hiB, S0); o[2] = prmt(loA, hiA, S1); o[3] = prmt(loB, hiB, S1); }
        else { o[0] = prmt(loA, hiA, S0); o[1] = prmt(loA, hiA, S1); o[2] = prmt(loB, hiB, S0); o[3] = prmt(loB, hiB, S1); }
    }
}

// Named barrier 1 over the epilogue warps, returning the OR of `pred` over all of them.
__device__ __forceinline__ bool bar_or_epilogue(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n.reg .pred p, q;\nsetp.ne.u32 q, %1, 0;\n"
        "bar.red.or.pred p, 1, %2, q;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(r) : "r"((uint32_t)pred), "n"(NUM_EPI_WARPS * 32) : "memory");
    return r != 0;
}

// 128-bit shared-memory accesses on 32-bit shared addresses (no 64-bit pointer arithmetic in the inner loops)
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void lds128(uint32_t addr, uint4& v) {
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
}

// Ring positions of a decode group.  A group serves every second k-block of the CTA's running count, so its
// slot in the 4-deep operand ring alternates between two values and its slot in the code ring advances by two;
// the phase bits flip when a slot index wraps.
struct RingPos {
    uint32_t s, ph, cs, cph;
    __device__ explicit RingPos(int grp) : s((uint32_t)grp), ph(0), cs((uint32_t)grp), cph(0) {}
    __device__ __forceinline__ void advance() {
        s += 2; if (s >= (uint32_t)STAGES) { s -= STAGES; ph ^= 1; }
        cs += 2; if (cs >= (uint32_t)CSTAGES) { cs -= CSTAGES; cph ^= 1; }
    }
};
static_assert(STAGES % 2 == 0 && CSTAGES % 2 == 0, "the two decode groups own alternate ring slots");

using namespace lrq_f2;

struct Params {
    const float* a_scale; const int32_t* a_zp;
    const float* levels; const float* wsum; const float* wscale; const float* bias;
    void* Y; long ldy; int M, N, K, G, y_dtype; int col_fastest; int* status;
};

template <int A_BITS, int W_BITS, int BN_T>
__global__ void __launch_bounds__(NUM_THREADS, 1)
qgemm_tc_kernel(const Params p, const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                const __grid_constant__ CUtensorMap tmY) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    unsigned char* sA = base;                                       // STAGES x 16 KB
    unsigned char* sB = sA + STAGES * A_STAGE_BYTES;                // STAGES x 16 KB
    unsigned char* sEpi = sB + STAGES * B_STAGE_BYTES;              // NUM_EPI_WARPS x EPI_TILES x 4 KB, 1024-byte aligned
    unsigned char* sAc = sEpi + NUM_EPI_WARPS * EPI_TILES * EPI_TILE_BYTES;   // CSTAGES x 8 KB
    unsigned char* sWc = sAc + CSTAGES * AC_STAGE_BYTES;            // CSTAGES x 4 KB
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(sWc + CSTAGES * WC_STAGE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                       // 0: issues the MMAs, 1: its peer
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    constexpr int BN_CTA_T = BN_T / 2;                              // weight rows decoded per CTA: 128 or 64
    constexpr uint32_t IDESC = umma_idesc_bf16(2 * BM_CTA, BN_T, false, false);
    const int tiles_m = (p.M + 2 * BM_CTA - 1) / (2 * BM_CTA), tiles_n = (p.N + BN_T - 1) / BN_T;
    const int num_tiles = tiles_m * tiles_n;
    // Which tiles a pair takes, and in which order.  col_fastest (the activation codes outweigh the weight codes: many
    // tokens): a contiguous run of tiles in the order (token tile, column tile) with the column fastest, so that the
    // pair's consecutive tiles share their activation codes, which then come from DRAM once.  Otherwise (few tokens, a
    // large weight matrix): round-robin with the token tile fastest, so that the pairs running at the same time share
    // a tile column's weight codes.
    const bool col_fastest = p.col_fastest != 0;
    const int tile_first = col_fastest ? (int)(((long long)pair * num_tiles) / num_pairs) : pair;
    const int tile_last = col_fastest ? (int)(((long long)(pair + 1) * num_tiles) / num_pairs) : num_tiles;
    const int tile_step = col_fastest ? 1 : num_pairs;
    auto tile_m = [&](int t) { return col_fastest ? t / tiles_n : t % tiles_m; };
    auto tile_n = [&](int t) { return col_fastest ? t % tiles_n : t / tiles_m; };
    const int kblocks = p.K / BK;
    constexpr int NLEV = 1 << W_BITS;
    constexpr int AC_ROW_BYTES = BK * A_BITS / 8;                   // 64 or 32 code bytes per token and k-block
    constexpr uint32_t CODE_TX_BYTES = BM_CTA * AC_ROW_BYTES + BN_CTA_T * (BK / 2);

    if (threadIdx.x == 0) {
        for (int s = 0; s < CSTAGES; ++s) {
            mbar_init(smem_u32(&ctl->cfull[s]), 1);
            mbar_init(smem_u32(&ctl->cempty[s]), GROUP_WARPS);
        }
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 2 * GROUP_WARPS);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[b]), 2 * NUM_EPI_WARPS);
        }
        ctl->abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmY);
    }
    if (warp == MMA_WARP) tmem_alloc_pair(smem_u32(&ctl->tmem_base), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                       // the peer's barriers exist before anyone arrives on them
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    // everything above touched no global memory: it may overlap the tail of the kernel before this one in the
    // stream (which produced the activation codes); everything below must see that kernel's writes
    lrq_pdl_trigger();
    lrq_pdl_wait();

    if (warp == TMA_WARP) {
        // =============================== packed codes: global -> shared (TMA) ===============================
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = tile_first; tile < tile_last && ok; tile += tile_step) {
                const int m_base = tile_m(tile) * 2 * BM_CTA + (int)rank * BM_CTA;
                const int n_base = tile_n(tile) * BN_T + (int)rank * BN_CTA_T;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int cs = it % CSTAGES;
                    ok = mbar_wait<200>(smem_u32(&ctl->cempty[cs]), ((it / CSTAGES) & 1) ^ 1, &ctl->abort_flag, p.status, 1);
                    if (!ok) break;
                    const uint32_t bar = smem_u32(&ctl->cfull[cs]);
                    mbar_arrive_expect_tx(bar, CODE_TX_BYTES);
                    tma_load_2d(smem_u32(sAc + cs * AC_STAGE_BYTES), &tmA, kb * AC_ROW_BYTES, m_base, bar);
                    tma_load_2d(smem_u32(sWc + cs * WC_STAGE_BYTES), &tmW, kb * (BK / 2), n_base, bar);
                }
            }
            if (!ok) {     // loads already issued still write this CTA's shared memory: let them land
                for (uint32_t back = 1; back <= (uint32_t)CSTAGES && back <= it; ++back) {
                    const uint32_t j = it - back;
                    const uint32_t bar = smem_u32(&ctl->cfull[j % CSTAGES]);
                    for (uint32_t i = 0; i < kWaitLimit; ++i)
                        if (mbar_try_wait(bar, (j / CSTAGES) & 1)) break;
                }
            }
        }
        __syncwarp();
    } else if (warp == MMA_WARP) {
        // =============================== MMA issuer (even CTA only) ========================================
        if (rank == 0 && lane == 0) {
            uint32_t it = 0, t = 0;
            bool ok = true;
            for (int tile = tile_first; tile < tile_last && ok; tile += tile_step, ++t) {
                const int buf = t & 1;
                ok = mbar_wait_cluster<64>(smem_u32(&ctl->tmem_empty[buf]), ((t >> 1) & 1) ^ 1, &ctl->abort_flag, p.status, 4);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN_T);
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % STAGES;
                    ok = mbar_wait_cluster<32>(smem_u32(&ctl->full[s]), (it / STAGES) & 1, &ctl->abort_flag, p.status, 5);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(sA + s * A_STAGE_BYTES), b_addr = smem_u32(sB + s * B_STAGE_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        tc_mma_f16_pair(d_tmem, umma_desc_sw128(a_addr + k * 32, 16, 1024),
                                        umma_desc_sw128(b_addr + k * 32, 16, 1024), IDESC, (kb | k) ? 1u : 0u);
                    tc_commit_pair(smem_u32(&ctl->empty[s]), 3);        // both CTAs may refill the stage
                }
                if (ok) tc_commit_pair(smem_u32(&ctl->tmem_full[buf]), 3);   // accumulator complete, both halves
            }
        }
        __syncwarp();
    } else if (warp < A_WARP0) {
        // =============================== B decode: one weight row (64 codes) per thread =====================
        // The eight warps form two groups that take alternate k-blocks, so that one group's barrier
        // latencies overlap the other's arithmetic.  A group's k-blocks are every second one of the CTA's
        // running count, across tile boundaries too, so ring slots and phases advance by fixed steps.
        const int t = threadIdx.x - B_WARP0 * 32;                  // 0..255
        // 256-wide tiles: a thread decodes a whole row of the CTA's 128 (two 32-code halves); 128-wide tiles: the
        // CTA has 64 rows and two threads share one, a half each
        constexpr int HALVES = BN_T == 256 ? 2 : 1;
        const int grp = t >> 7, row = BN_T == 256 ? (t & 127) : ((t & 127) >> 1), h0 = BN_T == 256 ? 0 : (t & 1);
        const int ngrp = p.K / p.G, kb_per_grp = p.G / BK;
        // the row's 16-byte chunk slots in a swizzled stage, and its code bytes in a code stage
        uint32_t off[4 * HALVES];
#pragma unroll
        for (int c = 0; c < 4 * HALVES; ++c) off[c] = swz(row, 4 * h0 + c);
        const uint32_t sB0 = smem_u32(sB), sWc0 = smem_u32(sWc) + (uint32_t)row * (BK / 2) + (uint32_t)h0 * 16;
        RingPos ring(grp);
        uint32_t it0 = 0;
        bool ok = true, have_next = false;
        float4 raw[NLEV / 4];
        for (int tile = tile_first; tile < tile_last && ok; tile += tile_step, it0 += kblocks) {
            const int n_base = tile_n(tile) * BN_T + (int)rank * BN_CTA_T;
            const int n = min(n_base + row, p.N - 1);               // rows past N decode a valid table; never stored
            const float4* tab = reinterpret_cast<const float4*>(p.levels + (size_t)n * ngrp * NLEV);
            const int kb0 = (grp ^ (int)it0) & 1;
            Lut L;
            // table index held in L / in raw, and the k-block at which the next table starts
            int gi = kb0 / kb_per_grp, fetched = gi, next_switch = (gi + 1) * kb_per_grp;
            if (kb0 < kblocks) {
                if (!(ngrp == 1 && have_next)) {                    // per-channel tables arrive a tile ahead (below)
#pragma unroll
                    for (int j = 0; j < NLEV / 4; ++j) raw[j] = __ldg(tab + (size_t)gi * (NLEV / 4) + j);
                }
                build_lut<W_BITS>(L, raw);
            }
            have_next = false;
            if (ngrp == 1 && tile + tile_step < tile_last) {
                // per-channel tables: the next tile's table is fetched now, a whole tile before it is needed
                const int nn = min(tile_n(tile + tile_step) * BN_T + (int)rank * BN_CTA_T + row, p.N - 1);
                const float4* tn = reinterpret_cast<const float4*>(p.levels + (size_t)nn * NLEV);
#pragma unroll
                for (int j = 0; j < NLEV / 4; ++j) raw[j] = __ldg(tn + j);
                have_next = true;
            }
            for (int kb = kb0; kb < kblocks; kb += 2) {
                if (ngrp > 1) {                                     // grouped tables: switch, and fetch one step ahead
                    if (kb >= next_switch) {
                        while (kb >= next_switch) { ++gi; next_switch += kb_per_grp; }
                        if (fetched != gi) {
#pragma unroll
                            for (int j = 0; j < NLEV / 4; ++j) raw[j] = __ldg(tab + (size_t)gi * (NLEV / 4) + j);
                            fetched = gi;
                        }
                        build_lut<W_BITS>(L, raw);
                    }
                    if (kb + 2 >= next_switch && kb + 2 < kblocks) {
                        int gn = gi, ns = next_switch;
                        while (kb + 2 >= ns) { ++gn; ns += kb_per_grp; }
                        if (gn != fetched) {
#pragma unroll
                            for (int j = 0; j < NLEV / 4; ++j) raw[j] = __ldg(tab + (size_t)gn * (NLEV / 4) + j);
                            fetched = gn;
                        }
                    }
                }
                ok = mbar_wait_warp<64>(smem_u32(&ctl->cfull[ring.cs]), ring.cph, &ctl->abort_flag, p.status, 2);
                if (!ok) break;
                uint4 cw2[HALVES];
#pragma unroll
                for (int h = 0; h < HALVES; ++h) lds128(sWc0 + ring.cs * WC_STAGE_BYTES + 16 * h, cw2[h]);
                ok = mbar_wait_warp<64>(smem_u32(&ctl->empty[ring.s]), ring.ph ^ 1, &ctl->abort_flag, p.status, 3);
                if (!ok) break;
                const uint32_t dst = sB0 + ring.s * B_STAGE_BYTES;
#pragma unroll
                for (int h = 0; h < HALVES; ++h) {
                    const uint4 cw = cw2[h];
                    uint32_t o[16];
                    decode_w<W_BITS, A_BITS == 4>(cw.x, L, o); decode_w<W_BITS, A_BITS == 4>(cw.y, L, o + 4);
                    decode_w<W_BITS, A_BITS == 4>(cw.z, L, o + 8); decode_w<W_BITS, A_BITS == 4>(cw.w, L, o + 12);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        sts128(dst + off[4 * h + j], o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive_cluster_light(smem_u32(&ctl->full[ring.s]), 0);      // the even CTA's barrier
                    // the code stage is handed back only here: every lane's loads from it have been consumed
                    // by the decode above, so none can still be in flight when the TMA overwrites it
                    mbar_arrive(smem_u32(&ctl->cempty[ring.cs]));
                }
                ring.advance();
            }
            if (__any_sync(0xffffffffu, ctl->abort_flag != 0)) ok = false;
        }
    } else if (warp < EPI_WARP0) {
        // =============================== A expansion: 16-byte chunks of the code stage ======================
        // Two groups of two warps, alternate k-blocks, like the B warps.  Chunk id = i * 64 + tl: consecutive
        // lanes read consecutive chunks; the row's low three bits, hence the swizzle, do not depend on i.
        const int t = threadIdx.x - A_WARP0 * 32;                  // 0..127
        const int grp = t >> 6, tl = t & 63;
        constexpr int CH_PER_ROW = AC_ROW_BYTES / 16;              // 4 or 2 code chunks per token row
        constexpr int TASKS = BM_CTA * CH_PER_ROW / 64;            // chunks per thread: 8 (8-bit) or 4 (4-bit)
        constexpr int OUT_CH = 8 / CH_PER_ROW;                     // bf16 chunks per code chunk: 2 or 4
        constexpr int ROWS_PER_TASK = 64 / CH_PER_ROW;             // rows between a thread's consecutive chunks
        const int row0 = tl / CH_PER_ROW, cc = tl % CH_PER_ROW;
        uint32_t off[OUT_CH];
#pragma unroll
        for (int j = 0; j < OUT_CH; ++j) off[j] = swz(row0, OUT_CH * cc + j);
        const uint32_t sA0 = smem_u32(sA), sAc0 = smem_u32(sAc) + (uint32_t)tl * 16;
        const ExpandConst kx;
        RingPos ring(grp);
        uint32_t it0 = 0;
        bool ok = true;
        for (int tile = tile_first; tile < tile_last && ok; tile += tile_step, it0 += kblocks) {
            for (int kb = (grp ^ (int)it0) & 1; kb < kblocks; kb += 2) {
                ok = mbar_wait_warp<64>(smem_u32(&ctl->cfull[ring.cs]), ring.cph, &ctl->abort_flag, p.status, 6);
                if (!ok) break;
                const uint32_t src = sAc0 + ring.cs * AC_STAGE_BYTES;
                uint4 cws[TASKS];
#pragma unroll
                for (int i = 0; i < TASKS; ++i) lds128(src + i * 1024, cws[i]);
                ok = mbar_wait_warp<64>(smem_u32(&ctl->empty[ring.s]), ring.ph ^ 1, &ctl->abort_flag, p.status, 7);
                if (!ok) break;
                uint32_t dst[OUT_CH];
#pragma unroll
                for (int j = 0; j < OUT_CH; ++j) dst[j] = sA0 + ring.s * A_STAGE_BYTES + off[j];
#pragma unroll
                for (int i = 0; i < TASKS; ++i) {
                    const uint4 cw = cws[i];
                    uint32_t o[4 * OUT_CH];
                    if constexpr (A_BITS == 8) {
                        expand_a8(cw.x, kx, o[0], o[1]); expand_a8(cw.y, kx, o[2], o[3]);
                        expand_a8(cw.z, kx, o[4], o[5]); expand_a8(cw.w, kx, o[6], o[7]);
                    } else {
                        expand_a4(cw.x, kx, o); expand_a4(cw.y, kx, o + 4); expand_a4(cw.z, kx, o + 8); expand_a4(cw.w, kx, o + 12);
                    }
#pragma unroll
                    for (int j = 0; j < OUT_CH; ++j)      // ROWS_PER_TASK rows further down: whole 1024-byte groups
                        sts128(dst[j] + i * (ROWS_PER_TASK / 8) * 1024, o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive_cluster_light(smem_u32(&ctl->full[ring.s]), 0);
                    mbar_arrive(smem_u32(&ctl->cempty[ring.cs]));
                }
                ring.advance();
            }
            if (__any_sync(0xffffffffu, ctl->abort_flag != 0)) ok = false;
        }
    } else {
        // =============================== epilogue: TMEM -> registers -> global ===============================
        const int ew = warp & 3;                                   // TMEM lane quadrant this warp may read
        const int et = threadIdx.x - EPI_WARP0 * 32;               // 0..127, for the cooperative column staging
        const int row = ew * 32 + lane;                            // accumulator row within the CTA
        const float zoff = (A_BITS == 8) ? 128.f : 8.f;            // the A operand is fed as q - 128 / q - 8
        const bool has_ws = p.wscale != nullptr, has_bias = p.bias != nullptr;
        uint32_t t = 0, nstore = 0;
        for (int tile = tile_first; tile < tile_last; tile += tile_step, ++t) {
            const int m0 = tile_m(tile) * 2 * BM_CTA + (int)rank * BM_CTA, n0 = tile_n(tile) * BN_T;
            const int buf = t & 1;
            // stage the tile's per-column terms (wsum, wscale, bias) in shared memory
            float (*col)[BN] = ctl->col[buf];
            for (int c = et; c < BN_T; c += NUM_EPI_WARPS * 32) {
                const int n = n0 + c;
                const bool okc = n < p.N;
                col[0][c] = okc ? __ldg(p.wsum + n) : 0.f;
                if (has_ws) col[1][c] = okc ? __ldg(p.wscale + n) : 1.f;
                if (has_bias) col[2][c] = okc ? __ldg(p.bias + n) : 0.f;
            }
            // barrier over the four epilogue warps; they leave together once any of them has seen the abort flag
            if (bar_or_epilogue(ctl->abort_flag != 0)) break;
            const int m = m0 + row;
            const bool row_ok = m < p.M;
            const float sm = row_ok ? __ldg(p.a_scale + m) : 0.f;
            const float zm = row_ok ? (float)__ldg(p.a_zp + m) + zoff : 0.f;
            const f32x2 SM = pack2(sm, sm), ZM = pack2(zm, zm);
            const bool okw = mbar_wait_warp<500>(smem_u32(&ctl->tmem_full[buf]), (t >> 1) & 1, &ctl->abort_flag, p.status, 8);
            tc_fence_after();
            if (okw) {
#pragma unroll 1
                for (int c0 = 0; c0 < BN_T; c0 += 32) {
                    if (n0 + c0 >= p.N) break;                     // warp-uniform
                    uint32_t acc[32];
                    tc_ld32(tmem_base + ((uint32_t)(ew * 32) << 16) + (uint32_t)(buf * BN_T + c0), acc);
                    tc_wait_ld();
                    f32x2 yq[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) yq[j] = 0ull;
                    if (row_ok) {
                        // y = s_m * (acc + z_m * wsum_n) [* wscale_n] [+ bias_n], two columns per instruction
                        f32x2* y = yq;
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float4 ws = *reinterpret_cast<const float4*>(&col[0][c0 + 4 * j]);
                            f32x2 a0 = fma2(ZM, pack2(ws.x, ws.y), pack2(__uint_as_float(acc[4 * j]), __uint_as_float(acc[4 * j + 1])));
                            f32x2 a1 = fma2(ZM, pack2(ws.z, ws.w), pack2(__uint_as_float(acc[4 * j + 2]), __uint_as_float(acc[4 * j + 3])));
                            a0 = mul2(a0, SM); a1 = mul2(a1, SM);
                            if (has_ws) {
                                const float4 sc = *reinterpret_cast<const float4*>(&col[1][c0 + 4 * j]);
                                a0 = mul2(a0, pack2(sc.x, sc.y)); a1 = mul2(a1, pack2(sc.z, sc.w));
                            }
                            if (has_bias) {
                                const float4 bi = *reinterpret_cast<const float4*>(&col[2][c0 + 4 * j]);
                                a0 = add2(a0, pack2(bi.x, bi.y)); a1 = add2(a1, pack2(bi.z, bi.w));
                            }
                            y[2 * j] = a0; y[2 * j + 1] = a1;
                        }
                    }
                    // A lane holds 32 consecutive outputs of its own row; stored as they are, every store would
                    // touch 32 different rows, a sector or less each.  The warp lays its chunk out in shared memory
                    // (rows of 128 bytes, 128-byte swizzle: conflict-free) and one lane hands it to the TMA, which
                    // writes whole lines, clips rows past M and columns past N, and runs while the next chunk is
                    // prepared.  fp32: one 32 x 32 tile per chunk; 16-bit: two chunks side by side, 32 rows x 64.
                    if (m0 + ew * 32 < p.M) {                          // warp-uniform; every store starts inside Y
                        const uint32_t tile = smem_u32(sEpi) + (uint32_t)((ew * EPI_TILES + (nstore % EPI_TILES)) * EPI_TILE_BYTES);
                        if (p.y_dtype == LRQ_F32) {
                            if (lane == 0) tma_store_wait_read<EPI_TILES - 1>();     // the store that last read this tile is done with it
                            __syncwarp();
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                float a, b, c2, d;
                                unpack2(yq[2 * j], a, b); unpack2(yq[2 * j + 1], c2, d);
                                sts128(tile + (uint32_t)(lane * 128 + ((j ^ (lane & 7)) << 4)), __float_as_uint(a), __float_as_uint(b),
                                       __float_as_uint(c2), __float_as_uint(d));
                            }
                            fence_async_smem();
                            __syncwarp();
                            if (lane == 0) tma_store_2d(&tmY, n0 + c0, m0 + ew * 32, tile);
                            ++nstore;
                        } else {
                            const int half = (c0 >> 5) & 1;
                            if (half == 0) {
                                if (lane == 0) tma_store_wait_read<EPI_TILES - 1>();
                                __syncwarp();
                            }
                            uint32_t h[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                float a, b; unpack2(yq[j], a, b);
                                if (p.y_dtype == LRQ_BF16) {
                                    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
                                    h[j] = *reinterpret_cast<uint32_t*>(&v);
                                } else {
                                    __half2 v = __floats2half2_rn(a, b);
                                    h[j] = *reinterpret_cast<uint32_t*>(&v);
                                }
                            }
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                sts128(tile + (uint32_t)(lane * 128 + (((half * 4 + j) ^ (lane & 7)) << 4)), h[4 * j], h[4 * j + 1],
                                       h[4 * j + 2], h[4 * j + 3]);
                            if (half == 1 || n0 + c0 + 32 >= p.N) {    // the pair is complete, or its second chunk lies past N
                                fence_async_smem();
                                __syncwarp();
                                if (lane == 0) tma_store_2d(&tmY, n0 + (c0 & ~63), m0 + ew * 32, tile);
                                ++nstore;
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            // CTA-scope release is enough: the accumulator reads above have completed (tcgen05.wait::ld)
            if (lane == 0) mbar_arrive_cluster_light(smem_u32(&ctl->tmem_empty[buf]), 0);
        }
        if (lane == 0) tma_store_wait_all();      // output tiles still in flight read this CTA's shared memory
    }

    // teardown: every role has left its loop.  Neither CTA may exit (or release TMEM) while its peer can
    // still arrive on its barriers or have MMAs reading its shared memory.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

template <int A_BITS, int W_BITS, int BN_T>
lrq_status launch(const Params& p, const CUtensorMap& tmA, const CUtensorMap& tmW, const CUtensorMap& tmY, int num_tiles, cudaStream_t st) {
    auto kern = qgemm_tc_kernel<A_BITS, W_BITS, BN_T>;
    // per device and kernel variant: the shared-memory opt-in (a per-device function attribute) and the number of
    // CTA pairs that can be resident; set up once under a lock, read-only afterwards
    static std::mutex mu;
    static int max_pairs_of[LRQ_MAX_DEVICES] = {};
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.blockDim = dim3(NUM_THREADS); cfg.dynamicSmemBytes = SMEM_BYTES; cfg.stream = st;
    cfg.attrs = attr; cfg.numAttrs = 2;
    int dev = 0, sms = 0, max_pairs = 0;
    if (lrq_current_device(&dev, &sms) != LRQ_OK) return LRQ_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!max_pairs_of[dev]) {
            LRQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
            int clusters = 0;
            cfg.gridDim = dim3(sms & ~1);
            cfg.numAttrs = 1;                 // the occupancy query looks at the cluster shape only
            LRQ_CUDA_TRY(cudaOccupancyMaxActiveClusters(&clusters, kern, &cfg));
            cfg.numAttrs = 2;
            if (clusters < 1) return LRQ_ERR_CUDA;
            max_pairs_of[dev] = clusters < sms / 2 ? clusters : sms / 2;
        }
        max_pairs = max_pairs_of[dev];
    }
    const int pairs = num_tiles < max_pairs ? num_tiles : max_pairs;
    cfg.gridDim = dim3(2 * pairs);
    LRQ_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, p, tmA, tmW, tmY));
    return LRQ_OK;
}

// Tile width.  A 128-wide tile was measured at about 0.87 of the time of a 256-wide one (the weight decode
// halves; the activation expansion, the hand-overs and the epilogue set-up do not), so it only pays when it
// cuts the number of rounds of tiles over the CTA pairs: small M with a narrow or ragged N (80 wide tiles on
// 74 pairs are two rounds, the same work as 144 narrow tiles is two cheaper rounds).
bool narrow_tiles(int M, int N, int sms, long* tiles) {
    const long pairs_avail = sms / 2 > 0 ? sms / 2 : 1;
    const long tiles_m = (M + 2 * BM_CTA - 1) / (2 * BM_CTA);
    const long t256 = tiles_m * ((N + 255) / 256), t128 = tiles_m * ((N + 127) / 128);
    const long r256 = (t256 + pairs_avail - 1) / pairs_avail, r128 = (t128 + pairs_avail - 1) / pairs_avail;
    const bool narrow = 0.87 * (double)r128 < (double)r256 - 1e-9;
    *tiles = narrow ? t128 : t256;
    return narrow;
}

bool tc_shape_ok(const lrq_layer* L) {
    // shapes this kernel takes: whole 64-wide k-blocks that never straddle a TLQ group; 16-byte aligned code rows
    if (L->K % BK || L->group % BK) return false;
    if (L->w_bits < 3 || L->w_bits > 4) return false;       // 2-bit tables take the CUDA-core kernel
    if (L->packed3) return false;                            // true 3-bit packing takes the small-M kernel
    return lrq_aligned(L->levels, 16) && lrq_aligned(L->codes, 16);
}

bool make_w_map(const lrq_layer* L, bool narrow, CUtensorMap* tm) {
    const uint64_t w_row = (uint64_t)L->K / 2;
    return lrq_tma::make_map_2d(tm, L->codes, 1, (uint64_t)L->N, w_row, w_row, BK / 2, narrow ? 64 : 128, false);
}

}  // namespace

void lrq_qgemm_tc_prepare(lrq_layer* L) {
    L->have_tm_w = tc_shape_ok(L) && make_w_map(L, false, &L->tm_w_wide) && make_w_map(L, true, &L->tm_w_narrow);
}

lrq_status lrq_launch_qgemm_tc(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale,
                               const int32_t* a_zp, int M, void* Y, lrq_dtype dt, long ldy, cudaStream_t st) {
    if (!tc_shape_ok(L) || !lrq_aligned(a_codes, 16)) return LRQ_ERR_UNSUPPORTED;
    const size_t es = dt == LRQ_F32 ? 4 : 2;
    if (!lrq_aligned(Y, 16) || ((size_t)ldy * es) % 16) return LRQ_ERR_UNSUPPORTED;
    const int ab = L->act.a_bits;
    Params p;
    p.a_scale = a_scale; p.a_zp = a_zp;
    p.levels = L->levels; p.wsum = L->wsum; p.wscale = L->wscale; p.bias = L->bias;
    p.Y = Y; p.ldy = ldy; p.M = M; p.N = L->N; p.K = L->K; p.G = L->group; p.y_dtype = (int)dt;
    // tile order: the operand whose codes weigh more is the one a pair keeps while it walks the other
    p.col_fastest = (size_t)M * ab > (size_t)L->N * 4 ? 1 : 0;      // M*K*ab/8 bytes of activation codes against N*K/2
    p.status = lrq_status_word();
    int sms = 0;
    if (lrq_current_device(nullptr, &sms) != LRQ_OK) return LRQ_ERR_CUDA;
    long tiles = 0;
    const bool narrow = narrow_tiles(M, L->N, sms, &tiles);
    // code matrices as byte tensors: a tile is 128 rows by one k-block of codes.  The weight side comes from the
    // layer handle; the activation codes and the output depend on this call's pointers and M.
    const uint64_t a_row = (uint64_t)L->K * ab / 8;
    CUtensorMap tmA, tmW_local;
    const CUtensorMap* tmW = narrow ? &L->tm_w_narrow : &L->tm_w_wide;
    if (!L->have_tm_w) {
        if (!make_w_map(L, narrow, &tmW_local)) return LRQ_ERR_CUDA;
        tmW = &tmW_local;
    }
    if (!lrq_tma::make_map_2d(&tmA, a_codes, 1, (uint64_t)M, a_row, a_row, BK * ab / 8, BM_CTA, false)) return LRQ_ERR_CUDA;
    // outputs leave through TMA stores of 32-row tiles, 128 bytes wide (32 fp32 or 64 16-bit columns)
    CUtensorMap tmY;
    if (!lrq_tma::make_map_2d(&tmY, Y, (int)es, (uint64_t)M, (uint64_t)L->N, (uint64_t)ldy, dt == LRQ_F32 ? 32 : 64, 32, true)) return LRQ_ERR_CUDA;
#define LRQ_GO(AB, WB) return narrow ? launch<AB, WB, 128>(p, tmA, *tmW, tmY, (int)tiles, st) : launch<AB, WB, 256>(p, tmA, *tmW, tmY, (int)tiles, st)
    if (ab == 8 && L->w_bits == 4) LRQ_GO(8, 4);
    if (ab == 8) LRQ_GO(8, 3);
    if (ab == 4 && L->w_bits == 4) LRQ_GO(4, 4);
    LRQ_GO(4, 3);
#undef LRQ_GO
}
