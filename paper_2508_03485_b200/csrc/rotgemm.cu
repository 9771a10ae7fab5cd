// Outlier-aware rotation y = x . R (Sec. 4.2, Eq. 12, second case) as a dense contraction on the
// 5th-generation tensor cores: X bf16 [M,K] times R bf16 [K,K] into an fp32 scratch that the
// per-token quantizer then reads.  bf16 x bf16 products are exact in fp32; sums are accumulated in fp32.
// The epilogue also folds every row's minimum and maximum into two integer arrays (atomic min / max on
// order-preserving images), so that the quantizer that follows is a single streaming pass.
//
// Persistent CTA per SM over 128 x 256 output tiles, 64-deep k-blocks, a 4-stage TMA pipeline:
//   warp 0      one lane issues the TMA tile loads (X: K-major box 64 x 128; R: four 64 x 64 boxes, each
//               64 output columns wide, one k-row per 128-byte line -> an MN-major UMMA operand)
//   warp 1      allocates TMEM, one lane issues tcgen05.mma (M = 128, N = 256, K = 16) and commits
//   warps 2-5   epilogue: tcgen05.ld of the finished accumulator, fp32 stores
// The accumulator is double-buffered in TMEM (2 x 256 columns).  Every wait is bounded; on expiry the
// CTA records a code in the status word, waits (bounded) for its TMA loads in flight and unwinds.
//
// The same kernel, instantiated with 128-wide tiles, multiplies by a block-diagonal matrix of 128 x 128
// blocks (the factors R1hat, R2hat of the dual transformation, Sec. 4.2): tile j of a token block only meets
// block j, so its k-loop covers 128 input channels instead of K.  There the left operand may come in `parts`
// column panels [M, parts*K] that are summed into one accumulator (the bf16 terms of an fp32 operand).
#include "lrq_internal.cuh"
#include "tc_ptx.cuh"
#include "tma_host.cuh"
#include <mutex>

namespace {
using namespace lrq_tc;

constexpr int BM = 128, BK = 64;
constexpr int STAGES = 4;
constexpr int A_STAGE_BYTES = BM * BK * 2;          // 16 KB
constexpr int B_CHUNK_BYTES = BK * 128;             // 8 KB: 64 k-rows of 64 output columns
constexpr int PRODUCER_WARP = 0, MMA_WARP = 1, EPI_WARP0 = 2, NUM_EPI_WARPS = 4;
constexpr int NUM_THREADS = (EPI_WARP0 + NUM_EPI_WARPS) * 32;   // 192
constexpr int TMEM_COLS = 512;

struct __align__(16) Ctl {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};
constexpr int EPI_TILE_BYTES = 32 * 32 * 4;         // one epilogue warp's 32 x 32 fp32 chunk, for the row/column trade
constexpr size_t smem_bytes(int bn) {
    return 1024 + (size_t)STAGES * (A_STAGE_BYTES + (bn / 64) * B_CHUNK_BYTES) + sizeof(Ctl) + NUM_EPI_WARPS * EPI_TILE_BYTES;
}

// BN: tile width (256 dense; 128 = the diagonal block size when DIAG).  DIAG: R is block-diagonal, stored as its
// blocks one after the other ([K/128][128][128], i.e. K rows of 128 columns); parts: column panels of the left operand.
template <int BN, bool DIAG>
__global__ void __launch_bounds__(NUM_THREADS, 1)
rotgemm_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmR,
                  float* __restrict__ Y, int M, int K, int parts, int* __restrict__ ext_min, int* __restrict__ ext_max,
                  int* status) {
    constexpr int B_STAGE_BYTES = (BN / 64) * B_CHUNK_BYTES;   // 32 KB (16 KB for 128-wide tiles)
    constexpr int STAGE_TX_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    constexpr uint32_t IDESC = umma_idesc_bf16(BM, BN, /*a_mn_major=*/false, /*b_mn_major=*/true);
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    unsigned char* sA = base;
    unsigned char* sB = base + STAGES * A_STAGE_BYTES;
    Ctl* ctl = reinterpret_cast<Ctl*>(sB + STAGES * B_STAGE_BYTES);
    const uint32_t sEpi = smem_u32(reinterpret_cast<unsigned char*>(ctl) + sizeof(Ctl));   // NUM_EPI_WARPS x 4 KB

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (M + BM - 1) / BM, tiles_n = (K + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    // dense: the whole of K (a ragged last k-block is zero-filled by TMA in both operands);
    // block-diagonal: the tile's own BN input channels, once per panel
    const int kblocks = DIAG ? parts * (BN / BK) : (K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(&ctl->full[s]), 1); mbar_init(smem_u32(&ctl->empty[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&ctl->tmem_full[b]), 1); mbar_init(smem_u32(&ctl->tmem_empty[b]), NUM_EPI_WARPS); }
        ctl->abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_desc(&tmX);
        tma_prefetch_desc(&tmR);
    }
    if (warp == MMA_WARP) tmem_alloc(smem_u32(&ctl->tmem_base), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    lrq_pdl_trigger();
    lrq_pdl_wait();                      // the set-up above overlaps the previous kernel's tail; X may be its output

    if (warp == PRODUCER_WARP) {
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % STAGES;
                    ok = mbar_wait<100>(smem_u32(&ctl->empty[s]), ((it / STAGES) & 1) ^ 1, &ctl->abort_flag, status, 11);
                    if (!ok) break;
                    const uint32_t bar = smem_u32(&ctl->full[s]);
                    mbar_arrive_expect_tx(bar, STAGE_TX_BYTES);
                    // k origin of this step in the left operand's columns and in R's rows
                    const int kx = DIAG ? (kb / (BN / BK)) * K + n0 + (kb % (BN / BK)) * BK : kb * BK;
                    const int kr = DIAG ? n0 + (kb % (BN / BK)) * BK : kb * BK;
                    tma_load_2d(smem_u32(sA + s * A_STAGE_BYTES), &tmX, kx, m0, bar);
#pragma unroll
                    for (int j = 0; j < BN / 64; ++j)
                        tma_load_2d(smem_u32(sB + s * B_STAGE_BYTES + j * B_CHUNK_BYTES), &tmR, (DIAG ? 0 : n0) + 64 * j, kr, bar);
                }
            }
            if (!ok) {
                // loads already issued still write this CTA's shared memory: let each stage's last fill land
                const uint32_t issued = it;
                for (uint32_t back = 1; back <= (uint32_t)STAGES && back <= issued; ++back) {
                    const uint32_t j = issued - back;
                    const uint32_t bar = smem_u32(&ctl->full[j % STAGES]);
                    for (uint32_t i = 0; i < kWaitLimit; ++i)
                        if (mbar_try_wait(bar, (j / STAGES) & 1)) break;
                }
            }
        }
        __syncwarp();
    } else if (warp == MMA_WARP) {
        if (lane == 0) {
            uint32_t it = 0, t = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++t) {
                const int buf = t & 1;
                ok = mbar_wait<64>(smem_u32(&ctl->tmem_empty[buf]), ((t >> 1) & 1) ^ 1, &ctl->abort_flag, status, 12);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % STAGES;
                    ok = mbar_wait<32>(smem_u32(&ctl->full[s]), (it / STAGES) & 1, &ctl->abort_flag, status, 13);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(sA + s * A_STAGE_BYTES), b_addr = smem_u32(sB + s * B_STAGE_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        tc_mma_f16(d_tmem,
                                   umma_desc_sw128(a_addr + k * 32, 16, 1024),                    // 16 k = 32 bytes along the row
                                   umma_desc_sw128(b_addr + k * 16 * 128, B_CHUNK_BYTES, 1024),   // 16 k = 16 rows of 128 bytes
                                   IDESC, (kb | k) ? 1u : 0u);
                    tc_commit(smem_u32(&ctl->empty[s]));
                }
                if (ok) tc_commit(smem_u32(&ctl->tmem_full[buf]));
            }
        }
        __syncwarp();
    } else {
        const int ew = warp & 3;                         // TMEM lane quadrant this warp may read
        const int row = ew * 32 + lane;
        uint32_t t = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++t) {
            const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
            const int buf = t & 1;
            const int m = m0 + row;
            const bool okw = mbar_wait<500>(smem_u32(&ctl->tmem_full[buf]), (t >> 1) & 1, &ctl->abort_flag, status, 14);
            tc_fence_after();
            float mn = INFINITY, mx = -INFINITY;         // extremes of this row over the tile's columns
            if (okw) {
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    if (n0 + c0 >= K) break;             // warp-uniform
                    uint32_t acc[32];
                    tc_ld32(tmem_base + ((uint32_t)(ew * 32) << 16) + (uint32_t)(buf * BN + c0), acc);
                    tc_wait_ld();
                    if (n0 + c0 + 32 <= K) {
                        // A lane holds 32 consecutive outputs of its own row.  The warp trades rows for columns through
                        // a 4 KB tile (chunk index XOR-ed with the row's low bits: conflict-free both ways) so that each
                        // store writes four rows' whole 128-byte lines instead of half a sector of 32 rows.
                        const uint32_t tile = sEpi + (uint32_t)(warp - EPI_WARP0) * EPI_TILE_BYTES;
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(tile + (uint32_t)(lane * 128 + ((j ^ (lane & 7)) << 4))),
                                         "r"(acc[4 * j]), "r"(acc[4 * j + 1]), "r"(acc[4 * j + 2]), "r"(acc[4 * j + 3]) : "memory");
                        __syncwarp();
                        const int rsub = lane >> 3, jq = lane & 7;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int r = 4 * i + rsub, mr = m0 + ew * 32 + r;
                            if (mr < M) {
                                uint4 v;
                                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                                             : "r"(tile + (uint32_t)(r * 128 + ((jq ^ (r & 7)) << 4))) : "memory");
                                *reinterpret_cast<uint4*>(Y + (size_t)mr * K + n0 + c0 + 4 * jq) = v;
                            }
                        }
                        if (m < M) {
#pragma unroll
                            for (int j = 0; j < 32; j += 2) {
                                asm("min.f32 %0, %0, %1, %2;" : "+f"(mn) : "f"(__uint_as_float(acc[j])), "f"(__uint_as_float(acc[j + 1])));
                                asm("max.f32 %0, %0, %1, %2;" : "+f"(mx) : "f"(__uint_as_float(acc[j])), "f"(__uint_as_float(acc[j + 1])));
                            }
                        }
                    } else if (m < M) {
                        float* dst = Y + (size_t)m * K + n0 + c0;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + c0 + j < K) {
                                const float v = __uint_as_float(acc[j]);
                                dst[j] = v; mn = fminf(mn, v); mx = fmaxf(mx, v);
                            }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[buf]));
            if (okw && m < M && ext_min) {                // fold this tile's share into the row's extremes
                atomicMin(ext_min + m, lrq_ordered_int(mn));
                atomicMax(ext_max + m, lrq_ordered_int(mx));
            }
            if (ctl->abort_flag) break;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace

template <int BN, bool DIAG>
static lrq_status launch_rotgemm(const CUtensorMap& tmX, const CUtensorMap& tmR, float* Y, int M, int K, int parts,
                                 int* ext_min, int* ext_max, cudaStream_t st) {
    int dev = 0, sms = 0;
    if (lrq_current_device(&dev, &sms) != LRQ_OK) return LRQ_ERR_CUDA;
    {   // the shared-memory opt-in is a per-device function attribute: set once per device
        static std::mutex mu;
        static bool configured[LRQ_MAX_DEVICES] = {};
        std::lock_guard<std::mutex> lock(mu);
        if (!configured[dev]) {
            LRQ_CUDA_TRY(cudaFuncSetAttribute(rotgemm_tc_kernel<BN, DIAG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)smem_bytes(BN)));
            configured[dev] = true;
        }
    }
    const int tiles = ((M + BM - 1) / BM) * ((K + BN - 1) / BN);
    if (ext_min) {
        // identity elements of the integer min / max: bytes 0x7f.. (a huge float), 0x80.. (a hugely negative one)
        LRQ_CUDA_TRY(cudaMemsetAsync(ext_min, 0x7f, (size_t)M * sizeof(int), st));
        LRQ_CUDA_TRY(cudaMemsetAsync(ext_max, 0x80, (size_t)M * sizeof(int), st));
    }
    LRQ_CUDA_TRY(lrq_launch_pdl(rotgemm_tc_kernel<BN, DIAG>, dim3(tiles < sms ? tiles : sms), dim3(NUM_THREADS), smem_bytes(BN),
                                st, tmX, tmR, Y, M, K, parts, ext_min, ext_max, lrq_status_word()));
    return LRQ_OK;
}

lrq_status lrq_launch_rotgemm(const void* X, int M, int K, long ldx, const void* R, float* Y,
                              int* ext_min, int* ext_max, cudaStream_t st) {
    // TMA needs 16-byte aligned bases and row pitches (K and ldx multiples of 8 elements); the C ABI has already
    // refused anything else
    if ((K % 8) || (ldx % 8) || !lrq_aligned(X, 16) || !lrq_aligned(R, 16) || !lrq_aligned(Y, 16) || !ext_min || !ext_max)
        return LRQ_ERR_INVALID_ARG;
    CUtensorMap tmX, tmR;
    if (!lrq_tma::make_map_2d(&tmX, X, 2, (uint64_t)M, (uint64_t)K, (uint64_t)ldx, BK, BM, true)) return LRQ_ERR_CUDA;
    if (!lrq_tma::make_map_2d(&tmR, R, 2, (uint64_t)K, (uint64_t)K, (uint64_t)K, 64, BK, true)) return LRQ_ERR_CUDA;
    return launch_rotgemm<256, false>(tmX, tmR, Y, M, K, 1, ext_min, ext_max, st);
}

// Y[M,K] (fp32) = sum over panels p of A[:, pK .. pK+K) . blockdiag(Rblk), Rblk bf16 [K/128][128][128].
// ext_min / ext_max may both be null (no per-row extremes wanted).
lrq_status lrq_launch_bdiag_gemm(const void* A, int M, int K, long lda, int parts, const void* Rblk, float* Y,
                                 int* ext_min, int* ext_max, cudaStream_t st) {
    if ((K % 128) || (lda % 8) || lda < (long)parts * K || parts < 1 || !lrq_aligned(A, 16) || !lrq_aligned(Rblk, 16) ||
        !lrq_aligned(Y, 16) || (ext_min == nullptr) != (ext_max == nullptr))
        return LRQ_ERR_INVALID_ARG;
    CUtensorMap tmA, tmR;
    if (!lrq_tma::make_map_2d(&tmA, A, 2, (uint64_t)M, (uint64_t)parts * K, (uint64_t)lda, BK, BM, true)) return LRQ_ERR_CUDA;
    if (!lrq_tma::make_map_2d(&tmR, Rblk, 2, (uint64_t)K, 128, 128, 64, BK, true)) return LRQ_ERR_CUDA;
    return launch_rotgemm<128, true>(tmA, tmR, Y, M, K, parts, ext_min, ext_max, st);
}
