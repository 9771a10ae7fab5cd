// Internal declarations shared by the translation units of the CUDA library.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include "../../include/lrq.h"

#define LRQ_CUDA_TRY(expr)                                   \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) { (void)cudaGetLastError(); return LRQ_ERR_CUDA; } \
    } while (0)

static inline bool lrq_is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }
static inline bool lrq_aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
static inline size_t lrq_round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

#include <cuda.h>

struct lrq_layer {
    int N, K, w_bits, group;          // group == K for per-channel tables
    int packed3;                      // 1: codes are true 3-bit packed (8 codes in 3 bytes, row pitch 3K/8 bytes)
    const uint8_t* codes;
    const float* levels;
    const float* wsum;
    const float* wscale;
    const float* bias;
    lrq_act_params act;
    // what does not change from call to call, prepared once by lrq_layer_create (read-only afterwards, so
    // concurrent calls on one layer need no lock): TMA descriptors of the weight codes for the two tile widths
    // of the tensor-core contraction.  have_tm_w is false when the shape takes the CUDA-core kernel, or when no
    // driver was present at creation (the launch then encodes the descriptors itself).
    bool have_tm_w;
    CUtensorMap tm_w_wide, tm_w_narrow;
};

constexpr int LRQ_MAX_DEVICES = 64;

// Current device and its SM count (queried once per device, thread-safe).
lrq_status lrq_current_device(int* dev, int* sms);

// Device status word: written by a kernel whose bounded wait expired.  A file-scope device variable of the
// library image; this returns its address on the current device.
int* lrq_status_word();

// Launch with programmatic stream serialization: the kernel may become resident while its predecessor in the
// stream is still draining; it must execute lrq_pdl_wait() before its first access to global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t lrq_launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// rotq.cu
lrq_status lrq_launch_rotq_hadamard(const void* X, int M, int K, long ldx, int B, int a_bits, int mode, const float* prescale,
                                    uint8_t* codes, float* scale, int32_t* zp, cudaStream_t st);
// rotq_blk.cu : the same for blocks of 8..128 channels with K a multiple of 128; LRQ_ERR_UNSUPPORTED otherwise
lrq_status lrq_launch_rotq_blk(const void* X, int M, int K, long ldx, int B, int a_bits, int mode, const float* prescale,
                               uint8_t* codes, float* scale, int32_t* zp, cudaStream_t st);
// rotgemm.cu : Y[M,K] (fp32) = X[M,K] (bf16) . R[K,K] (bf16) on the tensor cores; also leaves every row's minimum and
// maximum in ext_min[M] / ext_max[M] as order-preserving integers.
lrq_status lrq_launch_rotgemm(const void* X, int M, int K, long ldx, const void* R, float* Y,
                              int* ext_min, int* ext_max, cudaStream_t st);
// rotgemm.cu : Y[M,K] (fp32) = sum over the `parts` column panels of A[M, parts*K] (bf16) of panel . blockdiag(Rblk),
// Rblk bf16 [K/128][128][128]; row extremes as above when ext_min / ext_max are given (both or neither).
lrq_status lrq_launch_bdiag_gemm(const void* A, int M, int K, long lda, int parts, const void* Rblk, float* Y,
                                 int* ext_min, int* ext_max, cudaStream_t st);
// rotdual.cu : V3 bf16 [M,3K], panel p = p-th bf16 term of U[m, perm[i]] (the reordering between the two rotations)
lrq_status lrq_launch_dual_gather_split(const float* U, int M, int K, const int32_t* perm, void* V3, cudaStream_t st);
// rotq.cu : per-token quantization of fp32 rows whose extremes are already known (ext_min / ext_max alias the
// scale / zero-point outputs: each row's extremes are read before its results are written).
lrq_status lrq_launch_quantize_f32_ext(const float* Y, int M, int K, int a_bits, int mode, uint8_t* codes,
                                       float* scale, int32_t* zp, cudaStream_t st);

// rotq.cu : fluctuation metric J (Eq. 11) and the kind Eq. 12 picks; acc is one double of device scratch
lrq_status lrq_launch_ars_metric(const void* X, int M, int K, long ldx, double thr, float* J, int* kind, double* acc,
                                 cudaStream_t st);

// wrot.cu : W diag(colmul) R in fp64, rounded to fp32 (Eq. 2, weight side)
lrq_status lrq_launch_rotate_weights(const float* W, int N, int K, long ldw, const float* colmul, int kind,
                                     int had_block, const void* R, float* out, long ldo, cudaStream_t st);
lrq_status lrq_launch_rotate_weights_dual(const float* W, int N, int K, long ldw, const float* colmul, int Bd, const void* R1,
                                          const int32_t* perm, const void* R2, float* out, long ldo, cudaStream_t st);

#ifdef __CUDACC__
// Programmatic dependent launch.  Every hot kernel lets its successor in the stream start early (the successor's
// prologue - barrier set-up, TMEM allocation, descriptor prefetch - overlaps this kernel's tail) and, before its
// own first global access, waits until its predecessor has completed and its writes are visible.  Both are
// no-ops for a launch without the attribute.
__device__ __forceinline__ void lrq_pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void lrq_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Order-preserving map between fp32 and int32 (and back), so that integer min/max reductions serve floats.
__device__ __forceinline__ int lrq_ordered_int(float f) { const int i = __float_as_int(f); return i ^ ((i >> 31) & 0x7fffffff); }
__device__ __forceinline__ float lrq_ordered_float(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }
#endif
// qgemm_simple.cu / qgemm_tc.cu
lrq_status lrq_launch_qgemm_simple(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale,
                                   const int32_t* a_zp, int M, void* Y, lrq_dtype dt, long ldy, cudaStream_t st);
// qgemm_simple.cu : the integer form of Eq. 10 (mantissa products, shifts, exact integer accumulation) on the CUDA cores
lrq_status lrq_launch_qgemm_shift(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale,
                                  const int32_t* a_zp, int M, void* Y, lrq_dtype dt, long ldy, cudaStream_t st);
lrq_status lrq_launch_qgemm_tc(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale,
                               const int32_t* a_zp, int M, void* Y, lrq_dtype dt, long ldy, cudaStream_t st);
// qgemm_small.cu : 128 x 32 tiles, one CTA each, for small token counts and for packed 3-bit codes
bool lrq_qgemm_small_takes(const lrq_layer* L);
lrq_status lrq_launch_qgemm_small(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale,
                                  const int32_t* a_zp, int M, void* Y, lrq_dtype dt, long ldy, cudaStream_t st);
// fills the layer's cached TMA descriptors (called once by lrq_layer_create; never fails: without a driver, or for
// shapes the tensor-core kernel does not take, the layer is simply left without them)
void lrq_qgemm_tc_prepare(lrq_layer* L);
