/*
 * lrq.h - C ABI of the B200 (sm_100a) quantized-linear library for LRQ-DiT inference.
 *
 * The library implements the online path of one W-low-bit / A-low-bit linear layer of a
 * Diffusion Transformer and the offline weight quantizer that feeds it:
 *
 *   X[M,K] (bf16) --rotate (Sec. 4.2, Eq. 12)--> per-token quantize (Sec. 3.1, Eq. 1)
 *                 --contract with TLQ weight codes decoded through a level table
 *                   (Sec. 4.1, Eqs. 7-10)--> scale in the epilogue --> Y[M,N]
 *
 * Conventions that hold for every entry point unless its comment says otherwise
 * ---------------------------------------------------------------------------
 * Pointers   "dev"  = CUDA device memory owned by the caller, valid until the work enqueued by
 *            the call has finished; "host" = ordinary host memory, read during the call only.
 * Layout     all matrices are row-major.  4-bit data is packed two per byte, element 2j in the
 *            low nibble of byte j.  A weight nibble holds u = c + 2^(b-1) where c is the signed
 *            TLQ code of Eq. 5, so that u indexes the level table directly; 3-bit codes use the
 *            4-bit container.  The level table of a (row, group) has 2^b float entries in u order.
 * Streams    `cuda_stream` is a cudaStream_t passed as void* (NULL = legacy default stream).
 *            Calls enqueue work and return; they never synchronise and never allocate device
 *            memory.  Scratch comes from the caller's `workspace` (dev, 256-byte aligned).
 * Errors     every call returns an lrq_status; arguments are checked before anything is
 *            launched.  A device-side wait that runs out (every wait in the kernels is bounded)
 *            records a code that lrq_device_status() reports; the context stays usable.
 * Threads    calls on different streams with different workspaces may run concurrently.
 */
#ifndef LRQ_H_
#define LRQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LRQ_OK = 0,
    LRQ_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, misaligned pointer              */
    LRQ_ERR_UNSUPPORTED = 2,   /* bit-width, group or block size outside what the kernels cover   */
    LRQ_ERR_WORKSPACE = 3,     /* workspace missing or smaller than lrq_*_workspace_bytes reports */
    LRQ_ERR_CUDA = 4,          /* a CUDA runtime or driver call failed (launch, descriptor)        */
    LRQ_ERR_TIMEOUT = 5        /* a bounded device-side wait expired                               */
} lrq_status;

typedef enum { LRQ_ROT_NONE = 0, LRQ_ROT_HADAMARD = 1, LRQ_ROT_DENSE = 2, LRQ_ROT_DUAL = 3 } lrq_rot_kind;
typedef enum { LRQ_ACT_ASYM = 0, LRQ_ACT_SYM = 1 } lrq_act_mode;
typedef enum { LRQ_F32 = 0, LRQ_F16 = 1, LRQ_BF16 = 2 } lrq_dtype;
/* Storage of the weight codes (Sec. 4.1, Eq. 5: a b-bit code per weight).
 *   NIBBLE   two codes per byte, element 2j in the low nibble of byte j; row pitch K/2 bytes (b = 2..4)
 *   PACKED3  b = 3 only: eight codes in three bytes, code j of each eight at bits 3j..3j+2 of the little-endian
 *            24-bit word; row pitch 3K/8 bytes.  The storage TLQ's 3-bit codes actually need; taken by the
 *            weight-bandwidth-bound contraction for small token counts. */
typedef enum { LRQ_CODES_NIBBLE = 0, LRQ_CODES_PACKED3 = 1 } lrq_code_layout;

/* ---------------------------------------------------------------------------------------------
 * TLQ weight quantization (Sec. 4.1: Eqs. 4-5 twin-log quantizer, Eq. 6 search-based clipping,
 * Eq. 7 de-quantization, Eqs. 8-9 integerized levels).
 *
 * For every output row n and every group of `group_size` consecutive input channels the kernel
 * takes log2|w| of the positive and of the negative elements separately, searches the clipping
 * factor of each side over the caller's grid (squared error of the de-quantized magnitudes, summed in
 * fp64 over the side's elements in increasing k; first minimum in grid order wins), and emits the signed code of Eq. 5 plus the table of level values
 * II * 2^(f-I) of Eqs. 8-9.  Code 0 is shared by the lowest positive level, by negative elements
 * that round to the negative side's code 0, and by exact zeros; its table entry is the lowest
 * positive level.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    int w_bits;            /* b: 2, 3 or 4                                                        */
    int group_size;        /* G consecutive input channels per table; 0 means K (per channel)    */
    int integerize_I;      /* I of Eq. 9, 1..7 (7: every level is exactly a bf16 number)         */
    int n_alpha, n_beta;   /* grid sizes, 1..64                                                   */
    const double* alpha;   /* host: clipping factors tried on the positive side (Eq. 6)          */
    const double* beta;    /* host: clipping factors tried on the negative side                  */
    lrq_code_layout code_layout;   /* how `codes` is written; PACKED3 needs w_bits == 3                    */
} lrq_tlq_params;

/*
 * W_rot  dev  float [N,K]   weights in the rotated basis (W.R of Eq. 2), row-major, 16-byte aligned
 * codes  dev  uint8 [N,K/2] (NIBBLE) or [N,3K/8] (PACKED3) offset-binary codes u = c + 2^(b-1) (out)
 * levels dev  float [N,K/G,2^b] level tables (out)
 * meta   dev  double [N,K/G,6]  s+, z+, s-, z-, alpha, beta chosen per group (out, may be NULL)
 * wsum   dev  float [N]     sum over k of the de-quantized row, used by the zero-point term (out)
 * No workspace is needed (pass NULL, 0).  K must be even and a multiple of G; G a multiple of 8.
 */
lrq_status lrq_tlq_quantize_weights(const float* W_rot, int N, int K, const lrq_tlq_params* p,
                                    uint8_t* codes, float* levels, double* meta, float* wsum,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Rotation + per-token activation quantization (Sec. 4.2, Eq. 12; Sec. 3.1, Eq. 1 applied per
 * token as in Sec. 5.1).
 *
 *   HADAMARD  y = x . blockdiag(H_B), H_B the normalised Sylvester matrix of Eq. 3, B = had_block
 *             a power of two (8..4096) dividing K: one fused kernel, fp32 butterflies.
 *   DENSE     y = x . R with the composed outlier-aware rotation given as one bf16 K x K matrix
 *             (second case of Eq. 12): a tcgen05 GEMM into an fp32 scratch, then the quantizer.
 *   DUAL      the same outlier-aware transformation kept in the factors Sec. 4.2 builds it from,
 *             y = x . R1hat . P . R2hat: R1hat, R2hat block-diagonal with K/Bd orthogonal bf16 blocks of
 *             Bd x Bd, P the staggered channel reordering as an index map, (u P)_i = u[perm[i]].  Two
 *             block-diagonal tcgen05 products (2.M.K.Bd flop each instead of 2.M.K.K, and no K x K matrix to
 *             read) with a gather between them; the gathered fp32 intermediate is split into three bf16 terms
 *             so that the second product keeps fp32 accuracy.  Bd = 128, K a multiple of 128.
 *   NONE      y = x.
 * then, per token, ASYM: s = (max-min)/(2^b-1), z = rint(min/s), q = clamp(rint(y/s)-z, 0, 2^b-1);
 *                  SYM : s = max|y|/(2^(b-1)-1), z = -2^(b-1), same q.   Rounding is to nearest even.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    lrq_rot_kind kind;
    int had_block;           /* B for HADAMARD; ignored otherwise                                 */
    const void* R_bf16;      /* dev bf16 [K,K] row-major for DENSE (y_i = sum_l x_l R[l,i])        */
    int a_bits;              /* 4 or 8                                                            */
    lrq_act_mode mode;
    const float* prescale;   /* nullable dev float [K], 16-byte aligned: smoothing multipliers applied
                                channel-wise before the rotation (Sec. 5.1: X' = X diag(prescale), the
                                weights having absorbed diag(1/prescale)).  HADAMARD / NONE only; for a
                                DENSE or DUAL rotation fold diag(prescale) into R / R1.               */
    /* DUAL only (ignored otherwise): */
    int dual_block;          /* Bd: 128                                                            */
    const void* R1_bf16;     /* dev bf16 [K/Bd,Bd,Bd]: u_{jBd+i} = sum_l x_{jBd+l} R1[j][l][i]; 16-byte aligned */
    const int32_t* perm;     /* dev int32 [K]: a permutation of 0..K-1; position i takes channel perm[i].  An entry
                                outside 0..K-1 is read as channel 0 and recorded (lrq_device_status code 31).  */
    const void* R2_bf16;     /* dev bf16 [K/Bd,Bd,Bd], applied after the reordering                */
} lrq_act_params;

/* Bytes of workspace lrq_rotate_quantize_act needs for M tokens: 0 for HADAMARD / NONE, 4.M.K for DENSE (the fp32
 * rotated activations), 10.M.K for DUAL (an fp32 array that holds first u, later y, and the three bf16 terms of
 * the reordered u). */
size_t lrq_act_workspace_bytes(int M, int K, const lrq_act_params* p);

/*
 * X_bf16  dev  bf16 [M,ldx] activations, ldx >= K elements, rows 16-byte aligned
 * a_codes dev  uint8 [M,K] (a_bits = 8) or [M,K/2] packed (a_bits = 4)            (out)
 * a_scale dev  float [M]  s of Eq. 1 per token                                    (out)
 * a_zp    dev  int32 [M]  z of Eq. 1 per token                                    (out)
 * K must be a multiple of 8.
 */
lrq_status lrq_rotate_quantize_act(const void* X_bf16, int M, int K, long ldx, const lrq_act_params* p,
                                   uint8_t* a_codes, float* a_scale, int32_t* a_zp,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Adaptive Rotation Scheme, the per-layer choice (Sec. 4.2): fluctuation metric of a batch of
 * calibration activations, J = ||X||_F / sqrt(M K) (Eq. 11), and the rotation kind of Eq. 12:
 * LRQ_ROT_HADAMARD when J < threshold (the paper uses 1), LRQ_ROT_DENSE otherwise.
 *   X         dev bf16 [M,ldx], 32-byte aligned, K and ldx multiples of 16
 *   J, kind   dev float / int32, one element each (out)
 *   workspace dev, 8 bytes, 8-byte aligned (one double; cleared by the call)
 * ------------------------------------------------------------------------------------------- */
lrq_status lrq_ars_select(const void* X_bf16, int M, int K, long ldx, double threshold, float* J, int32_t* kind,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Weight side of the rotation identity (Sec. 3.2, Eq. 2: (X R)(W R)^T = X W^T), offline:
 *   W_rot = W diag(colmul) R,   evaluated in fp64 and rounded once to fp32,
 * the matrix lrq_tlq_quantize_weights reads.  R is the layer's rotation: blockdiag(H_B) (Eq. 3), the
 * stored bf16 matrix of the dense case (the same array lrq_act_params.R_bf16 points to, so both
 * sides of Eq. 2 use one R), or the identity.  colmul absorbs the smoothing of Sec. 5.1: with
 * activations multiplied by prescale[k], pass colmul[k] = 1 / prescale[k].
 *   W       dev float [N,ldw], ldw >= K
 *   colmul  dev float [K], nullable (all ones)
 *   R_bf16  dev bf16 [K,K] row-major, LRQ_ROT_DENSE only
 *   W_rot   dev float [N,ldo], ldo >= K (out); may be W itself except for LRQ_ROT_DENSE
 * LRQ_ROT_HADAMARD: had_block a power of two dividing K, K <= 25600 (the row is held in shared
 * memory as fp64).  No workspace.
 * ------------------------------------------------------------------------------------------- */
lrq_status lrq_rotate_weights(const float* W, int N, int K, long ldw, const float* colmul, lrq_rot_kind kind,
                              int had_block, const void* R_bf16, float* W_rot, long ldo, void* cuda_stream);

/* The same for the dual transformation in its factors (LRQ_ROT_DUAL): W_rot = W diag(colmul) R1hat P R2hat,
 * arguments as in lrq_act_params.  Each row is held in shared memory as fp64: K <= 12288. */
lrq_status lrq_rotate_weights_dual(const float* W, int N, int K, long ldw, const float* colmul, int dual_block,
                                   const void* R1_bf16, const int32_t* perm, const void* R2_bf16,
                                   float* W_rot, long ldo, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * lrq_rotate_quantize_act for callers that cannot hand over device scratch.
 *
 * (The paper has no counterpart; this entry point exists for integration reasons only.)
 *
 * Some hosts of this library have no way to allocate device memory at the point where they call
 * it: a plugin or a callback that runs inside someone else's pre-planned memory arena, a
 * real-time or safety-reviewed inference loop in which cudaMalloc (which may synchronise the
 * whole device and can fail) is forbidden after start-up, or a process whose allocator is owned
 * by another runtime.  The dense rotation needs an fp32 scratch of M*K elements between the
 * rotation GEMM and the quantizer; here that scratch is a fixed array inside the library image
 * (LRQ_STATIC_SCRATCH_BYTES, held by every GPU that loads the library until the process exits).
 *
 *   - Arguments and results are those of lrq_rotate_quantize_act without the workspace pair.
 *   - kind == LRQ_ROT_DENSE needs M*K*4 <= LRQ_STATIC_SCRATCH_BYTES (LRQ_ROT_DUAL: M*K*10), otherwise the
 *     call returns LRQ_ERR_WORKSPACE and launches nothing (split the tokens into several calls).  The
 *     other kinds use no scratch and have no size limit.
 *   - The call allocates nothing (no cudaMalloc/cudaFree, no allocating library routine).  Every call
 *     asks the runtime for the device address of the array (a host-side query, no launch, nothing cached
 *     here, so a device reset between calls is harmless).  The FIRST call of the process on each device
 *     may make the runtime load this library's device code, which reserves memory on the driver's side
 *     and is not allowed while a stream is being captured: make one call (any M, e.g. one token) on each
 *     device at start-up, before the phase in which allocation is forbidden.
 *   - All calls on a device share the one array.  Its contents after a call are the last rotation's
 *     output; nothing in it has to start at zero, because the rotation overwrites every element the
 *     quantizer reads.  Two calls that may overlap on the GPU (different streams) race on it:
 *     serialise them.
 * ------------------------------------------------------------------------------------------- */
#define LRQ_STATIC_SCRATCH_BYTES (8u << 20)
size_t lrq_static_scratch_bytes(void);   /* the value the library was built with */

lrq_status lrq_rotate_quantize_act_static(const void* X_bf16, int M, int K, long ldx, const lrq_act_params* p,
                                          uint8_t* a_codes, float* a_scale, int32_t* a_zp, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * A quantized layer: TLQ codes, level tables and the activation recipe of one linear.
 * The handle is a small host object; it stores the device pointers it is given (it does not
 * copy or own them) and must be destroyed with lrq_layer_destroy.
 *   codes [N,K/2] or [N,3K/8] (code_layout), levels [N,K/G,2^b], wsum [N] as produced by
 *   lrq_tlq_quantize_weights (codes, levels 16-byte aligned);
 *   wscale (nullable) float [N] per-channel output scale, bias (nullable) float [N].
 * ------------------------------------------------------------------------------------------- */
typedef struct lrq_layer lrq_layer;

lrq_status lrq_layer_create(lrq_layer** out, int N, int K, int w_bits, int group_size, lrq_code_layout code_layout,
                            const uint8_t* codes, const float* levels, const float* wsum,
                            const float* wscale, const float* bias, const lrq_act_params* act);
void lrq_layer_destroy(lrq_layer* L);

/* Bytes of workspace lrq_qlinear needs for M tokens of this layer (activation codes, scales,
 * zero-points, and the fp32 scratch of a dense rotation). */
size_t lrq_workspace_bytes(const lrq_layer* L, int M);

/* ---------------------------------------------------------------------------------------------
 * The quantized linear layer (Eq. 12 -> Eq. 1 -> Eq. 10 -> scaling):
 *   acc[m,n] = sum_k q[m,k] * T[n, k/G, u[n,k]]            tcgen05 MMA, exact products, fp32 accumulate
 *   Y[m,n]   = s_m * (acc + z_m * wsum_n) * wscale_n + bias_n
 * X as in lrq_rotate_quantize_act; Y dev [M,ldy] of `y_dtype`, ldy >= N elements, rows 16-byte aligned.
 * ------------------------------------------------------------------------------------------- */
lrq_status lrq_qlinear(const lrq_layer* L, const void* X_bf16, int M, long ldx,
                       void* Y, lrq_dtype y_dtype, long ldy,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same for n_layers independent layers, enqueued back to back on one stream and sharing one
 * workspace of at least the largest lrq_workspace_bytes(layers[i], M[i]).
 * layers, X, M, ldx, Y, ldy are host arrays of length n_layers (X[i], Y[i] are dev pointers). */
lrq_status lrq_qlinear_stack(const lrq_layer* const* layers, int n_layers,
                             const void* const* X, const int* M, const long* ldx,
                             void* const* Y, lrq_dtype y_dtype, const long* ldy,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Contraction and epilogue alone (Eq. 10), on activation codes produced earlier by
 * lrq_rotate_quantize_act.  `impl`: 0 = large-tile tcgen05 kernel (pairs of CTAs, 256 x 256 tiles), 1 = plain
 * CUDA-core kernel (kept as the in-library ablation baseline), 2 = small-tile tcgen05 kernel (128 x 32 tiles: the
 * one lrq_qlinear picks for a few hundred tokens or fewer, and the only tensor-core kernel that reads
 * LRQ_CODES_PACKED3), 3 = the integer form of Eq. 10 on the CUDA cores (mantissa products shifted by the level
 * exponents, exact integer accumulation; I = 7 tables; a slow cross-check of the two forms, not a production path).
 * LRQ_ERR_UNSUPPORTED when the kernel asked for does not take the layer's shape.
 * No workspace needed. */
lrq_status lrq_qgemm_codes(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale,
                           const int32_t* a_zp, int M, void* Y, lrq_dtype y_dtype, long ldy,
                           int impl, void* cuda_stream);

/* Code recorded by a bounded device-side wait that expired since the last call of this function
 * (0 if none).  Synchronises `cuda_stream` to read it. */
int lrq_device_status(void* cuda_stream);

/* Diagnostic of the bounded waits (no counterpart in the paper): launches a one-warp kernel that waits, through the
 * same bounded-wait routine the tensor-core kernels use, on a barrier nothing ever arrives on.  After
 * `limit_cycles` SM clock cycles (1 .. 1e8) the wait gives up, records LRQ_SELFTEST_WAIT_CODE in the status word
 * and the kernel returns; lrq_device_status() then reports that code once.  Nothing else is in flight in that
 * kernel, so the context stays usable. */
#define LRQ_SELFTEST_WAIT_CODE 99
lrq_status lrq_selftest_wait_timeout(long long limit_cycles, void* cuda_stream);

const char* lrq_status_string(lrq_status s);
int lrq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LRQ_H_ */
