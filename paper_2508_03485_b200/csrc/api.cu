// C-ABI entry points: argument checks, workspace carving, launches.  No entry point allocates
// device memory or synchronises (lrq_device_status excepted, which reads one word back).
#include "lrq_internal.cuh"
#include <mutex>
#include <new>

// Status word written by a kernel whose bounded wait expired.  A file-scope device variable: in
// host code its name is only a handle, the device address comes from cudaGetSymbolAddress (for
// the device that is current at the time of the call).
__device__ int g_lrq_status_word;

int* lrq_status_word() {
    int* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_lrq_status_word) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    return p;
}

// Current device and its SM count.  The attribute is queried once per device; the cache is filled under a
// lock and read-only afterwards.
lrq_status lrq_current_device(int* dev_out, int* sms_out) {
    static std::mutex mu;
    static int sms_of[LRQ_MAX_DEVICES] = {};
    int dev = -1;
    LRQ_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= LRQ_MAX_DEVICES) return LRQ_ERR_UNSUPPORTED;
    int sms;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!sms_of[dev]) {
            int v = 0;
            LRQ_CUDA_TRY(cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev));
            if (v < 1) return LRQ_ERR_CUDA;
            sms_of[dev] = v;
        }
        sms = sms_of[dev];
    }
    if (dev_out) *dev_out = dev;
    if (sms_out) *sms_out = sms;
    return LRQ_OK;
}

static lrq_status check_act(const lrq_act_params* p, int K) {
    if (!p) return LRQ_ERR_INVALID_ARG;
    if (p->a_bits != 4 && p->a_bits != 8) return LRQ_ERR_UNSUPPORTED;
    if (p->mode != LRQ_ACT_ASYM && p->mode != LRQ_ACT_SYM) return LRQ_ERR_INVALID_ARG;
    if (K <= 0 || K % 8) return LRQ_ERR_UNSUPPORTED;
    switch (p->kind) {
        case LRQ_ROT_NONE: break;
        case LRQ_ROT_HADAMARD:
            if (!lrq_is_pow2(p->had_block) || p->had_block < 8 || p->had_block > 4096 || K % p->had_block)
                return LRQ_ERR_UNSUPPORTED;
            break;
        case LRQ_ROT_DENSE:
            if (!p->R_bf16) return LRQ_ERR_INVALID_ARG;
            if (!lrq_aligned(p->R_bf16, 16)) return LRQ_ERR_INVALID_ARG;
            if (p->prescale) return LRQ_ERR_UNSUPPORTED;      // fold diag(prescale) into R instead
            break;
        case LRQ_ROT_DUAL:
            if (!p->R1_bf16 || !p->R2_bf16 || !p->perm) return LRQ_ERR_INVALID_ARG;
            if (!lrq_aligned(p->R1_bf16, 16) || !lrq_aligned(p->R2_bf16, 16) || !lrq_aligned(p->perm, 4)) return LRQ_ERR_INVALID_ARG;
            if (p->dual_block != 128 || K % 128 || K > 12288) return LRQ_ERR_UNSUPPORTED;
            if (p->prescale) return LRQ_ERR_UNSUPPORTED;      // fold diag(prescale) into R1 instead
            break;
        default: return LRQ_ERR_INVALID_ARG;
    }
    if (p->prescale && !lrq_aligned(p->prescale, 16)) return LRQ_ERR_INVALID_ARG;
    return LRQ_OK;
}

extern "C" size_t lrq_act_workspace_bytes(int M, int K, const lrq_act_params* p) {
    if (!p || M <= 0 || K <= 0) return 0;
    const size_t rotated = lrq_round_up((size_t)M * K * sizeof(float), 256);
    if (p->kind == LRQ_ROT_DENSE) return rotated;
    if (p->kind == LRQ_ROT_DUAL) return rotated + lrq_round_up((size_t)M * K * 6, 256);   // + three bf16 panels
    return 0;
}

extern "C" lrq_status lrq_rotate_quantize_act(const void* X, int M, int K, long ldx, const lrq_act_params* p,
                                              uint8_t* a_codes, float* a_scale, int32_t* a_zp,
                                              void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!X || !a_codes || !a_scale || !a_zp || M <= 0) return LRQ_ERR_INVALID_ARG;
    lrq_status st = check_act(p, K);
    if (st != LRQ_OK) return st;
    if (ldx < K || (ldx % 8) || !lrq_aligned(X, 16) || !lrq_aligned(a_codes, 16)) return LRQ_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (p->kind == LRQ_ROT_DENSE) {
        const size_t need = lrq_act_workspace_bytes(M, K, p);
        if (!workspace || workspace_bytes < need || !lrq_aligned(workspace, 256)) return LRQ_ERR_WORKSPACE;
        float* Yr = static_cast<float*>(workspace);
        // the rotation leaves each token's extremes in the scale / zero-point outputs (as integers); the
        // quantizer reads them and then writes the real values there
        st = lrq_launch_rotgemm(X, M, K, ldx, p->R_bf16, Yr, reinterpret_cast<int*>(a_scale), reinterpret_cast<int*>(a_zp), stream);
        if (st != LRQ_OK) return st;
        return lrq_launch_quantize_f32_ext(Yr, M, K, p->a_bits, p->mode, a_codes, a_scale, a_zp, stream);
    }
    if (p->kind == LRQ_ROT_DUAL) {
        const size_t need = lrq_act_workspace_bytes(M, K, p);
        if (!workspace || workspace_bytes < need || !lrq_aligned(workspace, 256)) return LRQ_ERR_WORKSPACE;
        float* Yr = static_cast<float*>(workspace);                       // u = x R1hat first, y later
        void* V3 = static_cast<unsigned char*>(workspace) + lrq_round_up((size_t)M * K * sizeof(float), 256);
        st = lrq_launch_bdiag_gemm(X, M, K, ldx, 1, p->R1_bf16, Yr, nullptr, nullptr, stream);
        if (st != LRQ_OK) return st;
        st = lrq_launch_dual_gather_split(Yr, M, K, p->perm, V3, stream);  // u P as three bf16 terms
        if (st != LRQ_OK) return st;
        st = lrq_launch_bdiag_gemm(V3, M, K, 3L * K, 3, p->R2_bf16, Yr, reinterpret_cast<int*>(a_scale),
                                   reinterpret_cast<int*>(a_zp), stream);
        if (st != LRQ_OK) return st;
        return lrq_launch_quantize_f32_ext(Yr, M, K, p->a_bits, p->mode, a_codes, a_scale, a_zp, stream);
    }
    const int B = p->kind == LRQ_ROT_HADAMARD ? p->had_block : 1;
    return lrq_launch_rotq_hadamard(X, M, K, ldx, B, p->a_bits, p->mode, p->prescale, a_codes, a_scale, a_zp, stream);
}

// ---------------------------------------------------------------------------------------------------
// Variant for callers that cannot allocate: the dense rotation's fp32 scratch is this fixed array.
// In host code `g_static_scratch` is only a handle to the symbol; its address on the current device
// comes from cudaGetSymbolAddress.  The address is asked for on every call (a host-side table lookup once
// the module is loaded) rather than cached, so that it stays right after the application resets a device.
// ---------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[LRQ_STATIC_SCRATCH_BYTES];

namespace {
// Device address of the static scratch on the current device (nullptr on failure).
void* static_scratch_address() {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    return ptr;
}
}  // namespace

extern "C" size_t lrq_static_scratch_bytes(void) { return (size_t)LRQ_STATIC_SCRATCH_BYTES; }

extern "C" lrq_status lrq_rotate_quantize_act_static(const void* X, int M, int K, long ldx, const lrq_act_params* p,
                                                     uint8_t* a_codes, float* a_scale, int32_t* a_zp,
                                                     void* cuda_stream) {
    if (!p) return LRQ_ERR_INVALID_ARG;
    if (p->kind != LRQ_ROT_DENSE && p->kind != LRQ_ROT_DUAL)   // no scratch involved: the ordinary path, no workspace
        return lrq_rotate_quantize_act(X, M, K, ldx, p, a_codes, a_scale, a_zp, nullptr, 0, cuda_stream);
    if (M <= 0 || K <= 0) return LRQ_ERR_INVALID_ARG;
    if (lrq_act_workspace_bytes(M, K, p) > (size_t)LRQ_STATIC_SCRATCH_BYTES) return LRQ_ERR_WORKSPACE;
    void* scratch = static_scratch_address();
    if (!scratch) return LRQ_ERR_CUDA;
    return lrq_rotate_quantize_act(X, M, K, ldx, p, a_codes, a_scale, a_zp, scratch, LRQ_STATIC_SCRATCH_BYTES,
                                   cuda_stream);
}

extern "C" lrq_status lrq_ars_select(const void* X, int M, int K, long ldx, double threshold, float* J, int32_t* kind,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!X || !J || !kind || M <= 0 || K <= 0) return LRQ_ERR_INVALID_ARG;
    if (K % 16 || ldx < K || ldx % 16 || !lrq_aligned(X, 32)) return LRQ_ERR_UNSUPPORTED;   // 256-bit loads
    if (!workspace || workspace_bytes < sizeof(double) || !lrq_aligned(workspace, 8)) return LRQ_ERR_WORKSPACE;
    return lrq_launch_ars_metric(X, M, K, ldx, threshold, J, reinterpret_cast<int*>(kind), static_cast<double*>(workspace),
                                 (cudaStream_t)cuda_stream);
}

extern "C" lrq_status lrq_rotate_weights(const float* W, int N, int K, long ldw, const float* colmul, lrq_rot_kind kind,
                                         int had_block, const void* R_bf16, float* W_rot, long ldo, void* cuda_stream) {
    if (!W || !W_rot || N <= 0 || K <= 0 || ldw < K || ldo < K) return LRQ_ERR_INVALID_ARG;
    if (kind == LRQ_ROT_HADAMARD) {
        if (had_block < 1 || (had_block & (had_block - 1)) || K % had_block) return LRQ_ERR_INVALID_ARG;
    } else if (kind == LRQ_ROT_DENSE) {
        if (!R_bf16) return LRQ_ERR_INVALID_ARG;
        if (W_rot == W) return LRQ_ERR_INVALID_ARG;               // the product reads whole rows of W per output tile
    } else if (kind != LRQ_ROT_NONE) {
        return LRQ_ERR_INVALID_ARG;
    }
    return lrq_launch_rotate_weights(W, N, K, ldw, colmul, (int)kind, had_block, R_bf16, W_rot, ldo, (cudaStream_t)cuda_stream);
}

extern "C" lrq_status lrq_rotate_weights_dual(const float* W, int N, int K, long ldw, const float* colmul, int dual_block,
                                              const void* R1_bf16, const int32_t* perm, const void* R2_bf16,
                                              float* W_rot, long ldo, void* cuda_stream) {
    if (!W || !W_rot || !R1_bf16 || !R2_bf16 || !perm || N <= 0 || K <= 0 || ldw < K || ldo < K) return LRQ_ERR_INVALID_ARG;
    if (dual_block < 1 || K % dual_block) return LRQ_ERR_INVALID_ARG;
    return lrq_launch_rotate_weights_dual(W, N, K, ldw, colmul, dual_block, R1_bf16, perm, R2_bf16, W_rot, ldo,
                                          (cudaStream_t)cuda_stream);
}

extern "C" lrq_status lrq_layer_create(lrq_layer** out, int N, int K, int w_bits, int group_size,
                                       lrq_code_layout code_layout, const uint8_t* codes, const float* levels, const float* wsum,
                                       const float* wscale, const float* bias, const lrq_act_params* act) {
    if (!out) return LRQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (!codes || !levels || !wsum || N <= 0 || K <= 0) return LRQ_ERR_INVALID_ARG;
    if (w_bits < 2 || w_bits > 4) return LRQ_ERR_UNSUPPORTED;
    if (code_layout != LRQ_CODES_NIBBLE && code_layout != LRQ_CODES_PACKED3) return LRQ_ERR_INVALID_ARG;
    if (code_layout == LRQ_CODES_PACKED3 && w_bits != 3) return LRQ_ERR_UNSUPPORTED;
    const int G = group_size > 0 ? group_size : K;
    if (K % G || G % 8) return LRQ_ERR_UNSUPPORTED;
    lrq_status st = check_act(act, K);
    if (st != LRQ_OK) return st;
    if (!lrq_aligned(codes, 16) || !lrq_aligned(levels, 16)) return LRQ_ERR_INVALID_ARG;
    lrq_layer* L = new (std::nothrow) lrq_layer;
    if (!L) return LRQ_ERR_INVALID_ARG;
    L->N = N; L->K = K; L->w_bits = w_bits; L->group = G; L->packed3 = code_layout == LRQ_CODES_PACKED3 ? 1 : 0;
    L->codes = codes; L->levels = levels; L->wsum = wsum; L->wscale = wscale; L->bias = bias;
    L->act = *act;
    L->have_tm_w = false;
    lrq_qgemm_tc_prepare(L);          // caches the weight-code TMA descriptors when the shape takes that kernel
    *out = L;
    return LRQ_OK;
}

extern "C" void lrq_layer_destroy(lrq_layer* L) { delete L; }

namespace {
struct WsLayout { size_t codes, scale, zp, rot, total; };
WsLayout ws_layout(const lrq_layer* L, int M) {
    WsLayout w;
    size_t off = 0;
    w.codes = off; off += lrq_round_up((size_t)M * L->K * L->act.a_bits / 8, 256);
    w.scale = off; off += lrq_round_up((size_t)M * sizeof(float), 256);
    w.zp = off;    off += lrq_round_up((size_t)M * sizeof(int32_t), 256);
    w.rot = off;   off += lrq_act_workspace_bytes(M, L->K, &L->act);
    w.total = off;
    return w;
}
}  // namespace

extern "C" size_t lrq_workspace_bytes(const lrq_layer* L, int M) {
    if (!L || M <= 0) return 0;
    return ws_layout(L, M).total;
}

static lrq_status check_out(const void* Y, lrq_dtype dt, long ldy, int N) {
    if (!Y || ldy < N) return LRQ_ERR_INVALID_ARG;
    if (dt != LRQ_F32 && dt != LRQ_F16 && dt != LRQ_BF16) return LRQ_ERR_INVALID_ARG;
    const size_t es = dt == LRQ_F32 ? 4 : 2;
    if (!lrq_aligned(Y, 16) || ((size_t)ldy * es) % 16) return LRQ_ERR_INVALID_ARG;
    return LRQ_OK;
}

// Which contraction kernel a call takes.  impl: 0 large-tile tcgen05, 1 CUDA cores, 2 small-tile tcgen05, 3 CUDA cores
// in the integer shift form, -1 automatic:
// the small-tile kernel for packed 3-bit codes and for batches that give the large-tile kernel fewer tiles than half
// the CTA pairs of the device (a few hundred tokens), the large-tile kernel otherwise, the CUDA cores for shapes
// neither takes.
static lrq_status qgemm_dispatch(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale,
                                 const int32_t* a_zp, int M, void* Y, lrq_dtype dt, long ldy, int impl,
                                 cudaStream_t st) {
    if (impl == 1) return lrq_launch_qgemm_simple(L, a_codes, a_scale, a_zp, M, Y, dt, ldy, st);
    if (impl == 2) return lrq_launch_qgemm_small(L, a_codes, a_scale, a_zp, M, Y, dt, ldy, st);
    if (impl == 3) return lrq_launch_qgemm_shift(L, a_codes, a_scale, a_zp, M, Y, dt, ldy, st);
    if (impl == 0) return lrq_launch_qgemm_tc(L, a_codes, a_scale, a_zp, M, Y, dt, ldy, st);
    lrq_status s = LRQ_ERR_UNSUPPORTED;
    if (lrq_qgemm_small_takes(L)) {
        int sms = 0;
        if (lrq_current_device(nullptr, &sms) != LRQ_OK) return LRQ_ERR_CUDA;
        const long narrow_tiles = (long)((M + 255) / 256) * ((L->N + 127) / 128);
        if (L->packed3 || narrow_tiles * 4 < sms) s = lrq_launch_qgemm_small(L, a_codes, a_scale, a_zp, M, Y, dt, ldy, st);
    }
    if (s == LRQ_ERR_UNSUPPORTED) s = lrq_launch_qgemm_tc(L, a_codes, a_scale, a_zp, M, Y, dt, ldy, st);
    if (s == LRQ_ERR_UNSUPPORTED) s = lrq_launch_qgemm_simple(L, a_codes, a_scale, a_zp, M, Y, dt, ldy, st);
    return s;
}

extern "C" lrq_status lrq_qgemm_codes(const lrq_layer* L, const uint8_t* a_codes, const float* a_scale,
                                      const int32_t* a_zp, int M, void* Y, lrq_dtype dt, long ldy, int impl,
                                      void* cuda_stream) {
    if (!L || !a_codes || !a_scale || !a_zp || M <= 0) return LRQ_ERR_INVALID_ARG;
    if (impl < 0 || impl > 3) return LRQ_ERR_INVALID_ARG;
    lrq_status st = check_out(Y, dt, ldy, L->N);
    if (st != LRQ_OK) return st;
    if (!lrq_aligned(a_codes, 16)) return LRQ_ERR_INVALID_ARG;
    return qgemm_dispatch(L, a_codes, a_scale, a_zp, M, Y, dt, ldy, impl, (cudaStream_t)cuda_stream);
}

// Every check lrq_qlinear makes on one layer's arguments; nothing is launched here.
static lrq_status validate_layer_call(const lrq_layer* L, const void* X, int M, long ldx, const void* Y, lrq_dtype dt,
                                      long ldy, const void* workspace, size_t workspace_bytes) {
    if (!L || !X || M <= 0) return LRQ_ERR_INVALID_ARG;
    lrq_status st = check_out(Y, dt, ldy, L->N);
    if (st != LRQ_OK) return st;
    if (ldx < L->K || (ldx % 8) || !lrq_aligned(X, 16)) return LRQ_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < ws_layout(L, M).total || !lrq_aligned(workspace, 256)) return LRQ_ERR_WORKSPACE;
    return LRQ_OK;
}

extern "C" lrq_status lrq_qlinear(const lrq_layer* L, const void* X, int M, long ldx, void* Y, lrq_dtype dt, long ldy,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream) {
    lrq_status st = validate_layer_call(L, X, M, ldx, Y, dt, ldy, workspace, workspace_bytes);
    if (st != LRQ_OK) return st;
    const WsLayout w = ws_layout(L, M);
    char* base = static_cast<char*>(workspace);
    uint8_t* a_codes = reinterpret_cast<uint8_t*>(base + w.codes);
    float* a_scale = reinterpret_cast<float*>(base + w.scale);
    int32_t* a_zp = reinterpret_cast<int32_t*>(base + w.zp);
    st = lrq_rotate_quantize_act(X, M, L->K, ldx, &L->act, a_codes, a_scale, a_zp, base + w.rot,
                                 w.total - w.rot, cuda_stream);
    if (st != LRQ_OK) return st;
    return qgemm_dispatch(L, a_codes, a_scale, a_zp, M, Y, dt, ldy, -1, (cudaStream_t)cuda_stream);
}

extern "C" lrq_status lrq_qlinear_stack(const lrq_layer* const* layers, int n_layers, const void* const* X,
                                        const int* M, const long* ldx, void* const* Y, lrq_dtype dt,
                                        const long* ldy, void* workspace, size_t workspace_bytes,
                                        void* cuda_stream) {
    if (!layers || !X || !M || !ldx || !Y || !ldy || n_layers <= 0) return LRQ_ERR_INVALID_ARG;
    // every layer's arguments are validated before the first launch
    for (int i = 0; i < n_layers; ++i) {
        lrq_status st = validate_layer_call(layers[i], X[i], M[i], ldx[i], Y[i], dt, ldy[i], workspace, workspace_bytes);
        if (st != LRQ_OK) return st;
    }
    for (int i = 0; i < n_layers; ++i) {
        lrq_status st = lrq_qlinear(layers[i], X[i], M[i], ldx[i], Y[i], dt, ldy[i], workspace, workspace_bytes,
                                    cuda_stream);
        if (st != LRQ_OK) return st;
    }
    return LRQ_OK;
}

extern "C" int lrq_device_status(void* cuda_stream) {
    int* w = lrq_status_word();
    if (!w) return -1;
    int v = 0;
    if (cudaMemcpyAsync(&v, w, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)cuda_stream) != cudaSuccess) return -1;
    if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return -1;
    if (v) cudaMemsetAsync(w, 0, sizeof(int), (cudaStream_t)cuda_stream);
    return v;
}

extern "C" const char* lrq_status_string(lrq_status s) {
    switch (s) {
        case LRQ_OK: return "ok";
        case LRQ_ERR_INVALID_ARG: return "invalid argument";
        case LRQ_ERR_UNSUPPORTED: return "unsupported configuration";
        case LRQ_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case LRQ_ERR_CUDA: return "CUDA call failed";
        case LRQ_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown";
}

extern "C" int lrq_version(void) { return 100; }
