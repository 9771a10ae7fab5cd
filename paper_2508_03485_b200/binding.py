"""ctypes binding of ``include/lrq.h``.  Argument marshalling only; torch supplies device memory
and streams.  Function names are those of the C ABI."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIBPATH = os.path.join(_HERE, "liblrq_b200.so")

ROT_NONE, ROT_HADAMARD, ROT_DENSE, ROT_DUAL = 0, 1, 2, 3
ACT_ASYM, ACT_SYM = 0, 1
F32, F16, BF16 = 0, 1, 2
CODES_NIBBLE, CODES_PACKED3 = 0, 1
_TORCH_DT = {F32: torch.float32, F16: torch.float16, BF16: torch.bfloat16}

EXPORTS = [
    "lrq_tlq_quantize_weights", "lrq_act_workspace_bytes", "lrq_rotate_quantize_act", "lrq_layer_create",
    "lrq_layer_destroy", "lrq_workspace_bytes", "lrq_qlinear", "lrq_qlinear_stack", "lrq_qgemm_codes",
    "lrq_device_status", "lrq_status_string", "lrq_version", "lrq_rotate_quantize_act_static", "lrq_ars_select",
    "lrq_rotate_weights", "lrq_selftest_wait_timeout", "lrq_static_scratch_bytes", "lrq_rotate_weights_dual",
]


class LrqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = load_library().lrq_status_string(code).decode()
        super().__init__(f"{where}: {msg} (status {code})")


class _TlqParams(C.Structure):
    _fields_ = [("w_bits", C.c_int), ("group_size", C.c_int), ("integerize_I", C.c_int),
                ("n_alpha", C.c_int), ("n_beta", C.c_int),
                ("alpha", C.POINTER(C.c_double)), ("beta", C.POINTER(C.c_double)), ("code_layout", C.c_int)]


class _ActParams(C.Structure):
    _fields_ = [("kind", C.c_int), ("had_block", C.c_int), ("R_bf16", C.c_void_p),
                ("a_bits", C.c_int), ("mode", C.c_int), ("prescale", C.c_void_p),
                ("dual_block", C.c_int), ("R1_bf16", C.c_void_p), ("perm", C.c_void_p), ("R2_bf16", C.c_void_p)]


_lib = None


def load_library() -> C.CDLL:
    """Load ``liblrq_b200.so`` (built in-tree by ``paper_2508_03485_b200/build.py``).  Raises if it is
    missing: there is no other implementation to fall back to."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIBPATH):
        raise RuntimeError(f"{_LIBPATH} not found: build it with `python -m paper_2508_03485_b200.build` "
                           "(nvcc, sm_100a); there is no CPU fallback")
    lib = C.CDLL(_LIBPATH)
    vp, ci, cl, sz = C.c_void_p, C.c_int, C.c_long, C.c_size_t
    lib.lrq_tlq_quantize_weights.argtypes = [vp, ci, ci, C.POINTER(_TlqParams), vp, vp, vp, vp, vp, sz, vp]
    lib.lrq_act_workspace_bytes.argtypes = [ci, ci, C.POINTER(_ActParams)]
    lib.lrq_act_workspace_bytes.restype = sz
    lib.lrq_rotate_quantize_act.argtypes = [vp, ci, ci, cl, C.POINTER(_ActParams), vp, vp, vp, vp, sz, vp]
    lib.lrq_rotate_quantize_act_static.argtypes = [vp, ci, ci, cl, C.POINTER(_ActParams), vp, vp, vp, vp]
    lib.lrq_layer_create.argtypes = [C.POINTER(vp), ci, ci, ci, ci, ci, vp, vp, vp, vp, vp, C.POINTER(_ActParams)]
    lib.lrq_layer_destroy.argtypes = [vp]
    lib.lrq_layer_destroy.restype = None
    lib.lrq_workspace_bytes.argtypes = [vp, ci]
    lib.lrq_workspace_bytes.restype = sz
    lib.lrq_qlinear.argtypes = [vp, vp, ci, cl, vp, ci, cl, vp, sz, vp]
    lib.lrq_qlinear_stack.argtypes = [C.POINTER(vp), ci, C.POINTER(vp), C.POINTER(ci), C.POINTER(cl),
                                      C.POINTER(vp), ci, C.POINTER(cl), vp, sz, vp]
    lib.lrq_qgemm_codes.argtypes = [vp, vp, vp, vp, ci, vp, ci, cl, ci, vp]
    lib.lrq_ars_select.argtypes = [vp, ci, ci, cl, C.c_double, vp, vp, vp, sz, vp]
    lib.lrq_rotate_weights.argtypes = [vp, ci, ci, cl, vp, ci, ci, vp, vp, cl, vp]
    lib.lrq_rotate_weights_dual.argtypes = [vp, ci, ci, cl, vp, ci, vp, vp, vp, vp, cl, vp]
    lib.lrq_device_status.argtypes = [vp]
    lib.lrq_selftest_wait_timeout.argtypes = [C.c_longlong, vp]
    lib.lrq_status_string.argtypes = [ci]
    lib.lrq_status_string.restype = C.c_char_p
    lib.lrq_static_scratch_bytes.argtypes = []
    lib.lrq_static_scratch_bytes.restype = sz
    for name in EXPORTS:
        getattr(lib, name)
    _lib = lib
    return lib


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _ptr(t: Optional[torch.Tensor]) -> C.c_void_p:
    return C.c_void_p(0 if t is None else t.data_ptr())


def _check(code: int, where: str):
    if code != 0:
        raise LrqError(code, where)


def _need_cuda(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise ValueError("device tensors required (there is no CPU path)")


def lrq_version() -> int:
    return int(load_library().lrq_version())


def lrq_device_status(stream=None) -> int:
    return int(load_library().lrq_device_status(_stream(stream)))


def lrq_selftest_wait_timeout(limit_cycles: int = 100000, stream=None) -> None:
    """Launch the diagnostic kernel whose bounded wait runs out; lrq_device_status() then returns SELFTEST_WAIT_CODE once."""
    _check(load_library().lrq_selftest_wait_timeout(int(limit_cycles), _stream(stream)), "lrq_selftest_wait_timeout")


SELFTEST_WAIT_CODE = 99


def lrq_static_scratch_bytes() -> int:
    """Size of the fixed scratch array behind lrq_rotate_quantize_act_static, as built into the library."""
    return int(load_library().lrq_static_scratch_bytes())


# ------------------------------------------------------------------------------------------------
@dataclass
class TLQWeights:
    codes: torch.Tensor    # uint8 [N, K/2] (nibbles) or [N, 3K/8] (packed 3-bit)
    levels: torch.Tensor   # float32 [N, K/G, 2^b]
    meta: torch.Tensor     # float64 [N, K/G, 6]
    wsum: torch.Tensor     # float32 [N]
    w_bits: int
    group: int             # 0 = per output channel
    code_layout: int = CODES_NIBBLE


def lrq_tlq_quantize_weights(W_rot: torch.Tensor, w_bits: int, group_size: int = 0, integerize_I: int = 7,
                             alpha: Sequence[float] = (1.0,), beta: Sequence[float] = (1.0,),
                             stream=None, code_layout: int = CODES_NIBBLE) -> TLQWeights:
    """TLQ weight quantization (Sec. 4.1, Eqs. 4-9) of a device float32 [N,K] matrix."""
    _need_cuda(W_rot)
    assert W_rot.dtype == torch.float32 and W_rot.is_contiguous() and W_rot.dim() == 2
    N, K = W_rot.shape
    G = K if group_size <= 0 else group_size
    dev = W_rot.device
    codes = torch.empty((N, 3 * K // 8 if code_layout == CODES_PACKED3 else K // 2), dtype=torch.uint8, device=dev)
    levels = torch.empty((N, max(1, K // max(G, 1)), 1 << w_bits), dtype=torch.float32, device=dev)
    meta = torch.empty((N, max(1, K // max(G, 1)), 6), dtype=torch.float64, device=dev)
    wsum = torch.empty((N,), dtype=torch.float32, device=dev)
    a = (C.c_double * len(alpha))(*[float(v) for v in alpha])
    b = (C.c_double * len(beta))(*[float(v) for v in beta])
    p = _TlqParams(int(w_bits), int(group_size), int(integerize_I), len(alpha), len(beta),
                   C.cast(a, C.POINTER(C.c_double)), C.cast(b, C.POINTER(C.c_double)), int(code_layout))
    rc = load_library().lrq_tlq_quantize_weights(_ptr(W_rot), N, K, C.byref(p), _ptr(codes), _ptr(levels),
                                                 _ptr(meta), _ptr(wsum), None, 0, _stream(stream))
    _check(rc, "lrq_tlq_quantize_weights")
    return TLQWeights(codes, levels, meta, wsum, int(w_bits), int(group_size), int(code_layout))


@dataclass
class DualRotation:
    """The dual transformation of Sec. 4.2 in its factors, y = x . blockdiag(R1) . P . blockdiag(R2)."""
    block: int             # Bd
    R1: torch.Tensor       # bfloat16 [K/Bd, Bd, Bd]
    perm: torch.Tensor     # int32 [K]: position i takes channel perm[i]
    R2: torch.Tensor       # bfloat16 [K/Bd, Bd, Bd]

    def check(self, K: int):
        nb = K // self.block
        for R in (self.R1, self.R2):
            assert R.is_cuda and R.dtype == torch.bfloat16 and R.shape == (nb, self.block, self.block) and R.is_contiguous()
        assert self.perm.is_cuda and self.perm.dtype == torch.int32 and self.perm.shape == (K,) and self.perm.is_contiguous()


def _act_params(kind: int, had_block: int, R: Optional[torch.Tensor], a_bits: int, mode: int,
                prescale: Optional[torch.Tensor] = None, dual: Optional[DualRotation] = None) -> _ActParams:
    if prescale is not None:
        assert prescale.dtype == torch.float32 and prescale.is_contiguous()
    p = _ActParams(int(kind), int(had_block), 0 if R is None else R.data_ptr(), int(a_bits), int(mode),
                   0 if prescale is None else prescale.data_ptr(), 0, 0, 0, 0)
    if dual is not None:
        p.dual_block, p.R1_bf16, p.perm, p.R2_bf16 = int(dual.block), dual.R1.data_ptr(), dual.perm.data_ptr(), dual.R2.data_ptr()
    return p


def lrq_rotate_weights_dual(W: torch.Tensor, dual: DualRotation, colmul: Optional[torch.Tensor] = None, stream=None,
                            out: Optional[torch.Tensor] = None):
    """W diag(colmul) R1hat P R2hat in fp64, rounded to fp32: the weight side of Eq. 2 for a layer whose rotation is kept
    in the factors of the dual transformation.  Returns W_rot float32 [N,K]."""
    _need_cuda(W)
    assert W.dtype == torch.float32 and W.dim() == 2 and W.stride(1) == 1
    N, K = W.shape
    dual.check(K)
    if colmul is not None:
        assert colmul.dtype == torch.float32 and colmul.shape == (K,) and colmul.is_contiguous()
    if out is None:
        out = torch.empty((N, K), dtype=torch.float32, device=W.device)
    assert out.dtype == torch.float32 and out.shape == (N, K) and out.stride(1) == 1
    _check(load_library().lrq_rotate_weights_dual(_ptr(W), N, K, W.stride(0), _ptr(colmul), dual.block, _ptr(dual.R1),
                                                  _ptr(dual.perm), _ptr(dual.R2), _ptr(out), out.stride(0),
                                                  _stream(stream)), "lrq_rotate_weights_dual")
    return out


def lrq_rotate_weights(W: torch.Tensor, kind: int, had_block: int = 0, R: Optional[torch.Tensor] = None,
                       colmul: Optional[torch.Tensor] = None, stream=None, out: Optional[torch.Tensor] = None):
    """W diag(colmul) R in fp64, rounded to fp32: the weight side of Eq. 2 (offline).  Returns W_rot float32 [N,K]."""
    _need_cuda(W)
    assert W.dtype == torch.float32 and W.dim() == 2 and W.stride(1) == 1
    N, K = W.shape
    if R is not None:
        assert R.dtype == torch.bfloat16 and R.shape == (K, K) and R.is_contiguous()
    if colmul is not None:
        assert colmul.dtype == torch.float32 and colmul.shape == (K,) and colmul.is_contiguous()
    if out is None:
        out = torch.empty((N, K), dtype=torch.float32, device=W.device)
    assert out.dtype == torch.float32 and out.shape == (N, K) and out.stride(1) == 1
    _check(load_library().lrq_rotate_weights(_ptr(W), N, K, W.stride(0), _ptr(colmul), kind, had_block, _ptr(R), _ptr(out),
                                             out.stride(0), _stream(stream)), "lrq_rotate_weights")
    return out


def lrq_ars_select(X: torch.Tensor, threshold: float = 1.0, stream=None):
    """Fluctuation metric J of calibration activations and the rotation kind it selects (Eqs. 11-12).
    Returns (J float32[1], kind int32[1]) device tensors."""
    _need_cuda(X)
    assert X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    M, K = X.shape
    J = torch.empty(1, dtype=torch.float32, device=X.device)
    kind = torch.empty(1, dtype=torch.int32, device=X.device)
    ws = torch.empty(1, dtype=torch.float64, device=X.device)
    rc = load_library().lrq_ars_select(_ptr(X), M, K, X.stride(0), float(threshold), _ptr(J), _ptr(kind), _ptr(ws), 8,
                                       _stream(stream))
    _check(rc, "lrq_ars_select")
    return J, kind


def lrq_rotate_quantize_act(X: torch.Tensor, kind: int, a_bits: int, had_block: int = 0,
                            R: Optional[torch.Tensor] = None, mode: int = ACT_ASYM,
                            workspace: Optional[torch.Tensor] = None, stream=None, out=None,
                            prescale: Optional[torch.Tensor] = None, dual: Optional[DualRotation] = None):
    """Rotation + per-token quantization (Eq. 12, Eq. 1) of device bf16 [M,K] activations.
    Returns (codes uint8, scale float32 [M], zero_point int32 [M])."""
    _need_cuda(X, R, workspace, prescale)
    assert X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    M, K = X.shape
    lib = load_library()
    if dual is not None:
        dual.check(K)
    p = _act_params(kind, had_block, R, a_bits, mode, prescale, dual)
    need = int(lib.lrq_act_workspace_bytes(M, K, C.byref(p)))
    if need and (workspace is None or workspace.numel() * workspace.element_size() < need):
        workspace = torch.empty(need, dtype=torch.uint8, device=X.device)
    dev = X.device
    if out is not None:
        codes, scale, zp = out
        assert codes.numel() == M * K * a_bits // 8 and scale.numel() == M and zp.numel() == M
    else:
        codes = torch.empty((M, K * a_bits // 8), dtype=torch.uint8, device=dev)
        scale = torch.empty((M,), dtype=torch.float32, device=dev)
        zp = torch.empty((M,), dtype=torch.int32, device=dev)
    wsb = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.lrq_rotate_quantize_act(_ptr(X), M, K, X.stride(0), C.byref(p), _ptr(codes), _ptr(scale), _ptr(zp),
                                     _ptr(workspace), wsb, _stream(stream))
    _check(rc, "lrq_rotate_quantize_act")
    return codes, scale, zp


def lrq_rotate_quantize_act_static(X: torch.Tensor, kind: int, a_bits: int, had_block: int = 0,
                                   R: Optional[torch.Tensor] = None, mode: int = ACT_ASYM, stream=None, out=None,
                                   dual: Optional[DualRotation] = None):
    """lrq_rotate_quantize_act for callers that cannot provide device scratch (a host that may not call
    cudaMalloc once it is running, or whose memory is planned by another runtime): the dense rotation's
    scratch is a fixed array of lrq_static_scratch_bytes() bytes inside the library.  ``out`` (codes, scale, zero_point)
    lets such a caller pass its own pre-planned result buffers; without it this wrapper allocates them with
    torch, the C entry point itself never allocates.  Raises LrqError (workspace) when M*K*4 exceeds the array."""
    _need_cuda(X, R)
    assert X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    M, K = X.shape
    if out is not None:
        codes, scale, zp = out
    else:
        codes = torch.empty((M, K * a_bits // 8), dtype=torch.uint8, device=X.device)
        scale = torch.empty((M,), dtype=torch.float32, device=X.device)
        zp = torch.empty((M,), dtype=torch.int32, device=X.device)
    if dual is not None:
        dual.check(K)
    p = _act_params(kind, had_block, R, a_bits, mode, None, dual)
    rc = load_library().lrq_rotate_quantize_act_static(_ptr(X), M, K, X.stride(0), C.byref(p), _ptr(codes),
                                                       _ptr(scale), _ptr(zp), _stream(stream))
    _check(rc, "lrq_rotate_quantize_act_static")
    return codes, scale, zp


class QLayer:
    """Owner of one ``lrq_layer`` handle and of the device tensors it points to."""

    def __init__(self, tlq: TLQWeights, N: int, K: int, kind: int, a_bits: int, had_block: int = 0,
                 R: Optional[torch.Tensor] = None, mode: int = ACT_ASYM,
                 wscale: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                 prescale: Optional[torch.Tensor] = None, dual: Optional[DualRotation] = None):
        _need_cuda(tlq.codes, tlq.levels, tlq.wsum, R, wscale, bias, prescale)
        if dual is not None:
            dual.check(K)
        self.prescale, self.dual = prescale, dual
        self.tlq, self.N, self.K, self.R, self.wscale, self.bias = tlq, N, K, R, wscale, bias
        self.kind, self.a_bits, self.had_block, self.mode = kind, a_bits, had_block, mode
        self._p = _act_params(kind, had_block, R, a_bits, mode, prescale, dual)
        h = C.c_void_p()
        rc = load_library().lrq_layer_create(C.byref(h), N, K, tlq.w_bits, tlq.group, tlq.code_layout, _ptr(tlq.codes),
                                             _ptr(tlq.levels), _ptr(tlq.wsum), _ptr(wscale), _ptr(bias),
                                             C.byref(self._p))
        _check(rc, "lrq_layer_create")
        self.handle = h

    def workspace_bytes(self, M: int) -> int:
        return int(load_library().lrq_workspace_bytes(self.handle, int(M)))

    def close(self):
        if getattr(self, "handle", None):
            load_library().lrq_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _ws(workspace: Optional[torch.Tensor], need: int, device) -> torch.Tensor:
    if workspace is None or workspace.numel() * workspace.element_size() < need:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=device)
    return workspace


def lrq_qlinear(layer: QLayer, X: torch.Tensor, y_dtype: int = F32, out: Optional[torch.Tensor] = None,
                workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Y = quantized-linear(X) for device bf16 X [M,K] (Eq. 12 -> Eq. 1 -> Eq. 10 -> scaling)."""
    _need_cuda(X, out, workspace)
    assert X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1 and X.shape[1] == layer.K
    M = X.shape[0]
    if out is None:
        out = torch.empty((M, layer.N), dtype=_TORCH_DT[y_dtype], device=X.device)
    assert out.dtype == _TORCH_DT[y_dtype] and out.stride(1) == 1
    workspace = _ws(workspace, layer.workspace_bytes(M), X.device)
    rc = load_library().lrq_qlinear(layer.handle, _ptr(X), M, X.stride(0), _ptr(out), y_dtype, out.stride(0),
                                    _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream))
    _check(rc, "lrq_qlinear")
    return out


class StackPlan:
    """Host-side argument arrays of one lrq_qlinear_stack call, built once and reused."""

    def __init__(self, layers: List[QLayer], Xs: List[torch.Tensor], Ys: List[torch.Tensor], y_dtype: int):
        n = len(layers)
        vp = C.c_void_p
        self.n, self.y_dtype = n, y_dtype
        self.layers = (vp * n)(*[l.handle for l in layers])
        self.X = (vp * n)(*[x.data_ptr() for x in Xs])
        self.Y = (vp * n)(*[y.data_ptr() for y in Ys])
        self.M = (C.c_int * n)(*[x.shape[0] for x in Xs])
        self.ldx = (C.c_long * n)(*[x.stride(0) for x in Xs])
        self.ldy = (C.c_long * n)(*[y.stride(0) for y in Ys])
        self.need = max(l.workspace_bytes(x.shape[0]) for l, x in zip(layers, Xs))
        self._keep = (layers, Xs, Ys)


def lrq_qlinear_stack(plan: StackPlan, workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    """All layers of ``plan`` back to back on one stream, one shared workspace."""
    dev = plan._keep[1][0].device
    workspace = _ws(workspace, plan.need, dev)
    rc = load_library().lrq_qlinear_stack(plan.layers, plan.n, plan.X, plan.M, plan.ldx, plan.Y, plan.y_dtype,
                                          plan.ldy, _ptr(workspace), workspace.numel() * workspace.element_size(),
                                          _stream(stream))
    _check(rc, "lrq_qlinear_stack")


def lrq_qgemm_codes(layer: QLayer, a_codes: torch.Tensor, a_scale: torch.Tensor, a_zp: torch.Tensor,
                    y_dtype: int = F32, impl: int = 0, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Contraction + epilogue alone (Eq. 10) on codes from lrq_rotate_quantize_act.
    impl 0: large-tile tcgen05 kernel, 1: CUDA-core baseline, 2: small-tile tcgen05 kernel (the only tensor-core kernel for
    packed 3-bit codes), 3: the integer shift form of Eq. 10 on the CUDA cores (exact sums; a slow cross-check)."""
    _need_cuda(a_codes, a_scale, a_zp, out)
    M = a_codes.shape[0]
    if out is None:
        out = torch.empty((M, layer.N), dtype=_TORCH_DT[y_dtype], device=a_codes.device)
    rc = load_library().lrq_qgemm_codes(layer.handle, _ptr(a_codes), _ptr(a_scale), _ptr(a_zp), M, _ptr(out),
                                        y_dtype, out.stride(0), impl, _stream(stream))
    _check(rc, "lrq_qgemm_codes")
    return out
