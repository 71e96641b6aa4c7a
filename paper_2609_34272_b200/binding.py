"""ctypes binding of the C ABI in ``include/gproj_attn.h`` (argument marshalling only).

Every step of the attention path runs in the CUDA library; PyTorch supplies device
memory and the stream.  There is no CPU fallback: if the library is missing or the
device is not sm_100a the calls raise.
"""
import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libgproj_attn.so")

GPROJ_OK = 0
FLAG_NO_Q_CORRECTION = 1
FLAG_NO_K_CORRECTION = 2
FLAG_ONLY_DQ_PASS = 4
FLAG_ONLY_DKV_PASS = 8
FWD_FLAG_FMA_SOFTMAX = 1

STATIC_SCRATCH_BYTES = 16 << 20

EXPORTS = ("gproj_attn_fwd", "gproj_attn_bwd_workspace_bytes", "gproj_attn_bwd", "gproj_attn_fwd_gqa", "gproj_attn_bwd_gqa", "gproj_attn_fwd_ex",
           "gproj_attn_bwd_static_scratch", "gproj_attn_fwd_rect", "gproj_attn_bwd_rect",
           "gproj_attn_varlen_plan_bytes", "gproj_attn_varlen_plan", "gproj_attn_fwd_varlen",
           "gproj_attn_bwd_varlen_workspace_bytes", "gproj_attn_bwd_varlen",
           "gproj_attn_varlen_qk_plan_bytes", "gproj_attn_varlen_qk_plan", "gproj_attn_fwd_varlen_qk", "gproj_attn_bwd_varlen_qk",
           "gproj_attn_host_staging_bytes", "gproj_attn_fwd_bwd_host", "gproj_key_smooth", "gproj_key_smooth_varlen",
           "gproj_fp32_attn_saved_bytes", "gproj_fp32_attn_fwd", "gproj_fp32_attn_bwd",
           "gproj_last_device_status", "gproj_selftest_wait_timeout",
           "gproj_status_string", "gproj_last_launch_count")

_lib = None


class GprojError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def load():
    """Load the shared library (no CUDA call is made by loading)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -c 'import __graft_entry__ as g; g.build()'` "
                               "(there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i, f, u, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_uint, ctypes.c_size_t
        lib.gproj_attn_fwd.restype = i
        lib.gproj_attn_fwd.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, f, i, vp]
        lib.gproj_attn_bwd_workspace_bytes.restype = sz
        lib.gproj_attn_bwd_workspace_bytes.argtypes = [i, i, i, i]
        lib.gproj_attn_bwd.restype = i
        lib.gproj_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, i, f, i, vp, sz, u, vp]
        lib.gproj_attn_fwd_gqa.restype = i
        lib.gproj_attn_fwd_gqa.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, f, i, vp]
        lib.gproj_attn_fwd_ex.restype = i
        lib.gproj_attn_fwd_ex.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, f, i, u, vp]
        lib.gproj_attn_bwd_gqa.restype = i
        lib.gproj_attn_bwd_gqa.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, f, i, vp, sz, u, vp]
        lib.gproj_attn_fwd_rect.restype = i
        lib.gproj_attn_fwd_rect.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, f, i, u, vp]
        lib.gproj_attn_bwd_rect.restype = i
        lib.gproj_attn_bwd_rect.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, f, i, vp, sz, u, vp]
        lib.gproj_attn_bwd_static_scratch.restype = i
        lib.gproj_attn_bwd_static_scratch.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, i, f, i, u, vp]
        ip = ctypes.POINTER(ctypes.c_int)
        lib.gproj_attn_varlen_plan_bytes.restype = ctypes.c_size_t
        lib.gproj_attn_varlen_plan_bytes.argtypes = [ip, i]
        lib.gproj_attn_varlen_plan.restype = i
        lib.gproj_attn_varlen_plan.argtypes = [ip, i, i, vp, ctypes.c_size_t]
        lib.gproj_attn_fwd_varlen.restype = i
        lib.gproj_attn_fwd_varlen.argtypes = [vp, vp, vp, vp, vp, ip, i, vp, i, i, i, f, i, u, vp]
        lib.gproj_attn_bwd_varlen_workspace_bytes.restype = ctypes.c_size_t
        lib.gproj_attn_bwd_varlen_workspace_bytes.argtypes = [ip, i, i, i]
        lib.gproj_attn_bwd_varlen.restype = i
        lib.gproj_attn_bwd_varlen.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, ip, i, vp, i, i, i, f, i, vp, ctypes.c_size_t, u, vp]
        lib.gproj_attn_varlen_qk_plan_bytes.restype = ctypes.c_size_t
        lib.gproj_attn_varlen_qk_plan_bytes.argtypes = [ip, ip, i]
        lib.gproj_attn_varlen_qk_plan.restype = i
        lib.gproj_attn_varlen_qk_plan.argtypes = [ip, ip, i, i, vp, ctypes.c_size_t]
        lib.gproj_attn_fwd_varlen_qk.restype = i
        lib.gproj_attn_fwd_varlen_qk.argtypes = [vp, vp, vp, vp, vp, ip, ip, i, vp, i, i, i, f, i, u, vp]
        lib.gproj_attn_bwd_varlen_qk.restype = i
        lib.gproj_attn_bwd_varlen_qk.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, ip, ip, i, vp, i, i, i, f, i, vp, ctypes.c_size_t, u, vp]
        lib.gproj_attn_host_staging_bytes.restype = ctypes.c_size_t
        lib.gproj_attn_host_staging_bytes.argtypes = [i, i, i, i, i]
        lib.gproj_attn_fwd_bwd_host.restype = i
        lib.gproj_attn_fwd_bwd_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, f, i, vp, ctypes.c_size_t, u, vp]
        lib.gproj_fp32_attn_saved_bytes.restype = sz
        lib.gproj_fp32_attn_saved_bytes.argtypes = [i, i, i, i]
        lib.gproj_fp32_attn_fwd.restype = i
        lib.gproj_fp32_attn_fwd.argtypes = [vp, vp, vp, vp, vp, sz, i, i, i, i, f, i, vp]
        lib.gproj_fp32_attn_bwd.restype = i
        lib.gproj_fp32_attn_bwd.argtypes = [vp, vp, vp, vp, vp, sz, vp, vp, vp, i, i, i, i, f, i, vp]
        lib.gproj_key_smooth.restype = i
        lib.gproj_key_smooth.argtypes = [vp, vp, i, i, i, i, vp]
        lib.gproj_key_smooth_varlen.restype = i
        lib.gproj_key_smooth_varlen.argtypes = [vp, vp, ip, i, i, i, vp]
        lib.gproj_selftest_wait_timeout.restype = i
        lib.gproj_selftest_wait_timeout.argtypes = [vp]
        lib.gproj_last_device_status.restype = i
        lib.gproj_last_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int)]
        lib.gproj_status_string.restype = ctypes.c_char_p
        lib.gproj_status_string.argtypes = [i]
        lib.gproj_last_launch_count.restype = i
        lib.gproj_last_launch_count.argtypes = []
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().gproj_status_string(int(status)).decode()


def _check_bf16(name, t, shape=None):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA bfloat16 tensor")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} has shape {tuple(t.shape)}, expected {tuple(shape)}")


def _kv_heads(Q, K):
    B, H, N, d = Q.shape
    if K.dim() != 4 or K.shape[0] != B or K.shape[2] != N or K.shape[3] != d or H % K.shape[1] != 0:
        raise ValueError(f"K/V shape {tuple(K.shape)} does not match Q {tuple(Q.shape)} (need [B, Hkv, N, d], H % Hkv == 0)")
    return K.shape[1]


def _stream(device):
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def gproj_attn_bwd_workspace_bytes(B, H, N, d) -> int:
    return int(load().gproj_attn_bwd_workspace_bytes(B, H, N, d))


def gproj_attn_fwd(Q, K, V, softmax_scale, causal, O=None, LSE=None, fwd_flags=0):
    """O, LSE = attention forward.  Q: CUDA bfloat16 [B, H, N, d]; K, V: [B, Hkv, N, d] with H a multiple of Hkv
    (Hkv < H = grouped-query attention)."""
    _check_bf16("Q", Q)
    B, H, N, d = Q.shape
    _check_bf16("K", K); _check_bf16("V", V, K.shape)
    Hkv = _kv_heads(Q, K)
    if O is None:
        O = torch.empty_like(Q)
    if LSE is None:
        LSE = torch.empty((B, H, N), dtype=torch.float32, device=Q.device)
    _check_bf16("O", O, Q.shape)
    with torch.cuda.device(Q.device):
        if fwd_flags:
            rc = load().gproj_attn_fwd_ex(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(), B, H, Hkv, N, d,
                                          float(softmax_scale), int(bool(causal)), int(fwd_flags), _stream(Q.device))
        elif Hkv == H:
            rc = load().gproj_attn_fwd(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(),
                                       B, H, N, d, float(softmax_scale), int(bool(causal)), _stream(Q.device))
        else:
            rc = load().gproj_attn_fwd_gqa(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(),
                                           B, H, Hkv, N, d, float(softmax_scale), int(bool(causal)), _stream(Q.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_attn_fwd")
    return O, LSE


def gproj_attn_bwd(Q, K, V, O, LSE, dO, softmax_scale, causal, flags=0, workspace=None, dQ=None, dK=None, dV=None):
    """dQ, dK, dV = attention backward with the GProj correction (flags: FLAG_NO_*_CORRECTION).
    K, V (and dK, dV) may have fewer heads than Q (grouped-query attention)."""
    _check_bf16("Q", Q)
    B, H, N, d = Q.shape
    _check_bf16("K", K); _check_bf16("V", V, K.shape)
    Hkv = _kv_heads(Q, K)
    for name, t in (("O", O), ("dO", dO)):
        _check_bf16(name, t, Q.shape)
    if not (LSE.is_cuda and LSE.dtype == torch.float32 and LSE.is_contiguous() and tuple(LSE.shape) == (B, H, N)):
        raise TypeError("LSE must be a contiguous CUDA float32 tensor [B, H, N]")
    need = gproj_attn_bwd_workspace_bytes(B, H, N, d)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=Q.device)
    dQ = torch.empty_like(Q) if dQ is None else dQ
    dK = torch.empty_like(K) if dK is None else dK
    dV = torch.empty_like(K) if dV is None else dV
    _check_bf16("dQ", dQ, Q.shape); _check_bf16("dK", dK, K.shape); _check_bf16("dV", dV, K.shape)
    with torch.cuda.device(Q.device):
        if Hkv == H:
            rc = load().gproj_attn_bwd(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(), dO.data_ptr(),
                                       dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), B, H, N, d, float(softmax_scale),
                                       int(bool(causal)), workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                       int(flags), _stream(Q.device))
        else:
            rc = load().gproj_attn_bwd_gqa(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(),
                                           dO.data_ptr(), dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), B, H, Hkv, N, d,
                                           float(softmax_scale), int(bool(causal)), workspace.data_ptr(),
                                           workspace.numel() * workspace.element_size(), int(flags), _stream(Q.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_attn_bwd")
    return dQ, dK, dV


def _rect_shapes(Q, K, V):
    _check_bf16("Q", Q)
    B, H, Nq, d = Q.shape
    _check_bf16("K", K); _check_bf16("V", V, K.shape)
    if K.dim() != 4 or K.shape[0] != B or K.shape[3] != d or H % K.shape[1] != 0:
        raise ValueError(f"K/V shape {tuple(K.shape)} does not match Q {tuple(Q.shape)} (need [B, Hkv, Nk, d], H % Hkv == 0)")
    return B, H, K.shape[1], Nq, K.shape[2], d


def gproj_attn_fwd_rect(Q, K, V, softmax_scale, causal, O=None, LSE=None, fwd_flags=0):
    """Forward with Nq queries and Nk keys: Q [B, H, Nq, d]; K, V [B, Hkv, Nk, d].  Causal: query i sees the keys
    j <= i + (Nk - Nq); a query that sees none gets O = 0 and LSE = +inf."""
    B, H, Hkv, Nq, Nk, d = _rect_shapes(Q, K, V)
    O = torch.empty_like(Q) if O is None else O
    LSE = torch.empty((B, H, Nq), dtype=torch.float32, device=Q.device) if LSE is None else LSE
    _check_bf16("O", O, Q.shape)
    with torch.cuda.device(Q.device):
        rc = load().gproj_attn_fwd_rect(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(), B, H, Hkv, Nq, Nk, d,
                                        float(softmax_scale), int(bool(causal)), int(fwd_flags), _stream(Q.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_attn_fwd_rect")
    return O, LSE


def gproj_attn_bwd_rect(Q, K, V, O, LSE, dO, softmax_scale, causal, flags=0, workspace=None, dQ=None, dK=None, dV=None):
    """Backward of gproj_attn_fwd_rect (same shapes; dK, dV like K).  Workspace: gproj_attn_bwd_workspace_bytes(B, H, Nq, d)."""
    B, H, Hkv, Nq, Nk, d = _rect_shapes(Q, K, V)
    for name, t in (("O", O), ("dO", dO)):
        _check_bf16(name, t, Q.shape)
    if not (LSE.is_cuda and LSE.dtype == torch.float32 and LSE.is_contiguous() and tuple(LSE.shape) == (B, H, Nq)):
        raise TypeError("LSE must be a contiguous CUDA float32 tensor [B, H, Nq]")
    if workspace is None:
        workspace = torch.empty(max(gproj_attn_bwd_workspace_bytes(B, H, Nq, d), 256), dtype=torch.uint8, device=Q.device)
    dQ = torch.empty_like(Q) if dQ is None else dQ
    dK = torch.empty_like(K) if dK is None else dK
    dV = torch.empty_like(K) if dV is None else dV
    _check_bf16("dQ", dQ, Q.shape); _check_bf16("dK", dK, K.shape); _check_bf16("dV", dV, K.shape)
    with torch.cuda.device(Q.device):
        rc = load().gproj_attn_bwd_rect(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(), dO.data_ptr(),
                                        dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), B, H, Hkv, Nq, Nk, d, float(softmax_scale),
                                        int(bool(causal)), workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                        int(flags), _stream(Q.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_attn_bwd_rect")
    return dQ, dK, dV


def gproj_attn_bwd_static_scratch(Q, K, V, O, LSE, dO, softmax_scale, causal, flags=0, dQ=None, dK=None, dV=None):
    """Backward that uses the library's built-in device scratch instead of a workspace tensor.

    For callers that may not allocate device memory when the gradient is needed.  Shapes needing more than
    ``STATIC_SCRATCH_BYTES`` of scratch raise ``GprojError`` (status -4).  Calls on one device share the scratch:
    do not let two of them overlap on the GPU.  The output tensors are the caller's (pass dQ, dK, dV to avoid
    even those allocations).
    """
    _check_bf16("Q", Q)
    B, H, N, d = Q.shape
    for name, t in (("K", K), ("V", V), ("O", O), ("dO", dO)):
        _check_bf16(name, t, Q.shape)
    if not (LSE.is_cuda and LSE.dtype == torch.float32 and LSE.is_contiguous() and tuple(LSE.shape) == (B, H, N)):
        raise TypeError("LSE must be a contiguous CUDA float32 tensor [B, H, N]")
    dQ = torch.empty_like(Q) if dQ is None else dQ
    dK = torch.empty_like(Q) if dK is None else dK
    dV = torch.empty_like(Q) if dV is None else dV
    for name, t in (("dQ", dQ), ("dK", dK), ("dV", dV)):      # a wrong output tensor would be overwritten out of bounds
        _check_bf16(name, t, Q.shape)
    with torch.cuda.device(Q.device):
        rc = load().gproj_attn_bwd_static_scratch(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(),
                                                  dO.data_ptr(), dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), B, H, N, d,
                                                  float(softmax_scale), int(bool(causal)), int(flags), _stream(Q.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_attn_bwd_static_scratch")
    return dQ, dK, dV


def gproj_fp32_attn_fwd(Q, K, V, softmax_scale, causal, saved=None):
    """O (bfloat16), saved = fused FP32 attention forward (the comparison arm; plain FP32 arithmetic on the CUDA cores)."""
    _check_bf16("Q", Q)
    B, H, N, d = Q.shape
    _check_bf16("K", K, Q.shape); _check_bf16("V", V, Q.shape)
    need = int(load().gproj_fp32_attn_saved_bytes(B, H, N, d))
    if saved is None:
        saved = torch.empty(max(need, 256), dtype=torch.uint8, device=Q.device)
    O = torch.empty_like(Q)
    with torch.cuda.device(Q.device):
        rc = load().gproj_fp32_attn_fwd(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), saved.data_ptr(), saved.numel(),
                                        B, H, N, d, float(softmax_scale), int(bool(causal)), _stream(Q.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_fp32_attn_fwd")
    return O, saved


def gproj_fp32_attn_bwd(Q, K, V, dO, saved, softmax_scale, causal):
    """dQ, dK, dV (bfloat16) = fused FP32 attention backward from the state gproj_fp32_attn_fwd saved."""
    _check_bf16("Q", Q)
    B, H, N, d = Q.shape
    for name, t in (("K", K), ("V", V), ("dO", dO)):
        _check_bf16(name, t, Q.shape)
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(Q), torch.empty_like(Q)
    with torch.cuda.device(Q.device):
        rc = load().gproj_fp32_attn_bwd(Q.data_ptr(), K.data_ptr(), V.data_ptr(), dO.data_ptr(), saved.data_ptr(), saved.numel(),
                                        dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), B, H, N, d, float(softmax_scale),
                                        int(bool(causal)), _stream(Q.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_fp32_attn_bwd")
    return dQ, dK, dV


def gproj_key_smooth(X, Y=None, cu_seqlens=None):
    """Y = X minus its per-sequence, per-head mean row (key smoothing; also the matching fix-up of dK).
    X: CUDA bfloat16 [B, Hkv, N, d], or packed [Hkv, T, d] with host offsets ``cu_seqlens``."""
    _check_bf16("X", X)
    Y = torch.empty_like(X) if Y is None else Y
    _check_bf16("Y", Y, X.shape)
    with torch.cuda.device(X.device):
        if cu_seqlens is None:
            B, Hkv, N, d = X.shape
            rc = load().gproj_key_smooth(X.data_ptr(), Y.data_ptr(), B, Hkv, N, d, _stream(X.device))
        else:
            Hkv, T, d = X.shape
            cu = (ctypes.c_int * len(cu_seqlens))(*[int(v) for v in cu_seqlens])
            rc = load().gproj_key_smooth_varlen(X.data_ptr(), Y.data_ptr(), cu, len(cu_seqlens) - 1, Hkv, d, _stream(X.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_key_smooth")
    return Y


def gproj_last_device_status(device=None):
    """Synchronise the current stream and return (status, raw device code)."""
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    detail = ctypes.c_int(0)
    with torch.cuda.device(device):
        rc = load().gproj_last_device_status(_stream(device), ctypes.byref(detail))
    return rc, detail.value


def gproj_selftest_wait_timeout(device=None):
    """Enqueue the bounded-wait self-test kernel (its wait can never be satisfied; see the header)."""
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else device
    with torch.cuda.device(device):
        rc = load().gproj_selftest_wait_timeout(_stream(device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_selftest_wait_timeout")


def gproj_last_launch_count() -> int:
    return int(load().gproj_last_launch_count())


class VarlenPlan:
    """Packed-sequence description: host cu_seqlens plus the device tile list the kernels walk (built once per packing).

    With ``cu_seqlens_k`` the sequences' key lengths differ from their query lengths (the ``*_varlen_qk`` calls)."""

    def __init__(self, cu_seqlens, causal, device="cuda", cu_seqlens_k=None):
        cu = [int(x) for x in cu_seqlens]
        self.num_seqs = len(cu) - 1
        self.cu = (ctypes.c_int * len(cu))(*cu)
        self.causal = bool(causal)
        self.total = cu[-1]
        self.cu_k, self.total_k = None, self.total
        if cu_seqlens_k is not None:
            ck = [int(x) for x in cu_seqlens_k]
            if len(ck) != len(cu):
                raise ValueError("cu_seqlens_k must have as many entries as cu_seqlens")
            self.cu_k = (ctypes.c_int * len(ck))(*ck)
            self.total_k = ck[-1]
            nbytes = int(load().gproj_attn_varlen_qk_plan_bytes(self.cu, self.cu_k, self.num_seqs))
        else:
            nbytes = int(load().gproj_attn_varlen_plan_bytes(self.cu, self.num_seqs))
        if nbytes == 0 and (self.total <= 0 or self.total_k <= 0):
            raise GprojError(-2, "gproj_attn_varlen_plan_bytes")
        host = torch.empty(max(nbytes, 16), dtype=torch.uint8)
        if self.cu_k is not None:
            rc = load().gproj_attn_varlen_qk_plan(self.cu, self.cu_k, self.num_seqs, int(self.causal), ctypes.c_void_p(host.data_ptr()), nbytes)
        else:
            rc = load().gproj_attn_varlen_plan(self.cu, self.num_seqs, int(self.causal), ctypes.c_void_p(host.data_ptr()), nbytes)
        if rc != GPROJ_OK:
            raise GprojError(rc, "gproj_attn_varlen_plan")
        self.host = host
        self.device = host.to(device)


def gproj_attn_fwd_varlen(Q, K, V, plan, softmax_scale, fwd_flags=0):
    """O, LSE = forward over packed sequences.  Q: CUDA bfloat16 [H, T, d]; K, V: [Hkv, T, d]; plan: VarlenPlan."""
    _check_bf16("Q", Q)
    H, T, d = Q.shape
    _check_bf16("K", K); _check_bf16("V", V, K.shape)
    if K.dim() != 3 or K.shape[1] != T or K.shape[2] != d or H % K.shape[0] != 0 or T != plan.total:
        raise ValueError("packed K/V must be [Hkv, T, d] with T = cu_seqlens[-1] and H a multiple of Hkv")
    O = torch.empty_like(Q)
    LSE = torch.empty((H, T), dtype=torch.float32, device=Q.device)
    with torch.cuda.device(Q.device):
        rc = load().gproj_attn_fwd_varlen(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(), plan.cu,
                                          plan.num_seqs, plan.device.data_ptr(), H, K.shape[0], d, float(softmax_scale),
                                          int(plan.causal), int(fwd_flags), _stream(Q.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_attn_fwd_varlen")
    return O, LSE


def gproj_attn_bwd_varlen(Q, K, V, O, LSE, dO, plan, softmax_scale, flags=0, workspace=None):
    """dQ, dK, dV = backward over packed sequences (same layout as gproj_attn_fwd_varlen)."""
    _check_bf16("Q", Q)
    H, T, d = Q.shape
    for name, t in (("O", O), ("dO", dO)):
        _check_bf16(name, t, Q.shape)
    _check_bf16("K", K); _check_bf16("V", V, K.shape)
    if not (LSE.is_cuda and LSE.dtype == torch.float32 and LSE.is_contiguous() and tuple(LSE.shape) == (H, T)):
        raise TypeError("LSE must be a contiguous CUDA float32 tensor [H, T]")
    need = int(load().gproj_attn_bwd_varlen_workspace_bytes(plan.cu, plan.num_seqs, H, d))
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=Q.device)
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
    with torch.cuda.device(Q.device):
        rc = load().gproj_attn_bwd_varlen(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(), dO.data_ptr(),
                                          dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), plan.cu, plan.num_seqs,
                                          plan.device.data_ptr(), H, K.shape[0], d, float(softmax_scale), int(plan.causal),
                                          workspace.data_ptr(), workspace.numel(), int(flags), _stream(Q.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_attn_bwd_varlen")
    return dQ, dK, dV


def gproj_attn_host_staging_bytes(B, H, Hkv, N, d) -> int:
    return int(load().gproj_attn_host_staging_bytes(B, H, Hkv, N, d))


def gproj_attn_fwd_bwd_host(Q, K, V, dO, dQ, dK, dV, softmax_scale, causal, staging, O=None, LSE=None, flags=0):
    """Forward + backward from HOST bfloat16 tensors (pinned for an asynchronous call) into HOST dQ, dK, dV (and O, LSE if
    given); `staging` is a CUDA uint8 tensor of gproj_attn_host_staging_bytes() bytes.  Work is enqueued on the current stream."""
    for name, t in (("Q", Q), ("K", K), ("V", V), ("dO", dO), ("dQ", dQ), ("dK", dK), ("dV", dV)):
        if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()):
            raise TypeError(f"{name} must be a contiguous CPU bfloat16 tensor")
    B, H, N, d = Q.shape
    Hkv = K.shape[1]
    if not (staging.is_cuda and staging.dtype == torch.uint8 and staging.is_contiguous()):
        raise TypeError("staging must be a contiguous CUDA uint8 tensor")
    ptr = lambda t: ctypes.c_void_p(t.data_ptr()) if t is not None else None
    with torch.cuda.device(staging.device):
        rc = load().gproj_attn_fwd_bwd_host(ptr(Q), ptr(K), ptr(V), ptr(dO), ptr(O), ptr(LSE), ptr(dQ), ptr(dK), ptr(dV), B, H, Hkv, N, d,
                                            float(softmax_scale), int(bool(causal)), ptr(staging), staging.numel(), int(flags),
                                            _stream(staging.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_attn_fwd_bwd_host")


def _packed_qk_shapes(Q, K, V, plan):
    _check_bf16("Q", Q)
    H, Tq, d = Q.shape
    _check_bf16("K", K); _check_bf16("V", V, K.shape)
    if plan.cu_k is None:
        raise ValueError("the plan has no cu_seqlens_k: build it with VarlenPlan(cu_q, causal, cu_seqlens_k=cu_k)")
    if K.dim() != 3 or K.shape[2] != d or H % K.shape[0] != 0 or Tq != plan.total or K.shape[1] != plan.total_k:
        raise ValueError("packed tensors must be Q [H, Tq, d], K/V [Hkv, Tk, d] with Tq, Tk the last offsets and H a multiple of Hkv")
    return H, K.shape[0], Tq, d


def gproj_attn_fwd_varlen_qk(Q, K, V, plan, softmax_scale, fwd_flags=0):
    """O, LSE = forward over packed sequences with their own query and key lengths.  Q: [H, Tq, d]; K, V: [Hkv, Tk, d]."""
    H, Hkv, Tq, d = _packed_qk_shapes(Q, K, V, plan)
    O = torch.empty_like(Q)
    LSE = torch.empty((H, Tq), dtype=torch.float32, device=Q.device)
    with torch.cuda.device(Q.device):
        rc = load().gproj_attn_fwd_varlen_qk(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(), plan.cu, plan.cu_k,
                                             plan.num_seqs, plan.device.data_ptr(), H, Hkv, d, float(softmax_scale),
                                             int(plan.causal), int(fwd_flags), _stream(Q.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_attn_fwd_varlen_qk")
    return O, LSE


def gproj_attn_bwd_varlen_qk(Q, K, V, O, LSE, dO, plan, softmax_scale, flags=0, workspace=None):
    """dQ, dK, dV = backward of gproj_attn_fwd_varlen_qk (same layout; dK, dV like K)."""
    H, Hkv, Tq, d = _packed_qk_shapes(Q, K, V, plan)
    for name, t in (("O", O), ("dO", dO)):
        _check_bf16(name, t, Q.shape)
    if not (LSE.is_cuda and LSE.dtype == torch.float32 and LSE.is_contiguous() and tuple(LSE.shape) == (H, Tq)):
        raise TypeError("LSE must be a contiguous CUDA float32 tensor [H, Tq]")
    need = int(load().gproj_attn_bwd_varlen_workspace_bytes(plan.cu, plan.num_seqs, H, d))
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=Q.device)
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
    with torch.cuda.device(Q.device):
        rc = load().gproj_attn_bwd_varlen_qk(Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(), dO.data_ptr(),
                                             dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), plan.cu, plan.cu_k, plan.num_seqs,
                                             plan.device.data_ptr(), H, Hkv, d, float(softmax_scale), int(plan.causal),
                                             workspace.data_ptr(), workspace.numel(), int(flags), _stream(Q.device))
    if rc != GPROJ_OK:
        raise GprojError(rc, "gproj_attn_bwd_varlen_qk")
    return dQ, dK, dV
