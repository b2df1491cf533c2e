"""Thin ctypes binding of libwush.so: argument marshalling only.

Every function has the name of the C entry point it calls (include/wush.h) minus the
`wush_` prefix, takes CUDA torch tensors, allocates the output tensors with torch
(torch is used for device memory and streams, nothing else) and enqueues the kernels
on torch's current stream.  Nothing is computed in Python, and there is no fallback:
if the library has not been built, or a call returns an error status, an exception
is raised.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwush.so")

MXFP4, NVFP4, MXFP4_CEIL = 0, 1, 2
SF_LINEAR, SF_TILED = 0, 1
OUT_F32, OUT_BF16 = 0, 1
FORMATS = {"mxfp4": (MXFP4, 32), "nvfp4": (NVFP4, 16), "mxfp4_ceil": (MXFP4_CEIL, 32)}

EXPORTS = [
    "wush_status_string", "wush_last_cuda_error", "wush_scale_bytes", "wush_quantize_act",
    "wush_quantize_weight", "wush_quantize_weight_workspace_bytes", "wush_gemm_fp4", "wush_linear",
    "wush_linear_workspace_bytes", "wush_calib_moments", "wush_calib_moments_workspace_bytes",
    "wush_quantize_f32", "wush_transform_act_f32", "wush_transform_weight_f32", "wush_calib_moments_static",
    "wush_build_transforms", "wush_quantize_act_dynamic", "wush_check_division", "wush_debug_gemm_clusters",
    "wush_debug_drop_tile", "wush_decode_status", "wush_build_transforms_kind", "wush_invert_transforms",
    "wush_act_tensor_scale", "wush_workspace_bytes", "wush_debug_quantiser_rows",
    "wush_gptq_quantize_weight", "wush_gptq_workspace_bytes",
]
STATIC_SCRATCH_BYTES = 4 << 20

_lib = None


class WushError(RuntimeError):
    pass


def lib():
    """Load libwush.so once.  Raises if it is missing: there is no other code path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise WushError(f"{LIB_PATH} not found: build it with `python -m paper_2512_00956_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
        L.wush_status_string.restype = ctypes.c_char_p
        L.wush_status_string.argtypes = [i32]
        L.wush_last_cuda_error.restype = ctypes.c_char_p
        L.wush_scale_bytes.restype = sz
        L.wush_scale_bytes.argtypes = [i64, i64, i32, i32]
        L.wush_quantize_act.argtypes = [vp, i64, i64, vp, i32, i32, vp, vp, vp, i32, vp]
        L.wush_quantize_act_dynamic.argtypes = [vp, i64, i64, vp, i32, vp, vp, vp, i32, vp]
        L.wush_quantize_weight.argtypes = [vp, i64, i64, vp, i32, i32, vp, vp, vp, i32, vp, sz, vp]
        L.wush_quantize_weight_workspace_bytes.restype = sz
        L.wush_quantize_weight_workspace_bytes.argtypes = [i64, i64, i32, i32]
        L.wush_gemm_fp4.argtypes = [vp, vp, vp, vp, i64, i64, i64, i32, i32, vp, vp, vp, i32, vp, vp]
        L.wush_linear.argtypes = [vp, i64, i64, vp, vp, vp, i64, vp, vp, i32, i32, vp, i32, vp, sz, vp]
        L.wush_linear_workspace_bytes.restype = sz
        L.wush_linear_workspace_bytes.argtypes = [i64, i64, i32]
        L.wush_gptq_workspace_bytes.restype = sz
        L.wush_gptq_workspace_bytes.argtypes = [i64, i64, i32]
        L.wush_gptq_quantize_weight.restype = i32
        L.wush_gptq_quantize_weight.argtypes = [vp, i64, i64, vp, i64, i32, i32, ctypes.c_float, vp, vp, vp, vp, vp, i32, vp, vp, sz, vp]
        L.wush_workspace_bytes.restype = sz
        L.wush_workspace_bytes.argtypes = [i64, i64, i64, i32, i32]
        L.wush_debug_quantiser_rows.argtypes = [i32]
        L.wush_debug_quantiser_rows.restype = i32
        L.wush_calib_moments.argtypes = [vp, i64, i64, i32, vp, vp, vp, sz, vp]
        L.wush_calib_moments_workspace_bytes.restype = sz
        L.wush_calib_moments_workspace_bytes.argtypes = [i64, i64, i32]
        L.wush_build_transforms.argtypes = [vp, i64, vp, i64, i64, i32, ctypes.c_float, vp, vp, vp, vp]
        L.wush_build_transforms.restype = i32
        L.wush_build_transforms_kind.argtypes = [vp, i64, vp, i64, i64, i32, ctypes.c_float, i32, vp, vp, vp, vp]
        L.wush_invert_transforms.argtypes = [vp, i64, i32, vp, vp, vp]
        L.wush_act_tensor_scale.argtypes = [vp, i64, i64, vp, i32, vp, vp]
        L.wush_calib_moments_static.argtypes = [vp, i64, i64, i32, vp, vp, vp]
        L.wush_debug_gemm_clusters.argtypes = [i32]
        L.wush_debug_gemm_clusters.restype = i32
        L.wush_debug_drop_tile.argtypes = [i32]
        L.wush_decode_status.argtypes = [i32]
        L.wush_calib_moments_static.restype = i32
        L.wush_quantize_f32.argtypes = [vp, i64, i64, i32, i32, vp, vp, vp, i32, vp]
        L.wush_check_division.argtypes = [vp, i32, vp, vp]
        L.wush_transform_act_f32.argtypes = [vp, i64, i64, vp, i32, vp, vp]
        L.wush_transform_weight_f32.argtypes = [vp, i64, i64, vp, i32, vp, vp]
        for name in ("wush_quantize_act", "wush_quantize_weight", "wush_gemm_fp4", "wush_linear",
                     "wush_calib_moments", "wush_quantize_f32", "wush_transform_act_f32",
                     "wush_transform_weight_f32"):
            getattr(L, name).restype = i32
        _lib = L
    return _lib


def check(status):
    if status != 0:
        L = lib()
        msg = L.wush_status_string(status).decode()
        if status == -6:
            msg += ": " + L.wush_last_cuda_error().decode()
        raise WushError(f"libwush status {status}: {msg}")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _fmt(fmt):
    return FORMATS[fmt] if isinstance(fmt, str) else (fmt, 16 if fmt == NVFP4 else 32)


def _dev(*ts):
    for t in ts:
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise WushError("expected contiguous CUDA tensors")


def scale_bytes(rows, K, g, sf):
    return lib().wush_scale_bytes(rows, K, g, sf)


def _alloc_q(rows, K, g, sf, device):
    codes = torch.empty((rows, K // 2), dtype=torch.uint8, device=device)
    nbytes = scale_bytes(rows, K, g, sf)
    if sf == SF_LINEAR:
        scales = torch.empty((rows, K // g), dtype=torch.uint8, device=device)
    else:
        scales = torch.zeros(max(nbytes, 16), dtype=torch.uint8, device=device)
    return codes, scales


def quantize_act(X, T, fmt, x_tensor_scale=None, sf=SF_LINEAR, out=None):
    """X bf16 [M,K], T bf16 [K/g,g,g] -> (codes uint8 [M,K/2], scale bytes)."""
    f, g = _fmt(fmt)
    _dev(X, T, x_tensor_scale)
    M, K = X.shape
    codes, scales = out if out is not None else _alloc_q(M, K, g, sf, X.device)
    check(lib().wush_quantize_act(_ptr(X), M, K, _ptr(T), f, g, _ptr(x_tensor_scale), _ptr(codes), _ptr(scales),
                                  sf, _stream()))
    return codes, scales


def quantize_act_dynamic(X, T, sf=SF_LINEAR, out=None, x_tensor_scale=None):
    """NVFP4 with the tensor scale of this batch.  Returns (codes, scale bytes, fp32[2] = scale used, AbsMax)."""
    _dev(X, T)
    M, K = X.shape
    codes, scales = out if out is not None else _alloc_q(M, K, 16, sf, X.device)
    ts = x_tensor_scale if x_tensor_scale is not None else torch.zeros(4, dtype=torch.float32, device=X.device)
    check(lib().wush_quantize_act_dynamic(_ptr(X), M, K, _ptr(T), 16, _ptr(ts), _ptr(codes), _ptr(scales), sf, _stream()))
    return codes, scales, ts


def act_tensor_scale(Xc, T, g=16):
    """Static NVFP4 activation tensor scale of calibration tokens: fp32[4] on the device, [0] = scale, [1] = AbsMax."""
    _dev(Xc, T)
    out = torch.zeros(4, dtype=torch.float32, device=Xc.device)
    check(lib().wush_act_tensor_scale(_ptr(Xc), Xc.shape[0], Xc.shape[1], _ptr(T), g, _ptr(out), _stream()))
    return out


def quantize_weight(W, Tinv, fmt, sf=SF_TILED, out=None):
    """W bf16 [N,K], Tinv fp32 [K/g,g,g] -> (codes, scale bytes, w_tensor_scale fp32[1] or None).
    `out` = (codes, scales, tensor_scale, workspace) reuses caller-owned buffers."""
    f, g = _fmt(fmt)
    _dev(W, Tinv)
    N, K = W.shape
    nws = lib().wush_quantize_weight_workspace_bytes(N, K, f, g)
    if out is not None:
        codes, scales, ts, ws = out
    else:
        codes, scales = _alloc_q(N, K, g, sf, W.device)
        ts = torch.zeros(4, dtype=torch.float32, device=W.device) if f == NVFP4 else None
        ws = torch.empty(nws, dtype=torch.uint8, device=W.device)
    check(lib().wush_quantize_weight(_ptr(W), N, K, _ptr(Tinv), f, g, _ptr(ts), _ptr(codes), _ptr(scales), sf,
                                     _ptr(ws), nws, _stream()))
    return codes, scales, ts


def gemm_fp4(Xq, Xs, Wq, Ws, K, fmt, x_tensor_scale=None, w_tensor_scale=None, out_dtype=torch.float32,
             out=None, status=None):
    """Packed codes [M,K/2], [N,K/2] + TILED scale bytes -> Y [M,N]."""
    f, g = _fmt(fmt)
    _dev(Xq, Xs, Wq, Ws)
    M, N = Xq.shape[0], Wq.shape[0]
    Y = out if out is not None else torch.empty((M, N), dtype=out_dtype, device=Xq.device)
    ydt = OUT_BF16 if Y.dtype == torch.bfloat16 else OUT_F32
    if status is None:
        status = torch.zeros(4, dtype=torch.int32, device=Xq.device)
    check(lib().wush_gemm_fp4(_ptr(Xq), _ptr(Xs), _ptr(Wq), _ptr(Ws), M, N, K, f, g, _ptr(x_tensor_scale),
                              _ptr(w_tensor_scale), _ptr(Y), ydt, _ptr(status), _stream()))
    return Y, status


def linear_workspace_bytes(M, K, g):
    return lib().wush_linear_workspace_bytes(M, K, g)


def workspace_bytes(M, N, K, fmt):
    """One workspace size that serves every call of a layer with up to M tokens (wush_workspace_bytes)."""
    f, g = _fmt(fmt)
    return lib().wush_workspace_bytes(M, N, K, f, g)


def linear(X, T, Wcodes, Wscales, fmt, x_tensor_scale=None, w_tensor_scale=None, out_dtype=torch.float32,
           out=None, workspace=None):
    """The whole online layer: Y = q(X T^T) (x) W~ (Eq. 7).  Returns (Y, workspace).
    NVFP4 with x_tensor_scale=None takes the activation tensor scale from this batch (see linear_dynamic_scale)."""
    f, g = _fmt(fmt)
    _dev(X, T, Wcodes, Wscales)
    M, K = X.shape
    N = Wcodes.shape[0]
    Y = out if out is not None else torch.empty((M, N), dtype=out_dtype, device=X.device)
    ydt = OUT_BF16 if Y.dtype == torch.bfloat16 else OUT_F32
    nws = linear_workspace_bytes(M, K, g)
    if workspace is None:
        workspace = torch.empty(nws, dtype=torch.uint8, device=X.device)
    check(lib().wush_linear(_ptr(X), M, K, _ptr(T), _ptr(Wcodes), _ptr(Wscales), N, _ptr(x_tensor_scale),
                            _ptr(w_tensor_scale), f, g, _ptr(Y), ydt, _ptr(workspace), workspace.numel(), _stream()))
    return Y, workspace


def linear_dynamic_scale(workspace, M, K, g):
    """(scale used, AbsMax) that an NVFP4 wush_linear call without x_tensor_scale left in its workspace.  Synchronises."""
    end = linear_workspace_bytes(M, K, g)
    v = workspace[end - 32:end - 24].view(torch.float32)
    return float(v[0].item()), float(v[1].item())


def linear_status(workspace, M, K, g):
    """The GEMM's diagnostic word, kept in the last 16 bytes of the wush_linear_workspace_bytes(M, K, g)
    region of the workspace (0 = no bounded wait expired).  Synchronises."""
    end = linear_workspace_bytes(M, K, g)
    return int(workspace[end - 16:end].view(torch.int32)[0].item())


def calib_moments(Xc, g, moments=None, count=None, workspace=None):
    """moments[c] += sum_t x_tc^T x_tc ; count += B.  Returns (moments fp32 [K/g,g,g], count int64[1])."""
    _dev(Xc, moments, count)
    B, K = Xc.shape
    if moments is None:
        moments = torch.zeros((K // g, g, g), dtype=torch.float32, device=Xc.device)
    if count is None:
        count = torch.zeros(2, dtype=torch.int64, device=Xc.device)
    nws = lib().wush_calib_moments_workspace_bytes(B, K, g)
    ws = workspace if workspace is not None else torch.empty(max(nws, 16), dtype=torch.uint8, device=Xc.device)
    check(lib().wush_calib_moments(_ptr(Xc), B, K, g, _ptr(moments), _ptr(count), _ptr(ws), ws.numel(), _stream()))
    return moments, count


KINDS = {"wush": 0, "wus": 1, "hadamard": 2, "identity": 3}


def fixed_transforms(kind, C, g, device):
    """The data-independent transforms "hadamard" / "identity" for C blocks, made by the library
    (wush_build_transforms_kind without moments).  Returns (T bf16 [C,g,g], Tinv fp32 [C,g,g], info)."""
    T = torch.empty((C, g, g), dtype=torch.bfloat16, device=device)
    Tinv = torch.empty((C, g, g), dtype=torch.float32, device=device)
    info = torch.zeros(max(C, 4), dtype=torch.int32, device=device)
    with torch.cuda.device(device):
        check(lib().wush_build_transforms_kind(None, 0, None, 0, C * g, g, 0.0, KINDS[kind], _ptr(T), _ptr(Tinv),
                                               _ptr(info), _stream()))
    return T, Tinv, info[:C]


def build_transforms(mom_w, rows_w, mom_x, rows_x, g, lam=0.01, kind="wush"):
    """Moment sums fp32 [K/g,g,g] (+ row counts) -> (T bf16 [K/g,g,g], Tinv fp32 [K/g,g,g], info int32 [K/g]).
    kind "wus" leaves the Hadamard factor out (the ablation of Table 1)."""
    _dev(mom_w, mom_x)
    C = mom_w.shape[0]
    K = C * g
    T = torch.empty((C, g, g), dtype=torch.bfloat16, device=mom_w.device)
    Tinv = torch.empty((C, g, g), dtype=torch.float32, device=mom_w.device)
    info = torch.zeros(max(C, 4), dtype=torch.int32, device=mom_w.device)
    check(lib().wush_build_transforms_kind(_ptr(mom_w), int(rows_w), _ptr(mom_x), int(rows_x), K, g, float(lam),
                                           KINDS[kind], _ptr(T), _ptr(Tinv), _ptr(info), _stream()))
    return T, Tinv, info[:C]


def gptq_quantize_weight(W, Xc, fmt, lam=0.01, w_tensor_scale=None, sf=SF_TILED):
    """Algorithm 2, GPTQ case (wush_gptq_quantize_weight).  W bf16 [N,K], Xc bf16 [B,K] ->
    (T bf16 [K/g,g,g], Tinv fp32 [K/g,g,g], codes, scale bytes, info int32 [K/g]).  NVFP4 needs w_tensor_scale (fp32, device)."""
    f, g = _fmt(fmt)
    _dev(W, Xc, w_tensor_scale)
    N, K = W.shape
    C = K // g
    T = torch.empty((C, g, g), dtype=torch.bfloat16, device=W.device)
    Tinv = torch.empty((C, g, g), dtype=torch.float32, device=W.device)
    codes, scales = _alloc_q(N, K, g, sf, W.device)
    info = torch.zeros(max(C, 4), dtype=torch.int32, device=W.device)
    nws = lib().wush_gptq_workspace_bytes(N, K, g)
    ws = torch.empty(nws + 256, dtype=torch.uint8, device=W.device)
    off = (-ws.data_ptr()) % 256
    check(lib().wush_gptq_quantize_weight(_ptr(W), N, K, _ptr(Xc), Xc.shape[0], f, g, float(lam), _ptr(w_tensor_scale),
                                          _ptr(T), _ptr(Tinv), _ptr(codes), _ptr(scales), sf, _ptr(info),
                                          ctypes.c_void_p(ws.data_ptr() + off), nws, _stream()))
    return T, Tinv, codes, scales, info[:C]


def invert_transforms(T, g):
    """T bf16 [K/g,g,g] -> (Tinv fp32 [K/g,g,g] = T^-T per block, info int32 [K/g])."""
    _dev(T)
    C = T.shape[0]
    Tinv = torch.empty((C, g, g), dtype=torch.float32, device=T.device)
    info = torch.zeros(max(C, 4), dtype=torch.int32, device=T.device)
    check(lib().wush_invert_transforms(_ptr(T), C * g, g, _ptr(Tinv), _ptr(info), _stream()))
    return Tinv, info[:C]


def calib_moments_static(Xc, g, moments=None, count=None):
    """wush_calib_moments_static: like calib_moments, but the library's built-in scratch array is
    used, so no workspace tensor is created here.  For processes that cannot allocate device
    memory when they call (the outputs are passed in, or made once by the caller)."""
    _dev(Xc, moments, count)
    B, K = Xc.shape
    if moments is None:
        moments = torch.zeros((K // g, g, g), dtype=torch.float32, device=Xc.device)
    if count is None:
        count = torch.zeros(2, dtype=torch.int64, device=Xc.device)
    check(lib().wush_calib_moments_static(_ptr(Xc), B, K, g, _ptr(moments), _ptr(count), _stream()))
    return moments, count


def quantize_f32(V, fmt, tensor_scale=None, sf=SF_LINEAR):
    f, g = _fmt(fmt)
    _dev(V, tensor_scale)
    R, K = V.shape
    codes, scales = _alloc_q(R, K, g, sf, V.device)
    check(lib().wush_quantize_f32(_ptr(V), R, K, f, g, _ptr(tensor_scale), _ptr(codes), _ptr(scales), sf, _stream()))
    return codes, scales


def debug_drop_tile(item):
    """Test hook: the next `linear` call does not load work item `item` of its quantiser (-1 cancels)."""
    check(lib().wush_debug_drop_tile(int(item)))


def decode_status(word):
    """WUSH_OK (0) or WUSH_ERR_TIMEOUT for a status word read back from the device."""
    return int(lib().wush_decode_status(int(word)))


def debug_quantiser_rows(rows):
    """Test hook: tile height (64 / 128, 0 = automatic) of the streaming quantiser; returns the old value."""
    r = int(lib().wush_debug_quantiser_rows(int(rows)))
    if r < 0:
        check(r)
    return r


def debug_gemm_clusters(clusters):
    """Test hook: limit the persistent GEMM to `clusters` clusters (0 = no limit); returns the old value."""
    return int(lib().wush_debug_gemm_clusters(int(clusters)))


def check_division(divisors):
    """Mismatch counts (int64 tensor) of the branch-free division against the IEEE one, per divisor, over all x."""
    _dev(divisors)
    out = torch.zeros(divisors.numel(), dtype=torch.int64, device=divisors.device)
    check(lib().wush_check_division(_ptr(divisors), divisors.numel(), _ptr(out), _stream()))
    return out


def transform_act_f32(X, T, g):
    _dev(X, T)
    M, K = X.shape
    V = torch.empty((M, K), dtype=torch.float32, device=X.device)
    check(lib().wush_transform_act_f32(_ptr(X), M, K, _ptr(T), g, _ptr(V), _stream()))
    return V


def transform_weight_f32(W, Tinv, g):
    _dev(W, Tinv)
    N, K = W.shape
    V = torch.empty((N, K), dtype=torch.float32, device=W.device)
    check(lib().wush_transform_weight_f32(_ptr(W), N, K, _ptr(Tinv), g, _ptr(V), _stream()))
    return V
