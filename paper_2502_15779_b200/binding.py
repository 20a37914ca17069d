"""Thin Python binding over the C ABI declared in include/rcp.h.

Argument marshalling only: tensors are allocated by torch (device memory and streams), every
computation runs in the library's CUDA kernels.  There is no fallback: if the shared library
is missing or a call fails, an exception is raised.
"""
import contextlib
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# RCP_W2A4_LIB names another build of the same library (the tests use it for the guarded build)
LIB_PATH = os.environ.get("RCP_W2A4_LIB") or os.path.join(_HERE, "librcp_w2a4.so")

GEMV_AUTO, GEMV_SIMPLE, GEMV_DP4A, GEMV_MMA, GEMV_MMA_ONLY, GEMV_MMA_STREAM = 0, 1, 2, 3, 4, 5
VARIANTS = {"auto": GEMV_AUTO, "simple": GEMV_SIMPLE, "dp4a": GEMV_DP4A, "mma": GEMV_MMA, "mma_only": GEMV_MMA_ONLY,
            "mma_stream": GEMV_MMA_STREAM}

_lib = None


class RcpError(RuntimeError):
    def __init__(self, fn, status, text, cuda_error):
        super().__init__(f"{fn} failed: {text} (status {status}, cuda error {cuda_error})")
        self.status = status


def lib():
    """Loads the shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} not found: build it with `python -m paper_2502_15779_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i, u64 = C.c_void_p, C.c_int, C.c_size_t
        L.rcp_status_str.restype = C.c_char_p
        L.rcp_status_str.argtypes = [i]
        L.rcp_last_cuda_error.restype = i
        L.rcp_pack_weights.restype = i
        L.rcp_pack_weights.argtypes = [vp, i, i, vp, vp]
        L.rcp_quantize_act.restype = i
        L.rcp_quantize_act.argtypes = [vp, i, i, i, C.c_float, vp, vp, vp]
        L.rcp_gemv_workspace_bytes.restype = u64
        L.rcp_gemv_workspace_bytes.argtypes = [i, i, i]
        L.rcp_gemv_w2a4.restype = i
        L.rcp_gemv_w2a4.argtypes = [vp, vp, vp, vp, i, i, i, vp, vp, vp, vp]
        L.rcp_gemv_w2a4_variant.restype = i
        L.rcp_gemv_w2a4_variant.argtypes = [i, vp, vp, vp, vp, i, i, i, vp, vp, vp, vp]
        L.rcp_gemv_w2a4_grouped.restype = i
        L.rcp_gemv_w2a4_grouped.argtypes = [vp, vp, i, vp, vp, i, i, i, vp, vp, vp, vp]
        L.rcp_gemv_w2a4_grouped_variant.restype = i
        L.rcp_gemv_w2a4_grouped_variant.argtypes = [i, vp, vp, i, vp, vp, i, i, i, vp, vp, vp, vp]
        L.rcp_ldp_export.restype = i
        L.rcp_ldp_export.argtypes = [vp, vp, vp, vp, vp, i, i, i, vp, vp, vp]
        L.rcp_nf3_export.restype = i
        L.rcp_nf3_export.argtypes = [vp, vp, vp, vp, C.POINTER(C.c_float), i, i, i, i, vp, vp, vp, vp]
        L.rcp_linear_w2a4.restype = i
        L.rcp_linear_w2a4.argtypes = [vp, i, i, i, C.c_float, vp, vp, i, i, vp, vp, vp, vp, vp]
        L.rcp_linear_w2a4_launches.restype = i
        L.rcp_linear_w2a4_launches.argtypes = [i, i, i, i, i]
        L.rcp_linear_w2a4_host.restype = i
        L.rcp_linear_w2a4_host.argtypes = [vp, i, i, i, C.c_float, vp, vp, i, vp, vp, vp, vp, vp, vp, vp]
        L.rcp_gemv_w2a4_static.restype = i
        L.rcp_gemv_w2a4_static.argtypes = [vp, vp, vp, vp, i, i, i, vp, vp]
        L.rcp_gemv_w2a16.restype = i
        L.rcp_gemv_w2a16.argtypes = [vp, vp, vp, i, i, i, vp, vp, vp, vp, vp]
        L.rcp_pack_weights3.restype = i
        L.rcp_pack_weights3.argtypes = [vp, i, i, vp, vp, vp]
        L.rcp_gemv_w3a4.restype = i
        L.rcp_gemv_w3a4.argtypes = [vp, vp, vp, i, vp, vp, i, i, i, vp, vp, vp]
        L.rcp_gemv_w2a4_static_status.restype = i
        L.rcp_gemv_w2a4_static_status.argtypes = [vp, vp]
        L.rcp_selftest_wait_timeout.restype = i
        L.rcp_selftest_wait_timeout.argtypes = [vp, i, vp]
        L.rcp_gemv_w2a16_checked.restype = i
        L.rcp_gemv_w2a16_checked.argtypes = [vp, vp, vp, i, i, i, vp, vp, vp, vp, vp, vp]
        L.rcp_linear_w2a4_checked.restype = i
        L.rcp_linear_w2a4_checked.argtypes = [vp, i, i, i, C.c_float, vp, vp, i, i, vp, vp, vp, vp, vp, vp]
        _lib = L
    return _lib


def _check(fn, status):
    if status != 0:
        L = lib()
        raise RcpError(fn, status, L.rcp_status_str(status).decode(), L.rcp_last_cuda_error())


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


_NULL_CTX = contextlib.nullcontext()


def _on(t):
    """Context that makes t's device current (nothing to do when it already is: the common case, and the
    device guard costs microseconds that a decode step notices)."""
    if torch.cuda.current_device() == t.device.index:
        return _NULL_CTX
    return torch.cuda.device(t.device)


def _stream(t):
    return C.c_void_p(torch.cuda.current_stream(t.device).cuda_stream)


def _dev(t, dtype, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of dtype {dtype}")
    return t


def rcp_pack_weights(codes: torch.Tensor, out: torch.Tensor = None) -> torch.Tensor:
    """codes uint8 [N][K] in {0..3} -> words int32 [N][K/16] (bit pattern of the uint32 words)."""
    _dev(codes, torch.uint8, "codes")
    N, K = codes.shape
    words = out if out is not None else torch.empty((N, K // 16), dtype=torch.int32, device=codes.device)
    with _on(codes):
        _check("rcp_pack_weights", lib().rcp_pack_weights(_ptr(codes), N, K, _ptr(words), _stream(codes)))
    return words


def rcp_ldp_export(w, sig_beta, sig_gamma, sig_s1, sig_s2, group):
    """Rotated weights fp16 [N][K] and the sigmoids of the clipping and partition parameters (float32
    [N][K/group]) -> (words int32 [N][K/16], lut fp16 [N][K/group][4])."""
    _dev(w, torch.float16, "w")
    N, K = w.shape
    group = int(group)
    for name, a in (("sig_beta", sig_beta), ("sig_gamma", sig_gamma), ("sig_s1", sig_s1), ("sig_s2", sig_s2)):
        _dev(a, torch.float32, name)
        if group < 1 or K % group or tuple(a.shape) != (N, K // group):
            raise ValueError(f"{name}: expected shape [N][K/group]")
    words = torch.empty((N, K // 16), dtype=torch.int32, device=w.device)
    lut = torch.empty((N, K // group, 4), dtype=torch.float16, device=w.device)
    with _on(w):
        _check("rcp_ldp_export",
               lib().rcp_ldp_export(_ptr(w), _ptr(sig_beta), _ptr(sig_gamma), _ptr(sig_s1), _ptr(sig_s2), N, K, group,
                                    _ptr(words), _ptr(lut), _stream(w)))
    return words, lut


def rcp_nf3_export(w, sig_beta, sig_gamma, sig_s1, table, zero_index, group):
    """Rotated weights fp16 [N][K], the sigmoids of the clipping parameters and of the centre (float32
    [N][K/group]) and the format's eight normalized levels (a sequence of floats, table[zero_index] == 0)
    -> (words2 int32 [N][K/16], words1 int32 [N][K/32], lut fp16 [N][K/group][8])."""
    _dev(w, torch.float16, "w")
    N, K = w.shape
    group = int(group)
    for name, a in (("sig_beta", sig_beta), ("sig_gamma", sig_gamma), ("sig_s1", sig_s1)):
        _dev(a, torch.float32, name)
        if group < 1 or K % group or tuple(a.shape) != (N, K // group):
            raise ValueError(f"{name}: expected shape [N][K/group]")
    table = [float(t) for t in table]
    if len(table) != 8:
        raise ValueError("table: eight levels expected")
    tab = (C.c_float * 8)(*table)
    words2 = torch.empty((N, K // 16), dtype=torch.int32, device=w.device)
    words1 = torch.empty((N, K // 32), dtype=torch.int32, device=w.device)
    lut = torch.empty((N, K // group, 8), dtype=torch.float16, device=w.device)
    with _on(w):
        _check("rcp_nf3_export",
               lib().rcp_nf3_export(_ptr(w), _ptr(sig_beta), _ptr(sig_gamma), _ptr(sig_s1), tab, int(zero_index), N, K,
                                    group, _ptr(words2), _ptr(words1), _ptr(lut), _stream(w)))
    return words2, words1, lut


def rcp_quantize_act(x: torch.Tensor, had_block: int, clip_ratio: float = 1.0, xq=None, scale=None):
    """x fp16 [M][K] -> (xq uint8 [M][K/2], scale fp16 [M])."""
    _dev(x, torch.float16, "x")
    M, K = x.shape
    if xq is None:
        xq = torch.empty((M, K // 2), dtype=torch.uint8, device=x.device)
    if scale is None:
        scale = torch.empty((M,), dtype=torch.float16, device=x.device)
    with _on(x):
        _check("rcp_quantize_act",
               lib().rcp_quantize_act(_ptr(x), M, K, int(had_block), float(clip_ratio), _ptr(xq), _ptr(scale),
                                      _stream(x)))
    return xq, scale


def rcp_gemv_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(lib().rcp_gemv_workspace_bytes(M, N, K))


def make_workspace(M: int, N: int, K: int, device) -> torch.Tensor:
    """Zero-filled scratch for rcp_gemv_w2a4 (at least 16 bytes so that a pointer always exists)."""
    n = max(16, rcp_gemv_workspace_bytes(M, N, K))
    return torch.zeros((n + 3) // 4, dtype=torch.int32, device=device)


def rcp_gemv_w2a4(words, lut, xq, scale, y=None, workspace=None, S_dbg=None, variant="auto"):
    """words int32 [N][K/16], lut fp16 [N][4], xq uint8 [M][K/2], scale fp16 [M] -> y fp16 [M][N]."""
    _dev(words, torch.int32, "words")
    _dev(lut, torch.float16, "lut")
    _dev(xq, torch.uint8, "xq")
    _dev(scale, torch.float16, "scale")
    N, W = words.shape
    K = W * 16
    M = xq.shape[0]
    if xq.shape != (M, K // 2) or lut.shape != (N, 4) or scale.shape != (M,):
        raise ValueError("shape mismatch between words, lut, xq and scale")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=words.device)
    if workspace is None and rcp_gemv_workspace_bytes(M, N, K) > 0:
        workspace = make_workspace(M, N, K, words.device)
    v = VARIANTS[variant] if isinstance(variant, str) else int(variant)
    with _on(words):
        _check("rcp_gemv_w2a4",
               lib().rcp_gemv_w2a4_variant(v, _ptr(words), _ptr(lut), _ptr(xq), _ptr(scale), M, N, K, _ptr(y),
                                           _ptr(workspace), _ptr(S_dbg), _stream(words)))
    return y


def rcp_gemv_w2a4_grouped(words, lut, xq, scale, group=128, y=None, workspace=None, S_dbg=None, variant="auto"):
    """Group-wise grid: words int32 [N][K/16], lut fp16 [N][K/group][4], xq uint8 [M][K/2], scale fp16 [M]
    -> y fp16 [M][N]. S_dbg: int32 [M][N][K/group][4]."""
    _dev(words, torch.int32, "words")
    _dev(lut, torch.float16, "lut")
    _dev(xq, torch.uint8, "xq")
    _dev(scale, torch.float16, "scale")
    N, W = words.shape
    K = W * 16
    M = xq.shape[0]
    group = int(group)
    if group < 1 or K % group or xq.shape != (M, K // 2) or lut.shape != (N, K // group, 4) or scale.shape != (M,):
        raise ValueError("shape mismatch between words, lut, group, xq and scale")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=words.device)
    if workspace is None and rcp_gemv_workspace_bytes(M, N, K) > 0:
        workspace = make_workspace(M, N, K, words.device)
    v = VARIANTS[variant] if isinstance(variant, str) else int(variant)
    with _on(words):
        _check("rcp_gemv_w2a4_grouped",
               lib().rcp_gemv_w2a4_grouped_variant(v, _ptr(words), _ptr(lut), group, _ptr(xq), _ptr(scale), M, N, K,
                                                   _ptr(y), _ptr(workspace), _ptr(S_dbg), _stream(words)))
    return y


def rcp_gemv_w2a16(words, lut, x, y=None, digits=None, unit=None, workspace=None, S_dbg=None):
    """Weight-only form: words int32 [N][K/16], lut fp16 [N][4], x fp16 [M][K] -> y fp16 [M][N].
    digits int8 [M][4][K] and unit fp32 [M][4] receive the fixed-point form of x the kernels used.
    S_dbg int32 [4 M][N][4]: the per-code sums of every digit plane (checked instantiation of the kernel)."""
    _dev(words, torch.int32, "words")
    _dev(lut, torch.float16, "lut")
    _dev(x, torch.float16, "x")
    N, W = words.shape
    K = W * 16
    M = x.shape[0]
    if x.shape != (M, K) or lut.shape != (N, 4):
        raise ValueError("shape mismatch between words, lut and x")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=words.device)
    if digits is None:
        digits = torch.empty((M, 4, K), dtype=torch.int8, device=words.device)
    if unit is None:
        unit = torch.empty((M, 4), dtype=torch.float32, device=words.device)
    if workspace is None:
        workspace = make_workspace(M, N, K, words.device)
    with _on(words):
        _check("rcp_gemv_w2a16",
               lib().rcp_gemv_w2a16_checked(_ptr(words), _ptr(lut), _ptr(x), M, N, K, _ptr(y), _ptr(digits), _ptr(unit),
                                            _ptr(workspace), _ptr(S_dbg), _stream(words)))
    return y


def rcp_pack_weights3(codes: torch.Tensor):
    """3-bit codes uint8 [N][K] in {0..7} -> (words2 int32 [N][K/16], words1 int32 [N][K/32])."""
    _dev(codes, torch.uint8, "codes")
    N, K = codes.shape
    words2 = torch.empty((N, K // 16), dtype=torch.int32, device=codes.device)
    words1 = torch.empty((N, K // 32), dtype=torch.int32, device=codes.device)
    with _on(codes):
        _check("rcp_pack_weights3",
               lib().rcp_pack_weights3(_ptr(codes), N, K, _ptr(words2), _ptr(words1), _stream(codes)))
    return words2, words1


def rcp_gemv_w3a4(words2, words1, lut, xq, scale, group=0, y=None, S_dbg=None):
    """W3A4 GEMV: words2 int32 [N][K/16], words1 int32 [N][K/32], lut fp16 [N][8] (group=0) or [N][K/128][8]
    (group=128), xq uint8 [M][K/2], scale fp16 [M] -> y fp16 [M][N]."""
    _dev(words2, torch.int32, "words2")
    _dev(words1, torch.int32, "words1")
    _dev(lut, torch.float16, "lut")
    _dev(xq, torch.uint8, "xq")
    _dev(scale, torch.float16, "scale")
    N, W = words2.shape
    K = W * 16
    M = xq.shape[0]
    group = int(group)
    want = (N, 8) if group == 0 else (N, K // max(group, 1), 8)
    if words1.shape != (N, K // 32) or xq.shape != (M, K // 2) or tuple(lut.shape) != want or scale.shape != (M,):
        raise ValueError("shape mismatch between words2, words1, lut, group, xq and scale")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=words2.device)
    with _on(words2):
        _check("rcp_gemv_w3a4",
               lib().rcp_gemv_w3a4(_ptr(words2), _ptr(words1), _ptr(lut), group, _ptr(xq), _ptr(scale), M, N, K, _ptr(y),
                                   _ptr(S_dbg), _stream(words2)))
    return y


STATIC_SCRATCH_BYTES = 4096


def rcp_gemv_w2a4_static(words, lut, xq, scale, y=None):
    """Same result as rcp_gemv_w2a4, for callers that may not allocate device memory: the scratch
    is an array inside the library (STATIC_SCRATCH_BYTES, shared by all calls on the device, so
    calls that can overlap on the GPU must be serialized). Pass `y` to keep this wrapper from
    allocating the output; shapes that need more scratch raise RcpError with status -8."""
    _dev(words, torch.int32, "words")
    _dev(lut, torch.float16, "lut")
    _dev(xq, torch.uint8, "xq")
    _dev(scale, torch.float16, "scale")
    N, W = words.shape
    K = W * 16
    M = xq.shape[0]
    if xq.shape != (M, K // 2) or lut.shape != (N, 4) or scale.shape != (M,):
        raise ValueError("shape mismatch between words, lut, xq and scale")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=words.device)
    with _on(words):
        _check("rcp_gemv_w2a4_static",
               lib().rcp_gemv_w2a4_static(_ptr(words), _ptr(lut), _ptr(xq), _ptr(scale), M, N, K, _ptr(y),
                                          _stream(words)))
    return y


def rcp_linear_w2a4(x, had_block, clip_ratio, words, lut, group=0, y=None, xq=None, scale=None, workspace=None,
                    S_dbg=None):
    """x fp16 [M][K] -> y fp16 [M][N]: activation quantization and LUT GEMV in one call (one kernel for
    one token of 4096 or 8192 under one rotation block). lut fp16 [N][4] with group=0, [N][K/group][4]
    otherwise. xq / scale: optional outputs on the one-kernel path, required staging otherwise (pass them to
    be safe). S_dbg int32 [M][N][4] ([M][N][K/group][4]): the integer sums, from the checked instantiation
    of the kernel that runs anyway."""
    _dev(x, torch.float16, "x")
    _dev(words, torch.int32, "words")
    _dev(lut, torch.float16, "lut")
    M, K = x.shape
    N, W = words.shape
    group = int(group)
    want = (N, 4) if group == 0 else (N, K // max(group, 1), 4)
    if W * 16 != K or tuple(lut.shape) != want:
        raise ValueError("shape mismatch between x, words, lut and group")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float16, device=words.device)
    if workspace is None:
        workspace = make_workspace(M, N, K, words.device)
    with _on(words):
        _check("rcp_linear_w2a4",
               lib().rcp_linear_w2a4_checked(_ptr(x), M, K, int(had_block), float(clip_ratio), _ptr(words), _ptr(lut),
                                             group, N, _ptr(y), _ptr(xq), _ptr(scale), _ptr(workspace), _ptr(S_dbg),
                                             _stream(words)))
    return y


def rcp_linear_w2a4_launches(M: int, N: int, K: int, had_block: int, group: int = 0) -> int:
    """Kernel launches one rcp_linear_w2a4 call makes for a shape (host only)."""
    n = int(lib().rcp_linear_w2a4_launches(M, N, K, int(had_block), int(group)))
    if n < 0:
        raise RcpError("rcp_linear_w2a4_launches", n, lib().rcp_status_str(n).decode(), 0)
    return n


def rcp_linear_w2a4_host(x_host, had_block, clip_ratio, words, lut, y_host, x_dev, xq_dev, scale_dev, y_dev, workspace):
    """x_host fp16 [M][K] (host, ideally pinned) -> y_host fp16 [M][N] (host). Asynchronous on the
    current stream: synchronize before reading y_host."""
    M, K = x_host.shape
    N = words.shape[0]
    if x_host.is_cuda or y_host.is_cuda or x_host.dtype != torch.float16 or y_host.dtype != torch.float16:
        raise TypeError("x_host / y_host must be fp16 host tensors")
    with _on(words):
        _check("rcp_linear_w2a4_host",
               lib().rcp_linear_w2a4_host(_ptr(x_host), M, K, int(had_block), float(clip_ratio), _ptr(words), _ptr(lut),
                                          N, _ptr(y_host), _ptr(x_dev), _ptr(xq_dev), _ptr(scale_dev), _ptr(y_dev),
                                          _ptr(workspace), _stream(words)))
    return y_host
