"""CPU oracle for the RCP W2A4 decode hot path -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Thin ctypes wrapper over ``rcp_oracle.cpp`` (plain single-threaded C++, written from the
paper's definitions: Appendix A.2 for the Hadamard matrix, Section 4.4 and Appendix A.7 for
the tensor formats and the LUT product).  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library never does, and the two share no
code.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rcp_oracle.cpp")
_LIB = os.path.join(_HERE, "librcp_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
             "-o", _LIB, _SRC])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_f16_to_f32.restype = C.c_float
        _lib.orc_f16_to_f32.argtypes = [C.c_uint16]
        _lib.orc_f32_to_f16.restype = C.c_uint16
        _lib.orc_f32_to_f16.argtypes = [C.c_float]
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _c(a, dtype):
    a = np.ascontiguousarray(a)
    assert a.dtype == dtype, (a.dtype, dtype)
    return a


def f16_to_f32(bits: int) -> float:
    return float(lib().orc_f16_to_f32(int(bits)))


def f32_to_f16(x: float) -> int:
    return int(lib().orc_f32_to_f16(C.c_float(x)))


def hadamard_matrix(n: int) -> np.ndarray:
    """Normalized Sylvester Hadamard matrix H_n (Appendix A.2), dense float64."""
    H = np.empty((n, n), dtype=np.float64)
    rc = lib().orc_hadamard_matrix(C.c_int(n), _p(H))
    if rc:
        raise ValueError("n must be a power of two")
    return H


def rotate_exact_f64(x_f16_bits: np.ndarray, B: int) -> np.ndarray:
    x = _c(x_f16_bits, np.uint16)
    y = np.empty(x.shape, dtype=np.float64)
    K = x.shape[-1]
    for m in range(x.reshape(-1, K).shape[0]):
        rc = lib().orc_rotate_exact_f64(_p(x.reshape(-1, K)[m]), C.c_int(K), C.c_int(B), _p(y.reshape(-1, K)[m]))
        if rc:
            raise ValueError("bad block")
    return y


def rotate_f32(x_f16_bits: np.ndarray, B: int) -> np.ndarray:
    x = _c(x_f16_bits, np.uint16).reshape(-1)
    v = np.empty(x.shape, dtype=np.float32)
    rc = lib().orc_rotate_f32(_p(x), C.c_int(x.size), C.c_int(B), _p(v))
    if rc:
        raise ValueError("bad block")
    return v


def quantize_act(x_f16_bits: np.ndarray, had_block: int, clip_ratio: float = 1.0):
    """x: uint16 [M][K] (fp16 bit patterns). Returns dict(xq u8 [M][K/2], scale u16 [M], q i8 [M][K], v f32 [M][K])."""
    x = _c(x_f16_bits, np.uint16)
    M, K = x.shape
    xq = np.empty((M, K // 2), dtype=np.uint8)
    scale = np.empty((M,), dtype=np.uint16)
    q = np.empty((M, K), dtype=np.int8)
    v = np.empty((M, K), dtype=np.float32)
    rc = lib().orc_quantize_act(_p(x), C.c_int(M), C.c_int(K), C.c_int(had_block), C.c_float(clip_ratio),
                                _p(xq), _p(scale), _p(q), _p(v))
    if rc:
        raise ValueError(f"orc_quantize_act failed: {rc}")
    return dict(xq=xq, scale=scale, q=q, v=v)


def unpack_act(xq: np.ndarray) -> np.ndarray:
    xq = _c(xq, np.uint8)
    q = np.empty(xq.shape[:-1] + (xq.shape[-1] * 2,), dtype=np.int8)
    lib().orc_unpack_act(_p(xq), C.c_size_t(xq.size), _p(q))
    return q


def pack_weights(codes: np.ndarray) -> np.ndarray:
    codes = _c(codes, np.uint8)
    N, K = codes.shape
    words = np.empty((N, K // 16), dtype=np.uint32)
    rc = lib().orc_pack_weights(_p(codes), C.c_int(N), C.c_int(K), _p(words))
    if rc:
        raise ValueError(f"orc_pack_weights failed: {rc}")
    return words


def unpack_weights(words: np.ndarray) -> np.ndarray:
    words = _c(words, np.uint32)
    N, W = words.shape
    codes = np.empty((N, W * 16), dtype=np.uint8)
    lib().orc_unpack_weights(_p(words), C.c_int(N), C.c_int(W * 16), _p(codes))
    return codes


def gemv_w2a4(words, lut_bits, xq, scale_bits):
    """Returns dict(S int32 [M][N][4], y float64 [M][N], tol float64 [M][N])."""
    words = _c(words, np.uint32)
    lut = _c(lut_bits, np.uint16)
    xq = _c(xq, np.uint8)
    scale = _c(scale_bits, np.uint16)
    N, W = words.shape
    K = W * 16
    M = xq.shape[0]
    assert xq.shape == (M, K // 2) and lut.shape == (N, 4) and scale.shape == (M,)
    S = np.empty((M, N, 4), dtype=np.int32)
    y = np.empty((M, N), dtype=np.float64)
    tol = np.empty((M, N), dtype=np.float64)
    rc = lib().orc_gemv_w2a4(_p(words), _p(lut), _p(xq), _p(scale), C.c_int(M), C.c_int(N), C.c_int(K),
                             _p(S), _p(y), _p(tol))
    if rc:
        raise ValueError(f"orc_gemv_w2a4 failed: {rc}")
    return dict(S=S, y=y, tol=tol)


def gemv_direct(words, lut_bits, xq, scale_bits):
    """Direct sum over k. Returns dict(y float64 [M][N], acc_int int64 [M][N])."""
    words = _c(words, np.uint32)
    lut = _c(lut_bits, np.uint16)
    xq = _c(xq, np.uint8)
    scale = _c(scale_bits, np.uint16)
    N, W = words.shape
    K = W * 16
    M = xq.shape[0]
    y = np.empty((M, N), dtype=np.float64)
    ai = np.empty((M, N), dtype=np.int64)
    rc = lib().orc_gemv_direct(_p(words), _p(lut), _p(xq), _p(scale), C.c_int(M), C.c_int(N), C.c_int(K),
                               _p(y), _p(ai))
    if rc:
        raise ValueError(f"orc_gemv_direct failed: {rc}")
    return dict(y=y, acc_int=ai)


def percode_int(lut_bits, S):
    lut = _c(lut_bits, np.uint16)
    S = _c(S, np.int32)
    M, N, _ = S.shape
    ai = np.empty((M, N), dtype=np.int64)
    lib().orc_percode_int(_p(lut), _p(S), C.c_int(M), C.c_int(N), _p(ai))
    return ai


def dequant_weights(words, lut_bits):
    words = _c(words, np.uint32)
    lut = _c(lut_bits, np.uint16)
    N, W = words.shape
    Wd = np.empty((N, W * 16), dtype=np.float64)
    lib().orc_dequant_weights(_p(words), _p(lut), C.c_int(N), C.c_int(W * 16), _p(Wd))
    return Wd


def gemv_w2a4_grouped(words, lut_bits, xq, scale_bits, G):
    """Group-wise grid: lut uint16 [N][K/G][4]. Returns dict(S int32 [M][N][K/G][4], y, tol float64 [M][N])."""
    words = _c(words, np.uint32)
    lut = _c(lut_bits, np.uint16)
    xq = _c(xq, np.uint8)
    scale = _c(scale_bits, np.uint16)
    N, W = words.shape
    K = W * 16
    M = xq.shape[0]
    assert K % G == 0 and lut.shape == (N, K // G, 4) and xq.shape == (M, K // 2) and scale.shape == (M,)
    S = np.empty((M, N, K // G, 4), dtype=np.int32)
    y = np.empty((M, N), dtype=np.float64)
    tol = np.empty((M, N), dtype=np.float64)
    rc = lib().orc_gemv_w2a4_grouped(_p(words), _p(lut), _p(xq), _p(scale), C.c_int(M), C.c_int(N), C.c_int(K),
                                     C.c_int(G), _p(S), _p(y), _p(tol))
    if rc:
        raise ValueError(f"orc_gemv_w2a4_grouped failed: {rc}")
    return dict(S=S, y=y, tol=tol)


def gemv_direct_grouped(words, lut_bits, xq, scale_bits, G):
    """Direct sum over k with a grid per group. Returns dict(y float64 [M][N], acc_int int64 [M][N])."""
    words = _c(words, np.uint32)
    lut = _c(lut_bits, np.uint16)
    xq = _c(xq, np.uint8)
    scale = _c(scale_bits, np.uint16)
    N, W = words.shape
    K = W * 16
    M = xq.shape[0]
    assert K % G == 0 and lut.shape == (N, K // G, 4)
    y = np.empty((M, N), dtype=np.float64)
    ai = np.empty((M, N), dtype=np.int64)
    rc = lib().orc_gemv_direct_grouped(_p(words), _p(lut), _p(xq), _p(scale), C.c_int(M), C.c_int(N), C.c_int(K),
                                       C.c_int(G), _p(y), _p(ai))
    if rc:
        raise ValueError(f"orc_gemv_direct_grouped failed: {rc}")
    return dict(y=y, acc_int=ai)


def percode_int_grouped(lut_bits, S):
    lut = _c(lut_bits, np.uint16)
    S = _c(S, np.int32)
    M, N, NG, _ = S.shape
    assert lut.shape == (N, NG, 4)
    ai = np.empty((M, N), dtype=np.int64)
    lib().orc_percode_int_grouped(_p(lut), _p(S), C.c_int(M), C.c_int(N), C.c_int(NG), _p(ai))
    return ai


def ldp_export(w_f16_bits, sb, sg, s1, s2, G):
    """Partitioning quantizer export. w uint16 [N][K] (fp16 bits); sb, sg, s1, s2 float32 [N][K/G] (the
    sigmoids of beta, gamma, s_1, s_2). Returns dict(codes u8 [N][K], lut uint16 [N][K/G][4])."""
    w = _c(w_f16_bits, np.uint16)
    N, K = w.shape
    assert K % G == 0
    arrs = [_c(a, np.float32) for a in (sb, sg, s1, s2)]
    for a in arrs:
        assert a.shape == (N, K // G)
    codes = np.empty((N, K), dtype=np.uint8)
    lut = np.empty((N, K // G, 4), dtype=np.uint16)
    rc = lib().orc_ldp_export(_p(w), _p(arrs[0]), _p(arrs[1]), _p(arrs[2]), _p(arrs[3]), C.c_int(N), C.c_int(K),
                              C.c_int(G), _p(codes), _p(lut))
    if rc:
        raise ValueError(f"orc_ldp_export failed: {rc}")
    return dict(codes=codes, lut=lut)


def pack_weights3(codes):
    """3-bit codes u8 [N][K] -> (words2 uint32 [N][K/16], words1 uint32 [N][K/32])."""
    codes = _c(codes, np.uint8)
    N, K = codes.shape
    w2 = np.empty((N, K // 16), dtype=np.uint32)
    w1 = np.empty((N, K // 32), dtype=np.uint32)
    rc = lib().orc_pack_weights3(_p(codes), C.c_int(N), C.c_int(K), _p(w2), _p(w1))
    if rc:
        raise ValueError(f"orc_pack_weights3 failed: {rc}")
    return w2, w1


def unpack_weights3(words2, words1):
    w2 = _c(words2, np.uint32)
    w1 = _c(words1, np.uint32)
    N, W = w2.shape
    codes = np.empty((N, W * 16), dtype=np.uint8)
    lib().orc_unpack_weights3(_p(w2), _p(w1), C.c_int(N), C.c_int(W * 16), _p(codes))
    return codes


def gemv_w3a4(words2, words1, lut_bits, xq, scale_bits, G=None):
    """W3A4 GEMV. lut uint16 [N][K/G][8] (or [N][8] with G None = one grid per row).
    Returns dict(S int32 [M][N][K/G][8], y float64 [M][N], tol float64 [M][N])."""
    w2 = _c(words2, np.uint32)
    w1 = _c(words1, np.uint32)
    lut = _c(lut_bits, np.uint16)
    xq = _c(xq, np.uint8)
    scale = _c(scale_bits, np.uint16)
    N, W = w2.shape
    K = W * 16
    M = xq.shape[0]
    if G is None:
        G = K
    NG = K // G
    lut = lut.reshape(N, NG, 8)
    assert xq.shape == (M, K // 2) and w1.shape == (N, K // 32) and scale.shape == (M,)
    S = np.empty((M, N, NG, 8), dtype=np.int32)
    y = np.empty((M, N), dtype=np.float64)
    tol = np.empty((M, N), dtype=np.float64)
    rc = lib().orc_gemv_w3a4(_p(w2), _p(w1), _p(lut), _p(xq), _p(scale), C.c_int(M), C.c_int(N), C.c_int(K), C.c_int(G),
                             _p(S), _p(y), _p(tol))
    if rc:
        raise ValueError(f"orc_gemv_w3a4 failed: {rc}")
    return dict(S=S, y=y, tol=tol)


def gemv_w3a4_direct_int(words2, words1, lut_bits, xq, G=None):
    w2 = _c(words2, np.uint32)
    w1 = _c(words1, np.uint32)
    lut = _c(lut_bits, np.uint16)
    xq = _c(xq, np.uint8)
    N, W = w2.shape
    K = W * 16
    M = xq.shape[0]
    if G is None:
        G = K
    acc = np.empty((M, N), dtype=np.int64)
    rc = lib().orc_gemv_w3a4_direct_int(_p(w2), _p(w1), _p(lut), _p(xq), C.c_int(M), C.c_int(N), C.c_int(K), C.c_int(G),
                                        _p(acc))
    if rc:
        raise ValueError(f"orc_gemv_w3a4_direct_int failed: {rc}")
    return acc


def nf3_export(w_f16_bits, sb, sg, s1, table, zero_index, G):
    """3-bit export with a learnable centre. w uint16 [N][K]; sb, sg, s1 float32 [N][K/G]; table float32 [8]
    ascending with table[zero_index] == 0. Returns dict(codes u8 [N][K], lut uint16 [N][K/G][8])."""
    w = _c(w_f16_bits, np.uint16)
    N, K = w.shape
    assert K % G == 0
    arrs = [_c(a, np.float32) for a in (sb, sg, s1)]
    for a in arrs:
        assert a.shape == (N, K // G)
    t = _c(table, np.float32)
    assert t.shape == (8,)
    codes = np.empty((N, K), dtype=np.uint8)
    lut = np.empty((N, K // G, 8), dtype=np.uint16)
    rc = lib().orc_nf3_export(_p(w), _p(arrs[0]), _p(arrs[1]), _p(arrs[2]), _p(t), C.c_int(int(zero_index)), C.c_int(N),
                              C.c_int(K), C.c_int(G), _p(codes), _p(lut))
    if rc:
        raise ValueError(f"orc_nf3_export failed: {rc}")
    return dict(codes=codes, lut=lut)


def gemv_w2a16(words, lut_bits, x_f16_bits):
    """Weight-only GEMV by its definition. Returns dict(y float64 [M][N], labsx float64 [M][N], labs float64 [N])."""
    words = _c(words, np.uint32)
    lut = _c(lut_bits, np.uint16)
    x = _c(x_f16_bits, np.uint16)
    N, W = words.shape
    K = W * 16
    M = x.shape[0]
    assert x.shape == (M, K) and lut.shape == (N, 4)
    y = np.empty((M, N), dtype=np.float64)
    labsx = np.empty((M, N), dtype=np.float64)
    labs = np.empty((N,), dtype=np.float64)
    rc = lib().orc_gemv_w2a16(_p(words), _p(lut), _p(x), C.c_int(M), C.c_int(N), C.c_int(K), _p(y), _p(labsx), _p(labs))
    if rc:
        raise ValueError(f"orc_gemv_w2a16 failed: {rc}")
    return dict(y=y, labsx=labsx, labs=labs)


def percode_sums_i8(words, planes):
    """Per-code sums of signed 8-bit activation planes: planes int8 [C][K] -> S int32 [C][N][4]."""
    words = _c(words, np.uint32)
    a = _c(planes, np.int8)
    N, W = words.shape
    K = W * 16
    Cn = a.shape[0]
    assert a.shape == (Cn, K)
    S = np.empty((Cn, N, 4), dtype=np.int32)
    rc = lib().orc_percode_sums_i8(_p(words), _p(a), C.c_int(Cn), C.c_int(N), C.c_int(K), _p(S))
    if rc:
        raise ValueError(f"orc_percode_sums_i8 failed: {rc}")
    return S


def split_act16(x_f16_bits):
    """Base-64 fixed-point digits of fp16 activations. Returns dict(digits int8 [M][4][K], unit float64 [M][4])."""
    x = _c(x_f16_bits, np.uint16)
    M, K = x.shape
    digits = np.empty((M, 4, K), dtype=np.int8)
    unit = np.empty((M, 4), dtype=np.float64)
    rc = lib().orc_split_act16(_p(x), C.c_int(M), C.c_int(K), _p(digits), _p(unit))
    if rc:
        raise ValueError(f"orc_split_act16 failed: {rc}")
    return dict(digits=digits, unit=unit)
