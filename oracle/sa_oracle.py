"""ctypes front end of the CPU oracle (``sa_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's
CPU-baseline leg, never by the library.  It marshals numpy arrays to the plain C++
functions and holds none of the method's arithmetic.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sa_oracle.cpp")
_LIB = os.path.join(_HERE, "libsa_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ if the shared object is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call([
            "g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
            "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ora_code_value.restype = C.c_double
        _lib.ora_code_value.argtypes = [C.c_uint8, C.c_int]
        _lib.ora_half_to_double.restype = C.c_double
        _lib.ora_half_to_double.argtypes = [C.c_uint16]
        _lib.ora_double_to_half.restype = C.c_uint16
        _lib.ora_double_to_half.argtypes = [C.c_double]
        _lib.ora_scores.restype = C.c_int64
        _lib.ora_decode_attention.restype = C.c_int64
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _half_bits(x):
    """Accept float16 or uint16 arrays; return a C-contiguous uint16 view of the bits."""
    x = np.ascontiguousarray(x)
    if x.dtype == np.float16:
        return x.view(np.uint16)
    assert x.dtype == np.uint16, x.dtype
    return x


def codebook(k: int):
    mags = np.zeros(7 * 16, dtype=np.float64)
    n = lib().ora_codebook(C.c_int(k), _p(mags), C.c_int(mags.size))
    return n, mags[: (n - 1) // 2].copy()


def code_value(code: int, k: int) -> float:
    return lib().ora_code_value(C.c_uint8(code), C.c_int(k))


def half_to_double(bits: int) -> float:
    return lib().ora_half_to_double(C.c_uint16(bits))


def double_to_half(x: float) -> int:
    return lib().ora_double_to_half(C.c_double(x))


def hadamard_fp16(x):
    """Rotate each length-d row of a float16 array; returns a new float16 array."""
    out = np.array(_half_bits(x), copy=True)
    d = out.shape[-1]
    lib().ora_hadamard_fp16(_p(out), C.c_int64(out.size // d), C.c_int(d))
    return out.view(np.float16)


def encode_keys(K, k: int):
    """K [..., d] float16 -> (codes uint8 [..., d], scales float16 [...])."""
    kb = _half_bits(K)
    d = kb.shape[-1]
    n = kb.size // d
    codes = np.empty(kb.shape, dtype=np.uint8)
    scales = np.empty(kb.shape[:-1], dtype=np.uint16)
    lib().ora_encode_keys(_p(kb), C.c_int64(n), C.c_int(d), C.c_int(k), _p(codes), _p(scales))
    return codes, scales.view(np.float16)


def quantise_query(Q):
    qb = _half_bits(Q)
    d = qb.shape[-1]
    n = qb.size // d
    qhat = np.empty(qb.shape, dtype=np.int8)
    delta = np.empty(qb.shape[:-1], dtype=np.float32)
    lib().ora_quantise_query(_p(qb), C.c_int64(n), C.c_int(d), _p(qhat), _p(delta))
    return qhat, delta


def quantise_value(V):
    vb = _half_bits(V)
    d = vb.shape[-1]
    n = vb.size // d
    vhat = np.empty(vb.shape, dtype=np.int8)
    g = np.empty(vb.shape[:-1], dtype=np.int8)
    lib().ora_quantise_value(_p(vb), C.c_int64(n), C.c_int(d), _p(vhat), _p(g))
    return vhat, g


def scores(qhat, codes, k: int, F: int):
    """qhat int8 [Hq, d]; codes uint8 [T, Hkv, d] -> (A int64 [Hq, T], n_overflow)."""
    qhat = np.ascontiguousarray(qhat, dtype=np.int8)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    Hq, d = qhat.shape
    T, Hkv, d2 = codes.shape
    assert d == d2 and Hq % Hkv == 0
    A = np.empty((Hq, T), dtype=np.int64)
    ov = lib().ora_scores(_p(qhat), _p(codes), C.c_int64(T), C.c_int(Hq), C.c_int(Hkv), C.c_int(d),
                          C.c_int(k), C.c_int(F), _p(A))
    return A, int(ov)


def attention_twopass(A, delta, scales, vhat, g, F: int):
    A = np.ascontiguousarray(A, dtype=np.int64)
    delta = np.ascontiguousarray(delta, dtype=np.float32)
    sb = _half_bits(scales)
    vhat = np.ascontiguousarray(vhat, dtype=np.int8)
    g = np.ascontiguousarray(g, dtype=np.int8)
    Hq, T = A.shape
    T2, Hkv, d = vhat.shape
    assert T == T2
    O = np.empty((Hq, d), dtype=np.float64)
    lib().ora_attention_twopass(_p(A), _p(delta), _p(sb), _p(vhat), _p(g), C.c_int64(T), C.c_int(Hq),
                                C.c_int(Hkv), C.c_int(d), C.c_int(F), _p(O))
    return O


def attention_online(A, delta, scales, vhat, g, F: int, tile: int = 128, splits: int = 1):
    A = np.ascontiguousarray(A, dtype=np.int64)
    delta = np.ascontiguousarray(delta, dtype=np.float32)
    sb = _half_bits(scales)
    vhat = np.ascontiguousarray(vhat, dtype=np.int8)
    g = np.ascontiguousarray(g, dtype=np.int8)
    Hq, T = A.shape
    T2, Hkv, d = vhat.shape
    assert T == T2
    O = np.empty((Hq, d), dtype=np.float32)
    lib().ora_attention_online(_p(A), _p(delta), _p(sb), _p(vhat), _p(g), C.c_int64(T), C.c_int(Hq),
                               C.c_int(Hkv), C.c_int(d), C.c_int(F), C.c_int(tile), C.c_int(splits), _p(O))
    return O


def attention_shiftav(A, delta, scales, vhat, g, F: int, N: int, k_max: int):
    """Eq. (6), (7): log2-quantised weights and shift-based A.V.  Returns (O float64 [Hq, d],
    zr int32 [Hq, T] rounded binary32 logits, M int32 [Hq])."""
    A = np.ascontiguousarray(A, dtype=np.int64)
    delta = np.ascontiguousarray(delta, dtype=np.float32)
    sb = _half_bits(scales)
    vhat = np.ascontiguousarray(vhat, dtype=np.int8)
    g = np.ascontiguousarray(g, dtype=np.int8)
    Hq, T = A.shape
    T2, Hkv, d = vhat.shape
    assert T == T2 and 0 <= k_max <= N <= 40
    O = np.empty((Hq, d), dtype=np.float64)
    zr = np.empty((Hq, max(T, 1)), dtype=np.int32)
    M = np.empty(Hq, dtype=np.int32)
    lib().ora_attention_shiftav(_p(A), _p(delta), _p(sb), _p(vhat), _p(g), C.c_int64(T), C.c_int(Hq),
                                C.c_int(Hkv), C.c_int(d), C.c_int(F), C.c_int(N), C.c_int(k_max), _p(O),
                                _p(zr), _p(M))
    return O, zr[:, :T], M


def sdpa_fp16(Q, K, V):
    """Q [Hq, d], K/V [T, Hkv, d] float16 -> O [Hq, d] float64."""
    qb, kb, vb = _half_bits(Q), _half_bits(K), _half_bits(V)
    Hq, d = qb.shape
    T, Hkv, _ = kb.shape
    O = np.empty((Hq, d), dtype=np.float64)
    lib().ora_sdpa_fp16(_p(qb), _p(kb), _p(vb), C.c_int64(T), C.c_int(Hq), C.c_int(Hkv), C.c_int(d), _p(O))
    return O


def decode_attention(Q, K, V, cu_lens, k: int, F: int, hadamard: bool = False,
                     want_scores: bool = False, n_threads: int = 1):
    """Whole decode step for a ragged batch.

    Q [B, Hq, d], K/V [sum T_b, Hkv, d] float16, cu_lens int64 [B + 1].
    Returns dict(O float64 [B, Hq, d], A int64 [B, Hq, max_T] or None, overflow, stage_seconds).
    """
    qb, kb, vb = _half_bits(Q), _half_bits(K), _half_bits(V)
    cu = np.ascontiguousarray(cu_lens, dtype=np.int64)
    B, Hq, d = qb.shape
    Hkv = kb.shape[1]
    lens = np.diff(cu)
    max_T = int(lens.max()) if B else 0
    O = np.zeros((B, Hq, d), dtype=np.float64)
    A = np.zeros((B, Hq, max(max_T, 1)), dtype=np.int64) if want_scores else None
    st = np.zeros(4, dtype=np.float64)
    ov = lib().ora_decode_attention(
        _p(qb), _p(kb), _p(vb), _p(cu), C.c_int(B), C.c_int(Hq), C.c_int(Hkv), C.c_int(d), C.c_int(k),
        C.c_int(F), C.c_int(1 if hadamard else 0), _p(O), _p(A) if want_scores else None,
        C.c_int64(max(max_T, 1)), C.c_int(n_threads), _p(st))
    return dict(O=O, A=A, overflow=int(ov), stage_seconds=st)


def encode_keys_int8(K):
    """Uniform INT8 comparison code: K [..., d] float16 -> (codes int8 [..., d], scales float16 [...])."""
    kb = _half_bits(K)
    d = kb.shape[-1]
    codes = np.empty(kb.shape, dtype=np.int8)
    scales = np.empty(kb.shape[:-1], dtype=np.uint16)
    lib().ora_encode_keys_int8(_p(kb), C.c_int64(kb.size // d), C.c_int(d), _p(codes), _p(scales))
    return codes, scales.view(np.float16)


def scores_int8(qhat, codes):
    """qhat int8 [Hq, d]; codes int8 [T, Hkv, d] -> A int64 [Hq, T]."""
    qhat = np.ascontiguousarray(qhat, dtype=np.int8)
    codes = np.ascontiguousarray(codes, dtype=np.int8)
    Hq, d = qhat.shape
    T, Hkv, _ = codes.shape
    A = np.empty((Hq, T), dtype=np.int64)
    lib().ora_scores_int8(_p(qhat), _p(codes), C.c_int64(T), C.c_int(Hq), C.c_int(Hkv), C.c_int(d), _p(A))
    return A


def attention_twopass_int8(A, delta, scales, vhat, g):
    A = np.ascontiguousarray(A, dtype=np.int64)
    delta = np.ascontiguousarray(delta, dtype=np.float32)
    sb = _half_bits(scales)
    vhat = np.ascontiguousarray(vhat, dtype=np.int8)
    g = np.ascontiguousarray(g, dtype=np.int8)
    Hq, T = A.shape
    _, Hkv, d = vhat.shape
    O = np.empty((Hq, d), dtype=np.float64)
    lib().ora_attention_twopass_int8(_p(A), _p(delta), _p(sb), _p(vhat), _p(g), C.c_int64(T), C.c_int(Hq),
                                     C.c_int(Hkv), C.c_int(d), _p(O))
    return O


def hardware_threads() -> int:
    return int(lib().ora_hardware_threads())
