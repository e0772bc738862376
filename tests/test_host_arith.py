"""The library's exact-arithmetic functions, compiled for the host, against the CPU oracle.

The key-element encoder, the value exponent and the packed-shift and table score datapaths are plain
integer code that nvcc also compiles for the host; this checks them exhaustively / on random
inputs without a GPU.  (The same functions run on the device in the -m gpu parity tests.)"""
import ctypes as C
import os
import subprocess

import numpy as np
import pytest

from oracle import sa_oracle as ora

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "host_harness.cu")
LIB = os.path.join(HERE, "_build", "libhh.so")
CSRC = os.path.join(HERE, "..", "paper_2609_09208_b200", "csrc")


@pytest.fixture(scope="module")
def hh():
    os.makedirs(os.path.dirname(LIB), exist_ok=True)
    deps = [SRC] + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cuh")]
    if not os.path.exists(LIB) or any(os.path.getmtime(d) > os.path.getmtime(LIB) for d in deps):
        subprocess.check_call(["/usr/local/cuda/bin/nvcc", "-std=c++17", "-O2", "-shared", "-Xcompiler", "-fPIC",
                               "-Wno-deprecated-gpu-targets", "-o", LIB, SRC])
    lib = C.CDLL(LIB)
    return lib


SCALES = [0x3C00, 0x7BFF, 0x3A66, 0x0400, 0x01F3, 0x4D2B, 0x0001, 0x2E66]


@pytest.mark.parametrize("k", [0, 1, 2, 4])
@pytest.mark.parametrize("s_bits", SCALES)
def test_encode_element_exhaustive_vs_oracle(hh, k, s_bits):
    mags = np.arange(0, s_bits + 1, dtype=np.uint16)
    vals = (mags | ((np.arange(len(mags)) % 2).astype(np.uint16) << 15)).astype(np.uint16)
    got = np.empty(len(vals), dtype=np.uint8)
    hh.hh_encode_many(C.c_int(k), vals.ctypes.data_as(C.c_void_p), C.c_int64(len(vals)), C.c_uint(s_bits),
                      got.ctypes.data_as(C.c_void_p))
    d = 64
    n_vec = (len(vals) + d - 2) // (d - 1)
    K = np.zeros((n_vec, d), dtype=np.uint16)
    K[:, 0] = s_bits
    flat = np.zeros(n_vec * (d - 1), dtype=np.uint16)
    flat[: len(vals)] = vals
    K[:, 1:] = flat.reshape(n_vec, d - 1)
    want = ora.encode_keys(K, k)[0][:, 1:].reshape(-1)[: len(vals)]
    assert np.array_equal(got, want)


def test_value_exponent_all_magnitudes(hh):
    mags = np.arange(0, 0x7C00, dtype=np.uint16)          # every finite binary16 magnitude
    V = np.zeros((len(mags), 64), dtype=np.uint16)
    V[:, 5] = mags
    _, g = ora.quantise_value(V)
    got = np.array([hh.hh_value_exponent(C.c_uint(int(m))) for m in mags], dtype=np.int8)
    assert np.array_equal(got, g)


@pytest.mark.parametrize("k", [0, 1, 2, 4])
@pytest.mark.parametrize("d", [64, 128])
def test_score_datapaths_equal_oracle_scores(hh, k, d):
    """Eight queries (two per 32-bit register) against one key through the kernel's word decoders
    and packed accumulators, including the cases that stress the 16-bit halves: every term
    negative at the largest shift, extreme queries, zero codes with and without a sign bit."""
    rng = np.random.default_rng(100 + k + d)
    out = np.zeros(8, dtype=np.int32)
    for trial in range(300):
        e = rng.integers(0, 8, d)
        j = rng.integers(0, 1 << k, d)
        sgn = rng.integers(0, 2, d)
        if trial % 7 == 1:
            e[:] = 0                                # largest shift everywhere
        if trial % 7 == 2:
            sgn[:] = 1
        if trial % 7 == 3:
            j[:] = (1 << k) - 1
        codes = ((sgn << 7) | (e << 4) | (j << (4 - k))).astype(np.uint8)
        if trial % 3 == 0:
            codes[e == 7] = 0x70                    # canonical zeros (otherwise: zero codes keep their sign bit)
        else:
            codes[e == 7] &= 0xF0                   # a zero code has no mantissa bits
        q = rng.integers(-127, 128, (8, d)).astype(np.int8)
        if trial % 5 == 1:
            q[:] = 127
        if trial % 5 == 2:
            q[::2] = -127
            q[1::2] = 127
        if trial % 5 == 3:
            q[:] = -127
        want, ov = ora.scores(q, codes[None, None, :], k, 6 + k)
        assert ov == 0
        hh.hh_score8(C.c_int(k), codes.ctypes.data_as(C.c_void_p), q.ctypes.data_as(C.c_void_p), C.c_int(d),
                     C.c_int(0), out.ctypes.data_as(C.c_void_p))
        assert np.array_equal(out.astype(np.int64), want[:, 0]), (trial, out, want[:, 0])
        if k == 0:
            hh.hh_score8(C.c_int(0), codes.ctypes.data_as(C.c_void_p), q.ctypes.data_as(C.c_void_p), C.c_int(d),
                         C.c_int(1), out.ctypes.data_as(C.c_void_p))
            assert np.array_equal(out.astype(np.int64), want[:, 0]), ("nibble", trial)
        else:
            # the table datapath of the mantissa codes gives the same integers
            hh.hh_score8_table(C.c_int(k), codes.ctypes.data_as(C.c_void_p), q.ctypes.data_as(C.c_void_p), C.c_int(d),
                               out.ctypes.data_as(C.c_void_p))
            assert np.array_equal(out.astype(np.int64), want[:, 0]), ("table", trial, out, want[:, 0])
            if k in (1, 2):
                # ... and so does the dense planar container (nibbles + mantissa bit planes)
                hh.hh_score8_planar(C.c_int(k), codes.ctypes.data_as(C.c_void_p), q.ctypes.data_as(C.c_void_p), C.c_int(d),
                                    out.ctypes.data_as(C.c_void_p))
                assert np.array_equal(out.astype(np.int64), want[:, 0]), ("planar", trial, out, want[:, 0])
        # the non-default kernels that run the shifts on the integer multiplier: the same integers again
        for path in (() if k == 0 else (0, 1) if k in (1, 2) else (0,)):
            hh.hh_score8_mul(C.c_int(k), codes.ctypes.data_as(C.c_void_p), q.ctypes.data_as(C.c_void_p), C.c_int(d),
                             C.c_int(path), out.ctypes.data_as(C.c_void_p))
            assert np.array_equal(out.astype(np.int64), want[:, 0]), ("shift by multiply", path, trial, out, want[:, 0])
        # the non-default kernels without any multiply-add (sign flip and add as logic and add instructions)
        for path in ((0, 1) if k in (0, 1, 2) else (0,)):
            hh.hh_score8_alu(C.c_int(k), codes.ctypes.data_as(C.c_void_p), q.ctypes.data_as(C.c_void_p), C.c_int(d),
                             C.c_int(path), out.ctypes.data_as(C.c_void_p))
            assert np.array_equal(out.astype(np.int64), want[:, 0]), ("adds on the ALU pipe", path, trial, out, want[:, 0])
