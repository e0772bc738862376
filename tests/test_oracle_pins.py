"""Pins for the CPU oracle: each check fixes the oracle to something other than itself —
constants the paper prints, closed forms, exhaustive brute force with exact arithmetic,
and library routines for the special cases that reduce to textbook operations.
No GPU is needed."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import sa_oracle as ora
from paper_2609_09208_b200 import synth

KS = [0, 1, 2, 4]
E = 6


def _golden():
    out = {}
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")
    for line in open(path):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


G = _golden()


# ------------------------------------------------------------------ helpers (independent of the oracle)
def half_bits_to_fraction(h: int) -> Fraction:
    sign = -1 if h >> 15 else 1
    ex, man = (h >> 10) & 0x1F, h & 0x3FF
    if ex == 0:
        return sign * Fraction(man, 1 << 24)
    return sign * Fraction(1024 + man) * Fraction(2) ** (ex - 25)


def decode_byte(code: int, k: int) -> Fraction:
    """Value of a canonical code byte, from the closed form of eq. (2) / eq. (5)."""
    e = (code >> 4) & 7
    if e == 7:
        return Fraction(0)
    j = (code & 0xF) >> (4 - k)
    v = Fraction((1 << k) + j, 1 << (k + e))
    return -v if code & 0x80 else v


def brute_force_codes(a_bits: np.ndarray, s_bits: int, k: int) -> np.ndarray:
    """Nearest codeword in log2 over the whole extended grid, by exhaustive search.

    float64 logs decide; any element whose two best candidates are closer than 1e-11 in
    log2 distance is re-decided with exact rational arithmetic."""
    a = a_bits.astype(np.uint16).view(np.float16).astype(np.float64)
    s = float(np.array([s_bits], dtype=np.uint16).view(np.float16)[0])
    es = np.arange(0, 48)
    js = np.arange(0, 1 << k)
    logc = (np.log2((1 << k) + js)[None, :] - k - es[:, None]).reshape(-1)       # [n_cand]
    cand_e = np.repeat(es, len(js))
    cand_j = np.tile(js, len(es))
    out = np.empty(a.shape, dtype=np.uint8)
    nz = np.abs(a) > 0
    out[~nz] = 0x70
    idx = np.nonzero(nz)[0]
    for lo in range(0, len(idx), 4096):
        sel = idx[lo:lo + 4096]
        logu = np.log2(np.abs(a[sel]) / s)
        dist = np.abs(logu[:, None] - logc[None, :])
        order = np.argsort(dist, axis=1)[:, :2]
        best = order[:, 0].copy()
        d0 = dist[np.arange(len(sel)), order[:, 0]]
        d1 = dist[np.arange(len(sel)), order[:, 1]]
        for r in np.nonzero(d1 - d0 < 1e-11)[0]:
            u = abs(half_bits_to_fraction(int(a_bits[sel[r]]))) / half_bits_to_fraction(s_bits)
            c0 = Fraction((1 << k) + int(cand_j[order[r, 0]]), 1 << (k + int(cand_e[order[r, 0]])))
            c1 = Fraction((1 << k) + int(cand_j[order[r, 1]]), 1 << (k + int(cand_e[order[r, 1]])))
            lo_c, hi_c = min(c0, c1), max(c0, c1)
            assert u * u != lo_c * hi_c, "an exact tie cannot occur"
            pick_hi = u * u > lo_c * hi_c
            want = hi_c if pick_hi else lo_c
            best[r] = order[r, 0] if want == c0 else order[r, 1]
        e = cand_e[best]
        j = cand_j[best]
        code = np.where(e >= 7, 0x70, ((a_bits[sel] >> 15) << 7) | (e << 4) | (j << (4 - k))).astype(np.uint8)
        out[sel] = code
    return out


# ------------------------------------------------------------------ number formats
def test_half_to_double_all_bit_patterns_match_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float64)
    got = np.array([ora.half_to_double(int(b)) for b in bits])
    finite = np.isfinite(ref)
    assert np.array_equal(got[finite], ref[finite])
    assert np.all(np.isinf(got[np.isinf(ref)]))


def test_double_to_half_matches_numpy_rounding():
    rng = np.random.default_rng(1)
    xs = np.concatenate([
        rng.standard_normal(20000) * np.exp(rng.uniform(-18, 11, 20000)),
        np.arange(65536, dtype=np.uint16).view(np.float16).astype(np.float64)[::7],
        # exact ties between neighbouring binary16 values, normal and subnormal
        np.array([1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 2.0 ** -25, 3 * 2.0 ** -25, 65519.9, 65504.0, 0.0]),
    ])
    xs = xs[np.isfinite(xs)]
    with np.errstate(over="ignore"):
        ref = xs.astype(np.float16).view(np.uint16)
    got = np.array([ora.double_to_half(float(x)) for x in xs], dtype=np.uint16)
    assert np.array_equal(got, ref)


# ------------------------------------------------------------------ codebook
@pytest.mark.parametrize("k,levels", [(0, 15), (1, 29), (2, 57), (4, 225)])
def test_codebook_level_counts_and_closed_form(k, levels):
    n, mags = ora.codebook(k)
    assert n == levels
    want = sorted(float(Fraction((1 << k) + j, 1 << (k + e))) for e in range(E + 1) for j in range(1 << k))
    assert mags.tolist() == want
    assert len(set(mags.tolist())) == len(mags)


def test_codebook_matches_paper_constants():
    assert ora.codebook(0)[0] == G["levels_min"]
    assert ora.codebook(4)[0] == G["levels_max"]
    assert G["E_for_4_bits"] == E


@pytest.mark.parametrize("k", KS)
def test_code_value_every_byte(k):
    for code in range(256):
        low_bits = (code & 0xF) & ((1 << (4 - k)) - 1)
        if low_bits:
            continue  # not a left-aligned k-bit mantissa
        assert ora.code_value(code, k) == float(decode_byte(code, k))


def test_binary_attention_is_the_e0_special_case():
    # restricted to e = 0 the PoT-4 code has the two levels -1 and +1
    assert {ora.code_value(0x00, 0), ora.code_value(0x80, 0)} == {1.0, -1.0}


# ------------------------------------------------------------------ key encode
SCALES = [0x3C00,  # 1.0
          0x7BFF,  # 65504, largest finite
          0x3A66,  # 0.7998
          0x0400,  # 2^-14, smallest normal
          0x01F3,  # a subnormal scale
          0x4D2B]  # 20.67


@pytest.mark.parametrize("k", KS)
@pytest.mark.parametrize("s_bits", SCALES)
def test_encode_exhaustive_against_brute_force(k, s_bits):
    """Every binary16 magnitude not above the scale, against exhaustive nearest-in-log2 search."""
    mags = np.arange(0, s_bits + 1, dtype=np.uint16)
    signs = (np.arange(len(mags)) % 3 == 0).astype(np.uint16) << 15
    vals = mags | signs
    d = 64
    per = d - 1
    n_vec = (len(vals) + per - 1) // per
    K = np.zeros((n_vec, d), dtype=np.uint16)
    K[:, 0] = s_bits                       # pins the vector's scale
    flat = np.zeros(n_vec * per, dtype=np.uint16)
    flat[: len(vals)] = vals
    K[:, 1:] = flat.reshape(n_vec, per)
    codes, scales = ora.encode_keys(K, k)
    assert np.all(scales.view(np.uint16) == s_bits)
    want = brute_force_codes(K.reshape(-1), s_bits, k).reshape(K.shape)
    bad = np.nonzero(codes != want)
    assert len(bad[0]) == 0, (k, hex(s_bits), K[bad][:5], codes[bad][:5], want[bad][:5])
    assert np.all(codes[:, 0] == 0x00)     # the scale element itself is +1.0: e = 0, j = 0


@pytest.mark.parametrize("k", KS)
def test_encode_tiny_tensor_exact_rational_brute_force(k):
    """Brute force with exact rationals only (no floating point anywhere) on a tiny tensor."""
    rng = np.random.default_rng(10 + k)
    K = (rng.standard_normal((6, 8)) * np.exp(rng.standard_normal((1, 8)))).astype(np.float16)
    K[0, 3] = 0.0
    K[2, 5] = -0.0
    codes, scales = ora.encode_keys(K, k)
    kb = K.view(np.uint16)
    grid = [(e, j, Fraction((1 << k) + j, 1 << (k + e))) for e in range(0, 48) for j in range(1 << k)]
    for v in range(K.shape[0]):
        s = max(abs(half_bits_to_fraction(int(b))) for b in kb[v])
        assert half_bits_to_fraction(int(scales.view(np.uint16)[v])) == s
        for m in range(K.shape[1]):
            a = abs(half_bits_to_fraction(int(kb[v, m])))
            if a == 0:
                assert codes[v, m] == 0x70
                continue
            u = a / s
            # nearest in log2 == smallest max(u/c, c/u)
            e, j, c = min(grid, key=lambda t: max(u / t[2], t[2] / u))
            want = 0x70 if e >= 7 else ((int(kb[v, m]) >> 15) << 7) | (e << 4) | (j << (4 - k))
            assert codes[v, m] == want


@pytest.mark.parametrize("k", KS)
def test_encode_relative_error_bounds(k):
    rng = np.random.default_rng(3)
    K = rng.standard_normal((512, 64)).astype(np.float16)
    codes, scales = ora.encode_keys(K, k)
    val = np.vectorize(lambda c: float(decode_byte(int(c), k)))(codes) * scales.astype(np.float64)[:, None]
    kept = codes != 0x70
    rel = val[kept] / K.astype(np.float64)[kept] - 1.0
    n = 1 << k
    lo, hi = math.sqrt(n / (n + 1)) - 1.0, math.sqrt((n + 1) / n) - 1.0   # widest gap: j = 0 -> 1
    assert rel.min() >= lo - 1e-12 and rel.max() <= hi + 1e-12
    if k == 0:
        assert abs(lo - G["log2_rel_err_lo"]) < 5e-4 and abs(hi - G["log2_rel_err_hi"]) < 5e-4
        assert rel.min() < -0.28 and rel.max() > 0.40       # the bounds are attained
    # dropped elements are exactly those below the geometric mean of c(6,0) and c(7, 2^k - 1)
    u = np.abs(K.astype(np.float64)) / scales.astype(np.float64)[:, None]
    thr = math.sqrt(float(Fraction(n, n << 6) * Fraction(2 * n - 1, n << 7)))
    assert np.array_equal(~kept, u < thr)


def test_encode_rms_error_log_uniform_matches_closed_form():
    # u = 2^-t, t uniform: RMS of the relative error is sqrt(int_{-1/2}^{1/2} (2^x - 1)^2 dx)
    closed = math.sqrt(1.5 / (2 * math.log(2)) - 2 * (math.sqrt(2) - 1 / math.sqrt(2)) / math.log(2) + 1)
    assert abs(closed - 0.2043) < 1e-4
    assert abs(closed - G["log2_rel_err_rms"]) < 2e-3            # the paper prints ~0.203
    t = (np.arange(63 * 4000) + 0.5) / (63 * 4000) * 6.0
    K = np.ones((4000, 64), dtype=np.float16)
    K[:, 1:] = (2.0 ** -t).reshape(4000, 63).astype(np.float16)
    codes, _ = ora.encode_keys(K, 0)
    val = np.vectorize(lambda c: float(decode_byte(int(c), 0)))(codes)
    rel = val[:, 1:] / K.astype(np.float64)[:, 1:] - 1.0
    assert abs(math.sqrt(np.mean(rel ** 2)) - closed) < 1.5e-3


@pytest.mark.parametrize("k", KS)
def test_encode_idempotent_sign_symmetric_scale_covariant(k):
    # every codeword times a power-of-two scale is representable and must encode to itself
    # (codewords with e = 0 and j > 0 lie above the scale, which is the row maximum, so no input maps to them)
    words = [(e, j) for e in range(E + 1) for j in range(1 << k) if not (e == 0 and j > 0)]
    for s in [1.0, 2.0 ** -3, 2.0 ** 7]:
        row = np.zeros((1, 128), dtype=np.float16)
        row[0, 0] = s
        for i, (e, j) in enumerate(words):
            row[0, 1 + i] = s * float(Fraction((1 << k) + j, 1 << (k + e))) * (-1 if i % 2 else 1)
        codes, scales = ora.encode_keys(row[:, : 1 + len(words)], k)
        for i, (e, j) in enumerate(words):
            assert codes[0, 1 + i] == ((0x80 if i % 2 else 0) | (e << 4) | (j << (4 - k)))
    rng = np.random.default_rng(5)
    K = rng.standard_normal((64, 64)).astype(np.float16)
    c0, s0 = ora.encode_keys(K, k)
    c1, s1 = ora.encode_keys(-K, k)
    assert np.array_equal(s0, s1)
    assert np.array_equal(np.where(c0 == 0x70, 0x70, c0 ^ 0x80), c1)
    c2, s2 = ora.encode_keys(K * np.float16(8.0), k)
    assert np.array_equal(c0, c2) and np.array_equal(s2.astype(np.float64), s0.astype(np.float64) * 8)


def test_encode_zero_vector_and_underflow_fraction():
    codes, scales = ora.encode_keys(np.zeros((2, 64), dtype=np.float16), 4)
    assert np.all(codes == 0x70) and np.all(scales.view(np.uint16) == 0)
    K = np.random.default_rng(7).standard_normal((4096, 64)).astype(np.float16)
    codes, _ = ora.encode_keys(K, 0)
    frac = np.mean(codes == 0x70)
    assert 0.01 < frac < 0.06      # a few per cent of Gaussian entries fall below 2^-6.5 of the row maximum


# ------------------------------------------------------------------ query and value quantisers
def test_query_quantiser_hand_example_and_properties():
    Q = np.zeros((1, 64), dtype=np.float16)
    Q[0, :6] = [1.0, -0.5, 0.25, 0.5, -1.0, 0.0078125]
    qhat, delta = ora.quantise_query(Q)
    # 63.5 rounds to the even 64, 31.75 to 32, 0.9921875 to 1
    assert qhat[0, :6].tolist() == [127, -64, 32, 64, -127, 1]
    assert delta[0] == np.float32(1.0) / np.float32(127.0)
    rng = np.random.default_rng(11)
    Q = rng.standard_normal((256, 64)).astype(np.float16)
    qhat, delta = ora.quantise_query(Q)
    assert np.all(np.abs(qhat).max(axis=1) == 127)
    err = np.abs(Q.astype(np.float64) - delta[:, None].astype(np.float64) * qhat)
    assert np.all(err <= 0.5 * delta[:, None] * (1 + 1e-5))
    qz, dz = ora.quantise_query(np.zeros((1, 64), dtype=np.float16))
    assert not qz.any() and dz[0] == 0


def test_value_quantiser_hand_examples_and_properties():
    V = np.zeros((4, 64), dtype=np.float16)
    V[0, 0], V[1, 0], V[2, 0] = 1.0, 127.0 / 64.0, 2.0
    V[0, 1] = 0.0234375        # 1.5 / 64 -> tie, rounds to even 2
    V[0, 2] = 0.0390625        # 2.5 / 64 -> tie, rounds to even 2
    vhat, g = ora.quantise_value(V)
    assert g.tolist() == [6, 6, 5, 0]
    assert vhat[0, 0] == 64 and vhat[1, 0] == 127 and vhat[2, 0] == 64
    assert vhat[0, 1] == 2 and vhat[0, 2] == 2
    rng = np.random.default_rng(12)
    V = (rng.standard_normal((512, 64)) * np.exp(rng.uniform(-8, 8, (512, 1)))).astype(np.float16)
    vhat, g = ora.quantise_value(V)
    amax = np.abs(V.astype(np.float64)).max(axis=1)
    scaled = amax * 2.0 ** g
    assert np.all((scaled > 63.5) & (scaled <= 127))
    err = np.abs(V.astype(np.float64) - vhat * 2.0 ** (-g[:, None].astype(np.float64)))
    assert np.all(err <= 2.0 ** (-g[:, None].astype(np.float64) - 1))
    # extreme magnitudes of binary16
    big = np.full((1, 64), 65504.0, dtype=np.float16)
    tiny = np.zeros((1, 64), dtype=np.float16)
    tiny.view(np.uint16)[0, 0] = 1
    assert ora.quantise_value(big)[1][0] == -10 and ora.quantise_value(tiny)[1][0] == 30


# ------------------------------------------------------------------ integer scores
@pytest.mark.parametrize("k", KS)
def test_scores_equal_exact_rational_sum(k):
    rng = np.random.default_rng(20 + k)
    Hq, Hkv, d, T, F = 4, 2, 64, 40, E + k
    K = (rng.standard_normal((T, Hkv, d)) * np.exp(rng.standard_normal((1, Hkv, d)))).astype(np.float16)
    codes, _ = ora.encode_keys(K, k)
    qhat, _ = ora.quantise_query(rng.standard_normal((Hq, d)).astype(np.float16))
    A, ov = ora.scores(qhat, codes, k, F)
    assert ov == 0
    for h in range(Hq):
        for t in range(T):
            exact = sum(Fraction(int(qhat[h, m])) * decode_byte(int(codes[t, h // (Hq // Hkv), m]), k)
                        for m in range(d)) * (1 << F)
            assert exact.denominator == 1 and int(exact) == A[h, t]
    bound = d * 127 * ((1 << (k + 1)) - 1) * (1 << (F - k))
    assert np.abs(A).max() <= bound < 2 ** 31


def test_scores_bound_special_cases_and_family_consistency():
    assert 64 * 127 * 2 ** 7 == G["acc_bound_d64_F7"]
    d = 64
    qhat = np.full((1, d), 127, dtype=np.int8)
    ones = np.zeros((3, 1, d), dtype=np.uint8)          # e = 0, sigma = +, j = 0 everywhere
    A, _ = ora.scores(qhat, ones, 0, 7)
    assert np.all(A == G["acc_bound_d64_F7"])            # the bound of section II-C is attained
    rng = np.random.default_rng(30)
    qhat = rng.integers(-127, 128, (2, d)).astype(np.int8)
    A, _ = ora.scores(qhat, ones, 0, 6)
    assert np.all(A == 64 * qhat.astype(np.int64).sum(axis=1, keepdims=True))
    zeros = np.full((3, 1, d), 0x70, dtype=np.uint8)
    assert not ora.scores(qhat, zeros, 4, 10)[0].any()
    # a PoT-Mk key with all-zero mantissas equals the PoT-4 key of the same (sigma, e), times 2^k
    c0 = (rng.integers(0, 2, (9, 1, d)) << 7 | rng.integers(0, 8, (9, 1, d)) << 4).astype(np.uint8)
    c0[c0 == 0xF0] = 0x70
    base, _ = ora.scores(qhat, c0, 0, E)
    for k in (1, 2, 4):
        Ak, _ = ora.scores(qhat, c0, k, E + k)
        assert np.array_equal(Ak, base << k)
    # a left-aligned M1 / M2 byte read as an M4 code has the same value
    for k in (1, 2):
        ck = c0 | (rng.integers(0, 1 << k, c0.shape) << (4 - k)).astype(np.uint8)
        ck[(c0 >> 4) & 7 == 7] = 0x70
        Ak, _ = ora.scores(qhat, ck, k, E + k)
        A4, _ = ora.scores(qhat, ck, 4, E + 4)
        assert np.array_equal(A4, Ak << (4 - k))


def test_scores_gqa_mapping():
    rng = np.random.default_rng(31)
    Hq, Hkv, d, T = 8, 2, 64, 5
    codes = ora.encode_keys(rng.standard_normal((T, Hkv, d)).astype(np.float16), 1)[0]
    qhat = rng.integers(-127, 128, (Hq, d)).astype(np.int8)
    A, _ = ora.scores(qhat, codes, 1, 7)
    for h in range(Hq):
        single, _ = ora.scores(qhat[h:h + 1], codes[:, h // 4:h // 4 + 1], 1, 7)
        assert np.array_equal(single[0], A[h])


# ------------------------------------------------------------------ softmax and A.V
def _attention_inputs(seed, Hq=8, Hkv=2, d=64, T=300, k=1):
    rng = np.random.default_rng(seed)
    K = rng.standard_normal((T, Hkv, d)).astype(np.float16)
    V = rng.standard_normal((T, Hkv, d)).astype(np.float16)
    Q = (rng.standard_normal((Hq, d)) * 2).astype(np.float16)
    codes, scales = ora.encode_keys(K, k)
    qhat, delta = ora.quantise_query(Q)
    vhat, g = ora.quantise_value(V)
    A, _ = ora.scores(qhat, codes, k, E + k)
    return A, delta, scales, vhat, g, E + k


def test_twopass_matches_library_softmax():
    from scipy.special import softmax
    A, delta, scales, vhat, g, F = _attention_inputs(40)
    Hq, T = A.shape
    Hkv, d = vhat.shape[1], vhat.shape[2]
    O = ora.attention_twopass(A, delta, scales, vhat, g, F)
    for h in range(Hq):
        kv = h // (Hq // Hkv)
        logits = A[h] * float(delta[h]) * scales[:, kv].astype(np.float64) / 2 ** F / math.sqrt(d)
        w = softmax(logits)
        want = w @ (vhat[:, kv].astype(np.float64) * 2.0 ** (-g[:, kv, None].astype(np.float64)))
        assert abs(w.sum() - 1) < 1e-12
        assert np.max(np.abs(O[h] - want)) < 1e-12


def test_online_equals_twopass_for_any_tile_and_split():
    A, delta, scales, vhat, g, F = _attention_inputs(41, T=700)
    ref = ora.attention_twopass(A, delta, scales, vhat, g, F)
    base = ora.attention_online(A, delta, scales, vhat, g, F, tile=128, splits=1)
    assert np.max(np.abs(base - ref)) < 1e-5
    for tile, splits in [(1, 1), (7, 3), (64, 5), (128, 8), (700, 1), (33, 64)]:
        o = ora.attention_online(A, delta, scales, vhat, g, F, tile=tile, splits=splits)
        assert np.max(np.abs(o - ref)) < 1e-5
        assert np.max(np.abs(o - base)) < 2e-6


def test_softmax_special_cases():
    A, delta, scales, vhat, g, F = _attention_inputs(42, T=64)
    # one cached key: the output is that key's dequantised value row, exactly
    O1 = ora.attention_twopass(A[:, :1], delta, scales[:1], vhat[:1], g[:1], F)
    for h in range(A.shape[0]):
        kv = h // 4
        assert np.array_equal(O1[h], vhat[0, kv] * 2.0 ** (-float(g[0, kv])))
    # equal scores: the output is the mean of the dequantised values
    Oz = ora.attention_twopass(np.zeros_like(A), delta, scales, vhat, g, F)
    mean = (vhat.astype(np.float64) * 2.0 ** (-g[..., None].astype(np.float64))).mean(axis=0)
    assert np.max(np.abs(Oz[0] - mean[0])) < 1e-12
    # permuting the keys does not change the result
    perm = np.random.default_rng(1).permutation(A.shape[1])
    Op = ora.attention_twopass(A[:, perm], delta, scales[perm], vhat[perm], g[perm], F)
    assert np.max(np.abs(Op - ora.attention_twopass(A, delta, scales, vhat, g, F))) < 1e-12
    # identical value rows: the weights sum to one, so the output is that row
    vsame = np.broadcast_to(vhat[:1], vhat.shape).copy()
    gsame = np.broadcast_to(g[:1], g.shape).copy()
    Os = ora.attention_twopass(A, delta, scales, vsame, gsame, F)
    assert np.max(np.abs(Os[0] - vhat[0, 0] * 2.0 ** (-float(g[0, 0])))) < 1e-12
    # empty cache
    assert not ora.attention_twopass(A[:, :0], delta, scales[:0], vhat[:0], g[:0], F).any()
    assert not ora.attention_online(A[:, :0], delta, scales[:0], vhat[:0], g[:0], F).any()


# ------------------------------------------------------------------ eq. (6), (7): log2 weights, shift A.V
def test_shiftav_rounded_logits_and_integer_maximum():
    """The rounded logits are the nearest integers of the logit (formed in binary32, so compared
    with the fp64 logit up to binary32 rounding), M is the ceiling of the largest one, k >= 0 and
    the best key has k in {0, 1}."""
    A, delta, scales, vhat, g, F = _attention_inputs(50, T=300)
    Hq, T = A.shape
    Hkv, d = vhat.shape[1], vhat.shape[2]
    _, zr, M = ora.attention_shiftav(A, delta, scales, vhat, g, F, 15, 15)
    for h in range(Hq):
        kv = h // (Hq // Hkv)
        z = A[h] * float(delta[h]) * scales[:, kv].astype(np.float64) / 2 ** F / math.sqrt(d) * math.log2(math.e)
        tol = 1e-5 * (1 + np.abs(z))
        assert np.all(np.abs(zr[h] - z) <= 0.5 + tol)
        assert M[h] >= z.max() - tol.max() and M[h] < z.max() + 1 + tol.max()
        k = M[h] - zr[h]
        assert k.min() in (0, 1) and np.all(k >= 0)


def test_shiftav_equals_exact_rational_softmax_of_rounded_logits():
    """With N and k_max large enough that nothing is dropped, eq. (7) over eq. (6) is the softmax in
    base 2 of the ROUNDED logits applied to the dequantised values: checked with exact rationals and
    against the library softmax."""
    from scipy.special import softmax
    A, delta, scales, vhat, g, F = _attention_inputs(51, T=60)
    Hq, T = A.shape
    Hkv, d = vhat.shape[1], vhat.shape[2]
    O, zr, M = ora.attention_shiftav(A, delta, scales, vhat, g, F, 40, 40)
    assert int((M[:, None] - zr).max()) + int(g.max()) - int(g.min()) <= 40       # nothing is dropped
    for h in range(Hq):
        kv = h // (Hq // Hkv)
        w = [Fraction(2) ** int(zr[h, t]) for t in range(T)]
        den = sum(w)
        for m in range(0, d, 7):
            num = sum(w[t] * int(vhat[t, kv, m]) * Fraction(2) ** (-int(g[t, kv])) for t in range(T))
            assert abs(float(num / den) - O[h, m]) <= 1e-12 * max(1.0, abs(O[h, m]))
        wl = softmax(zr[h].astype(np.float64) * math.log(2.0))
        want = wl @ (vhat[:, kv].astype(np.float64) * 2.0 ** (-g[:, kv, None].astype(np.float64)))
        assert np.max(np.abs(O[h] - want)) < 1e-11


def test_shiftav_hand_cases_for_both_drop_rules():
    """One head, d = 1, F = 6, three keys with logits 0.2, -3.1, -19.8 (or -2.2): rounded logits
    0, -3, -20 (-2), M = 1, k = 1, 4, 21 (3).  Worked by hand:
      k_max = 15 drops the third key everywhere:  O = (10*2^14 - 20*2^11) / (2^14 + 2^11) * 2^-2 = 5/3;
      g = (0, 0, 20) makes the third key's shift index 15 - 3 + 0 - 20 < 0: it leaves the numerator but
      stays in the normaliser:  O = (10*2^14 - 20*2^11) / (2^14 + 2^11 + 2^12) = 60/11."""
    c = math.log2(math.e) / 64.0
    delta = np.array([1.0], dtype=np.float32)
    scales = np.ones((3, 1), dtype=np.float16)
    vhat = np.array([10, -20, 99], dtype=np.int8).reshape(3, 1, 1)
    A = np.array([[round(0.2 / c), round(-3.1 / c), round(-19.8 / c)]], dtype=np.int64)
    O, zr, M = ora.attention_shiftav(A, delta, scales, vhat, np.array([[2], [2], [5]], dtype=np.int8), 6, 15, 15)
    assert zr.tolist() == [[0, -3, -20]] and M.tolist() == [1]
    assert abs(O[0, 0] - 5.0 / 3.0) < 1e-12
    A[0, 2] = round(-2.2 / c)
    O, zr, M = ora.attention_shiftav(A, delta, scales, vhat, np.array([[0], [0], [20]], dtype=np.int8), 6, 15, 15)
    assert zr.tolist() == [[0, -3, -2]] and M.tolist() == [1]
    assert abs(O[0, 0] - 60.0 / 11.0) < 1e-12
    # with room for the small value (N = 24) the third key comes back: 99 * 2^-20 * 2^-3 joins the numerator
    O, _, _ = ora.attention_shiftav(A, delta, scales, vhat, np.array([[0], [0], [20]], dtype=np.int8), 6, 24, 24)
    want = (10 * 2.0 ** -1 - 20 * 2.0 ** -4 + 99 * 2.0 ** -23) / (2.0 ** -1 + 2.0 ** -4 + 2.0 ** -3)
    assert abs(O[0, 0] - want) < 1e-12


def test_shiftav_special_cases_and_distance_to_the_unquantised_softmax():
    A, delta, scales, vhat, g, F = _attention_inputs(52, T=64)
    # one cached key: its dequantised value row, exactly; equal scores: the mean (equal value scales)
    O1, _, _ = ora.attention_shiftav(A[:, :1], delta, scales[:1], vhat[:1], g[:1], F, 15, 15)
    for h in range(A.shape[0]):
        assert np.array_equal(O1[h], vhat[0, h // 4] * 2.0 ** (-float(g[0, h // 4])))
    g0 = np.zeros_like(g)
    Oz, _, _ = ora.attention_shiftav(np.zeros_like(A), delta, scales, vhat, g0, F, 15, 15)
    assert np.max(np.abs(Oz[0] - vhat[:, 0].astype(np.float64).mean(axis=0))) < 1e-12
    # empty cache
    assert not ora.attention_shiftav(A[:, :0], delta, scales[:0], vhat[:0], g[:0], F, 15, 15)[0].any()
    # every weight is within a factor sqrt(2) of the unquantised one, so the output stays near the
    # two-pass softmax (a second quantisation: the paper reports +0.13 .. +0.15 perplexity for it)
    Oq, _, _ = ora.attention_shiftav(A, delta, scales, vhat, g, F, 15, 15)
    Or = ora.attention_twopass(A, delta, scales, vhat, g, F)
    spread = (vhat.astype(np.float64) * 2.0 ** (-g[..., None].astype(np.float64))).std()
    assert 0 < np.abs(Oq - Or).mean() < 0.25 * spread


# ------------------------------------------------------------------ rotation
@pytest.mark.parametrize("d", [64, 128])
def test_hadamard_matches_library_matrix_and_is_an_involution(d):
    from scipy.linalg import hadamard
    rng = np.random.default_rng(50)
    x = rng.standard_normal((32, d)).astype(np.float16)
    y = ora.hadamard_fp16(x)
    want = x.astype(np.float64) @ hadamard(d).T / math.sqrt(d)
    assert np.max(np.abs(y.astype(np.float64) - want)) < 2.5e-3       # one binary16 rounding of O(1) values
    back = ora.hadamard_fp16(y)
    assert np.max(np.abs(back.astype(np.float64) - x.astype(np.float64))) < 6e-3
    if d == 64:
        # small integers stay exact through the butterflies and the 1/8 scale
        xi = rng.integers(-4, 5, (8, d)).astype(np.float16)
        assert np.array_equal(ora.hadamard_fp16(xi).astype(np.float64),
                              xi.astype(np.float64) @ hadamard(d).T / 8)


def test_hadamard_preserves_scores_and_flattens_outliers():
    rng = np.random.default_rng(51)
    d = 64
    K = synth.outlier_keys_fp16(rng, 256, 1, d)[:, 0]
    Q = rng.standard_normal((4, d)).astype(np.float16)
    s0 = Q.astype(np.float64) @ K.astype(np.float64).T
    s1 = ora.hadamard_fp16(Q).astype(np.float64) @ ora.hadamard_fp16(K).astype(np.float64).T
    assert np.max(np.abs(s0 - s1)) < 5e-3 * np.abs(s0).max()

    def eps_s(kk, qq, k=4):
        codes, scales = ora.encode_keys(kk, k)
        qhat, delta = ora.quantise_query(qq)
        A, _ = ora.scores(qhat, codes[:, None, :], k, E + k)
        S_hat = A * delta[:, None].astype(np.float64) * scales.astype(np.float64)[None, :] / 2 ** (E + k)
        S = qq.astype(np.float64) @ kk.astype(np.float64).T
        return np.linalg.norm(S_hat - S) / np.linalg.norm(S)
    assert eps_s(ora.hadamard_fp16(K), ora.hadamard_fp16(Q)) < eps_s(K, Q)


# ------------------------------------------------------------------ FP16 reference and the whole step
def test_sdpa_fp16_matches_torch():
    import torch
    rng = np.random.default_rng(60)
    Hq, Hkv, d, T = 8, 2, 64, 200
    Q = rng.standard_normal((Hq, d)).astype(np.float16)
    K = rng.standard_normal((T, Hkv, d)).astype(np.float16)
    V = rng.standard_normal((T, Hkv, d)).astype(np.float16)
    O = ora.sdpa_fp16(Q, K, V)
    q = torch.from_numpy(Q.astype(np.float64))[:, None, :]                            # [Hq, 1, d]
    kk = torch.from_numpy(K.astype(np.float64)).permute(1, 0, 2).repeat_interleave(Hq // Hkv, 0)
    vv = torch.from_numpy(V.astype(np.float64)).permute(1, 0, 2).repeat_interleave(Hq // Hkv, 0)
    want = torch.nn.functional.scaled_dot_product_attention(q, kk, vv)[:, 0].numpy()
    assert np.max(np.abs(O - want)) < 1e-12


def test_decode_step_is_the_composition_and_threads_do_not_change_it():
    case = synth.make_case("t", [37, 0, 130], 8, 2, 64, 2, outliers=True, seed=70)
    r1 = ora.decode_attention(case.Q, case.K, case.V, case.cu_lens, 2, E + 2, want_scores=True)
    r4 = ora.decode_attention(case.Q, case.K, case.V, case.cu_lens, 2, E + 2, want_scores=True, n_threads=4)
    assert np.array_equal(r1["O"], r4["O"]) and np.array_equal(r1["A"], r4["A"]) and r1["overflow"] == 0
    assert not r1["O"][1].any()                        # the empty sequence gives zeros
    b = 2
    K = case.K[case.cu_lens[b]:case.cu_lens[b + 1]]
    V = case.V[case.cu_lens[b]:case.cu_lens[b + 1]]
    codes, scales = ora.encode_keys(K, 2)
    qhat, delta = ora.quantise_query(case.Q[b])
    vhat, g = ora.quantise_value(V)
    A, _ = ora.scores(qhat, codes, 2, E + 2)
    assert np.array_equal(A, r1["A"][b][:, :130])
    assert np.array_equal(ora.attention_twopass(A, delta, scales, vhat, g, E + 2), r1["O"][b])
    # with rotation: same as rotating Q and K first
    rh = ora.decode_attention(case.Q, case.K, case.V, case.cu_lens, 2, E + 2, hadamard=True)
    rr = ora.decode_attention(ora.hadamard_fp16(case.Q), ora.hadamard_fp16(case.K), case.V, case.cu_lens, 2, E + 2)
    assert np.array_equal(rh["O"], rr["O"])


def test_score_error_roughly_halves_per_mantissa_bit():
    """Soft check of the trend the paper reports for its quantiser family (synthetic Gaussian keys)."""
    rng = np.random.default_rng(80)
    d, T = 64, 2048
    K = rng.standard_normal((T, d)).astype(np.float16)
    Q = rng.standard_normal((16, d)).astype(np.float16)
    S = Q.astype(np.float64) @ K.astype(np.float64).T
    eps = {}
    for k in KS:
        codes, scales = ora.encode_keys(K, k)
        val = np.vectorize(lambda c: float(decode_byte(int(c), k)))(codes) * scales.astype(np.float64)[:, None]
        Sh = Q.astype(np.float64) @ val.T
        eps[k] = np.linalg.norm(Sh - S) / np.linalg.norm(S)
    assert 1.6 < eps[0] / eps[1] < 2.6 and 1.6 < eps[1] / eps[2] < 2.6 and 2.8 < eps[2] / eps[4] < 5.0
    assert 0.15 < eps[0] < 0.25


def test_quantised_attention_approaches_fp16_attention():
    case = synth.make_case("t", [512], 8, 2, 64, 4, seed=81)
    ref = ora.sdpa_fp16(case.Q[0], case.K, case.V)
    err = {}
    for k in KS:
        O = ora.decode_attention(case.Q, case.K, case.V, case.cu_lens, k, E + k)["O"][0]
        err[k] = np.max(np.abs(O - ref))
    assert err[4] < err[1] < err[0] and err[4] < 0.03


# ------------------------------------------------------------------ uniform INT8 comparison code
def test_int8_key_code_hand_example_and_error_bound():
    K = np.zeros((2, 64), dtype=np.float16)
    K[0, :6] = [2.0, -1.0, 0.5, 1.0, -2.0, 0.015625]
    codes, scales = ora.encode_keys_int8(K)
    assert codes[0, :6].tolist() == [127, -64, 32, 64, -127, 1]      # 63.5 -> 64 and 31.75 -> 32: ties to even / nearest
    assert float(scales[0]) == 2.0 and not codes[1].any() and float(scales[1]) == 0.0
    rng = np.random.default_rng(90)
    K = (rng.standard_normal((300, 64)) * np.exp(rng.standard_normal((1, 64)))).astype(np.float16)
    codes, scales = ora.encode_keys_int8(K)
    step = scales.astype(np.float64) / 127.0
    assert np.all(np.abs(codes).max(axis=1) == 127)
    assert np.all(np.abs(K.astype(np.float64) - step[:, None] * codes) <= 0.5 * step[:, None] * (1 + 1e-5))


def test_int8_scores_are_integer_dot_products_and_softmax_matches_library():
    from scipy.special import softmax
    rng = np.random.default_rng(91)
    Hq, Hkv, d, T = 8, 2, 64, 200
    K = rng.standard_normal((T, Hkv, d)).astype(np.float16)
    V = rng.standard_normal((T, Hkv, d)).astype(np.float16)
    Q = rng.standard_normal((Hq, d)).astype(np.float16)
    codes, scales = ora.encode_keys_int8(K)
    qhat, delta = ora.quantise_query(Q)
    vhat, g = ora.quantise_value(V)
    A = ora.scores_int8(qhat, codes)
    for h in range(Hq):
        kv = h // 4
        want = codes[:, kv].astype(np.int64) @ qhat[h].astype(np.int64)          # numpy integer matmul
        assert np.array_equal(A[h], want)
    O = ora.attention_twopass_int8(A, delta, scales, vhat, g)
    for h in range(Hq):
        kv = h // 4
        logits = A[h] * float(delta[h]) * scales[:, kv].astype(np.float64) / 127.0 / math.sqrt(d)
        w = softmax(logits)
        want = w @ (vhat[:, kv].astype(np.float64) * 2.0 ** (-g[:, kv, None].astype(np.float64)))
        assert np.max(np.abs(O[h] - want)) < 1e-12
    # whole step with k = 8, and its accuracy next to the 8-bit power-of-two code (the paper: within ~2x)
    case = synth.make_case("t", [400], 8, 2, 64, 4, seed=92)
    ref = ora.sdpa_fp16(case.Q[0], case.K, case.V)
    o8 = ora.decode_attention(case.Q, case.K, case.V, case.cu_lens, 8, 0)["O"][0]
    o4 = ora.decode_attention(case.Q, case.K, case.V, case.cu_lens, 4, 10)["O"][0]
    e8, e4 = np.max(np.abs(o8 - ref)), np.max(np.abs(o4 - ref))
    assert e8 < 0.02 and e8 < e4 < 6 * e8
