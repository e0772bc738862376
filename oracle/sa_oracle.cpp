// CPU oracle for shift-accumulate decode attention.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the CUDA
// library is checked against.  It shares no code, header, table or helper with the
// CUDA path, and nothing in the product path may call it.  Only the tests, the
// smoke check and the benchmark's CPU-baseline leg load it.
//
// Every function follows one passage of the paper ("Shift-Accumulate Attention:
// Multiplier-Free Query-Key Products for Transformer Decoding"); the passage is
// named above the function.  Floating point is fp64 except where a decision that
// produces an integer (a quantised code) has to be taken in one fixed precision on
// both sides; those places say so.
//
// Parity status: every function here is pinned by tests that do not use the oracle
// to check itself (exhaustive brute force, exact rational arithmetic, closed forms,
// textbook special cases).  One exception: ora_attention_shiftav (the paper's
// non-default shift-based A.V) takes two constants, N and k_max, whose values the paper
// does not print: its arithmetic is pinned, those two values are "parity unpinned".
//
// Plain loops, no SIMD, no blocking, no fusion.  Compile with
//   g++ -O2 -std=c++17 -ffp-contract=off -fPIC -shared -pthread
#include <cmath>
#include <cstdint>
#include <cstring>
#include <ctime>
#include <limits>
#include <thread>
#include <vector>

namespace {

// ---------------------------------------------------------------------------------
// IEEE binary16 <-> double, written out from the format definition.
// ---------------------------------------------------------------------------------
double half_bits_to_double(uint16_t h) {
    const int sign = (h >> 15) & 1;
    const int ex = (h >> 10) & 0x1f;
    const int man = h & 0x3ff;
    double v;
    if (ex == 0) {
        v = std::ldexp(static_cast<double>(man), -24);  // subnormal or zero
    } else if (ex == 31) {
        v = man ? std::numeric_limits<double>::quiet_NaN()
                : std::numeric_limits<double>::infinity();
    } else {
        v = std::ldexp(static_cast<double>(1024 + man), ex - 25);
    }
    return sign ? -v : v;
}

// Round a double to the nearest binary16 (ties to even) and return its bits.
uint16_t double_to_half_bits(double x) {
    const uint16_t sign = std::signbit(x) ? 0x8000u : 0u;
    double a = std::fabs(x);
    if (std::isnan(a)) return static_cast<uint16_t>(sign | 0x7e00u);
    if (a == 0.0) return sign;
    int e2;
    std::frexp(a, &e2);               // a = f * 2^e2, f in [0.5, 1)
    int e = e2 - 1;                   // a in [2^e, 2^(e+1))
    const int qexp = (e < -14) ? -24 : (e - 10);  // spacing of binary16 values near a
    // a / 2^qexp is exact (power-of-two scaling); nearbyint rounds ties to even
    // in the default rounding mode.
    double n = std::nearbyint(std::ldexp(a, -qexp));
    double r = std::ldexp(n, qexp);
    if (r >= 65520.0) return static_cast<uint16_t>(sign | 0x7c00u);  // overflow -> inf
    if (r == 0.0) return sign;
    std::frexp(r, &e2);
    e = e2 - 1;
    if (e < -14) {                    // subnormal: value = man * 2^-24
        const int man = static_cast<int>(std::ldexp(r, 24));
        return static_cast<uint16_t>(sign | man);
    }
    const int man = static_cast<int>(std::ldexp(r, 10 - e)) - 1024;
    return static_cast<uint16_t>(sign | ((e + 15) << 10) | man);
}

constexpr int kE = 6;          // largest exponent of a 3-bit exponent field, eq. (2)
constexpr int kZeroExp = 7;    // the reserved code e = E + 1, eq. (2)

// Canonical one-byte form of a code used for comparisons with the CUDA library:
// bit 7 = sign (1 = negative), bits 6..4 = e (7 = exact zero), bits 3..0 = mantissa
// j left-aligned (j << (4 - k)).  The zero code is always 0x70.
uint8_t pack_code(int negative, int e, int j, int k) {
    if (e >= kZeroExp) return 0x70;
    return static_cast<uint8_t>((negative ? 0x80 : 0) | (e << 4) | (j << (4 - k)));
}

// Magnitude of codeword (e, j) of the k-bit-mantissa family relative to the scale,
// eq. (2) for k = 0 and eq. (5) for k >= 1:  (1 + j / 2^k) * 2^-e.
double codeword(int e, int j, int k) {
    return std::ldexp(static_cast<double>((1 << k) + j), -k - e);
}

// ---------------------------------------------------------------------------------
// Key element encode.  Section II-A (signed power-of-two code with per-vector scale,
// zero code), section II-D (nearest-in-log2 rounding; mantissa family).
//
// a  = |K_jm| and s = the vector's scale, both exact binary16 values held in double.
// The codewords are taken on the grid extended to every integer e >= 0 ("underflow"
// is decided after rounding).  With c_lo <= a/s < c_hi adjacent grid points, the
// nearer one in log2 is c_hi exactly when (a/s)^2 >= c_lo * c_hi.  That test is
// evaluated without division as a^2 >= s^2 * c_lo * c_hi; all four factors are
// short dyadic rationals, so every product below is exact in double.
// ---------------------------------------------------------------------------------
void encode_element(double a, double s, int k, int* e_out, int* j_out) {
    // smallest e with s * 2^-e <= a
    int e = 0;
    while (std::ldexp(s, -e) > a) ++e;
    // largest j in the binade with s * c(e, j) <= a
    int j = 0;
    while (j + 1 < (1 << k) && s * codeword(e, j + 1, k) <= a) ++j;
    const double c_lo = codeword(e, j, k);
    const double c_hi = codeword(e, j + 1, k);  // j + 1 == 2^k is 2^-(e-1): next binade
    const double lhs = a * a;
    const double rhs = (s * s) * (c_lo * c_hi);
    if (lhs >= rhs) {
        ++j;
        if (j == (1 << k)) { j = 0; --e; }
    }
    *e_out = e;
    *j_out = j;
}

}  // namespace

extern "C" {

int ora_version() { return 1; }

// Positive magnitudes of the codebook in ascending order; returns the number of
// distinct signed levels including zero.  Eq. (2), eq. (5), Table I ("15-225").
int ora_codebook(int k, double* mags, int cap) {
    int n = 0;
    for (int e = kE; e >= 0; --e)
        for (int j = 0; j < (1 << k); ++j) {
            if (n < cap) mags[n] = codeword(e, j, k);
            ++n;
        }
    return 2 * n + 1;
}

// Signed value (relative to the scale) of a canonical code byte.
double ora_code_value(uint8_t code, int k) {
    const int e = (code >> 4) & 7;
    if (e == kZeroExp) return 0.0;
    const int j = (code & 0xf) >> (4 - k);
    const double v = codeword(e, j, k);
    return (code & 0x80) ? -v : v;
}

double ora_half_to_double(uint16_t h) { return half_bits_to_double(h); }
uint16_t ora_double_to_half(double x) { return double_to_half_bits(x); }

// ---------------------------------------------------------------------------------
// Walsh-Hadamard rotation (the score-preserving outlier transform of the related-
// work and results sections).  Sylvester order, in-place butterflies with strides
// 1, 2, 4, ..., d/2; each butterfly is (a, b) <- (a + b, a - b).  The arithmetic is
// binary32 with one rounding per add, in this fixed order, so that a second
// implementation of the same recipe gives the same bits; the result is scaled by
// 1/sqrt(d) (one binary32 multiply) and rounded to binary16.  The rotated vector
// feeds a quantiser, so this is a place where both sides must round identically.
// ---------------------------------------------------------------------------------
void ora_hadamard_fp16(uint16_t* x, int64_t n_vec, int d) {
    const float scale = (d == 64) ? 0.125f : (d == 128 ? 0.088388346f
                                  : static_cast<float>(1.0 / std::sqrt(static_cast<double>(d))));
    std::vector<float> buf(d);
    for (int64_t v = 0; v < n_vec; ++v) {
        uint16_t* row = x + v * d;
        for (int m = 0; m < d; ++m) buf[m] = static_cast<float>(half_bits_to_double(row[m]));
        for (int h = 1; h < d; h <<= 1)
            for (int i = 0; i < d; ++i)
                if ((i & h) == 0) {
                    const float a = buf[i], b = buf[i + h];
                    buf[i] = a + b;
                    buf[i + h] = a - b;
                }
        for (int m = 0; m < d; ++m) {
            const float r = buf[m] * scale;
            row[m] = double_to_half_bits(static_cast<double>(r));
        }
    }
}

// ---------------------------------------------------------------------------------
// Key encode: per-vector scale and per-element code.  Section II-A: the scale is
// per key vector and the key is normalised by it so that all exponents are >= 0;
// here the scale is the vector's largest magnitude, which is itself a binary16
// value.  An all-zero vector has scale 0 and all-zero codes.
// K is [n_vec, d] binary16 bits; codes [n_vec, d] canonical bytes; scales [n_vec].
// ---------------------------------------------------------------------------------
void ora_encode_keys(const uint16_t* K, int64_t n_vec, int d, int k,
                     uint8_t* codes, uint16_t* scales) {
    for (int64_t v = 0; v < n_vec; ++v) {
        const uint16_t* row = K + v * d;
        uint16_t smax_bits = 0;
        for (int m = 0; m < d; ++m) {
            const uint16_t mag = row[m] & 0x7fff;  // binary16 magnitudes order like their bits
            if (mag > smax_bits) smax_bits = mag;
        }
        scales[v] = smax_bits;
        const double s = half_bits_to_double(smax_bits);
        for (int m = 0; m < d; ++m) {
            const double a = half_bits_to_double(row[m] & 0x7fff);
            if (a == 0.0) { codes[v * d + m] = 0x70; continue; }
            int e, j;
            encode_element(a, s, k, &e, &j);
            codes[v * d + m] = pack_code(row[m] >> 15, e, j, k);
        }
    }
}

// ---------------------------------------------------------------------------------
// Query quantisation, eq. (2): Q_im ~ Delta_i * qhat_im with a per-vector step and
// qhat in [-127, 127] (the bound 127 is the one used in the exactness paragraph).
// The integer qhat is decided in binary32, the precision the kernel uses:
//   inv = 127 / amax (one IEEE divide), qhat = clamp(round-half-even(Q * inv)),
//   Delta = amax / 127 (one IEEE divide).  amax = 0 gives Delta = 0 and qhat = 0.
// ---------------------------------------------------------------------------------
void ora_quantise_query(const uint16_t* Q, int64_t n_vec, int d, int8_t* qhat, float* delta) {
    for (int64_t v = 0; v < n_vec; ++v) {
        const uint16_t* row = Q + v * d;
        float amax = 0.0f;
        for (int m = 0; m < d; ++m) {
            const float a = std::fabs(static_cast<float>(half_bits_to_double(row[m])));
            if (a > amax) amax = a;
        }
        if (amax == 0.0f) {
            delta[v] = 0.0f;
            for (int m = 0; m < d; ++m) qhat[v * d + m] = 0;
            continue;
        }
        const float inv = 127.0f / amax;
        delta[v] = amax / 127.0f;
        for (int m = 0; m < d; ++m) {
            const float x = static_cast<float>(half_bits_to_double(row[m]));
            float r = std::nearbyintf(x * inv);
            if (r > 127.0f) r = 127.0f;
            if (r < -127.0f) r = -127.0f;
            qhat[v * d + m] = static_cast<int8_t>(r);
        }
    }
}

// ---------------------------------------------------------------------------------
// Value quantisation, section II-E: V in INT8 with a power-of-two per-token scale
// 2^-g.  g is the largest integer with amax * 2^g <= 127; vhat = round-half-even
// (V * 2^g) (the scaling is exact).  amax = 0 gives g = 0, vhat = 0.
// ---------------------------------------------------------------------------------
void ora_quantise_value(const uint16_t* V, int64_t n_vec, int d, int8_t* vhat, int8_t* g_out) {
    for (int64_t v = 0; v < n_vec; ++v) {
        const uint16_t* row = V + v * d;
        double amax = 0.0;
        for (int m = 0; m < d; ++m) amax = std::fmax(amax, std::fabs(half_bits_to_double(row[m])));
        int g = 0;
        if (amax > 0.0) {
            g = 64;
            while (std::ldexp(amax, g) > 127.0) --g;
        }
        g_out[v] = static_cast<int8_t>(g);
        for (int m = 0; m < d; ++m)
            vhat[v * d + m] = static_cast<int8_t>(std::nearbyint(std::ldexp(half_bits_to_double(row[m]), g)));
    }
}

// ---------------------------------------------------------------------------------
// Integer scores, eq. (3) with the mantissa code of eq. (5) substituted:
//   A_ij = sum_m sigma_jm * qhat_im * (2^k + j_jm) * 2^(F - k - e_jm),
// the zero code contributing nothing.  With F >= E + k every factor 2^(F-k-e) is an
// integer (eq. (4): all shifts are left shifts), so the sum is an exact integer; it
// is formed in 64 bits.  Query head h reads KV head h / (Hq / Hkv).
// qhat [Hq, d]; codes [T, Hkv, d]; A [Hq, T].  Returns the number of scores that do
// not fit in INT32 (must be 0 for a valid F).
// ---------------------------------------------------------------------------------
int64_t ora_scores(const int8_t* qhat, const uint8_t* codes, int64_t T, int Hq, int Hkv, int d,
                   int k, int F, int64_t* A) {
    const int G = Hq / Hkv;
    int64_t overflow = 0;
    for (int h = 0; h < Hq; ++h) {
        const int kv = h / G;
        for (int64_t t = 0; t < T; ++t) {
            const uint8_t* c = codes + (t * Hkv + kv) * d;
            int64_t acc = 0;
            for (int m = 0; m < d; ++m) {
                const int e = (c[m] >> 4) & 7;
                if (e == kZeroExp) continue;
                const int j = (c[m] & 0xf) >> (4 - k);
                const int64_t mag = static_cast<int64_t>((1 << k) + j) << (F - k - e);
                const int64_t term = static_cast<int64_t>(qhat[h * d + m]) * mag;
                acc += (c[m] & 0x80) ? -term : term;
            }
            if (acc > INT32_MAX || acc < INT32_MIN) ++overflow;
            A[static_cast<int64_t>(h) * T + t] = acc;
        }
    }
    return overflow;
}

// ---------------------------------------------------------------------------------
// Two-pass softmax and floating-point A.V, eq. (1) with the dequantised score of
// eq. (3):  logit in the log2 domain  z_ij = A_ij * Delta_i * s_j * 2^-F * log2(e)
// / sqrt(d);  w_j = 2^(z_j - max z);  O_i = sum_j w_j * vhat_j * 2^-g_j / sum_j w_j.
// Everything in fp64.  T = 0 gives O = 0.
// A [Hq, T]; delta [Hq]; scales [T, Hkv] binary16 bits; vhat [T, Hkv, d]; g [T, Hkv];
// O [Hq, d].
// ---------------------------------------------------------------------------------
static void twopass_core(const int64_t* A, const float* delta, const uint16_t* scales,
                         const int8_t* vhat, const int8_t* g, int64_t T, int Hq, int Hkv,
                         int d, double unit, double* O) {
    const int G = Hq / Hkv;
    const double log2e = 1.4426950408889634074;
    std::vector<double> z(static_cast<size_t>(T));
    for (int h = 0; h < Hq; ++h) {
        const int kv = h / G;
        double* out = O + static_cast<int64_t>(h) * d;
        for (int m = 0; m < d; ++m) out[m] = 0.0;
        if (T == 0) continue;
        const double qf = static_cast<double>(delta[h]) * unit * log2e /
                          std::sqrt(static_cast<double>(d));
        double zmax = -std::numeric_limits<double>::infinity();
        for (int64_t t = 0; t < T; ++t) {
            z[t] = static_cast<double>(A[static_cast<int64_t>(h) * T + t]) * qf *
                   half_bits_to_double(scales[t * Hkv + kv]);
            zmax = std::fmax(zmax, z[t]);
        }
        double wsum = 0.0;
        for (int64_t t = 0; t < T; ++t) {
            const double w = std::exp2(z[t] - zmax);
            wsum += w;
            const double vs = std::ldexp(1.0, -g[t * Hkv + kv]);
            const int8_t* vr = vhat + (t * Hkv + kv) * d;
            for (int m = 0; m < d; ++m) out[m] += w * (static_cast<double>(vr[m]) * vs);
        }
        for (int m = 0; m < d; ++m) out[m] /= wsum;
    }
}

void ora_attention_twopass(const int64_t* A, const float* delta, const uint16_t* scales,
                           const int8_t* vhat, const int8_t* g, int64_t T, int Hq, int Hkv,
                           int d, int F, double* O) {
    twopass_core(A, delta, scales, vhat, g, T, Hq, Hkv, d, std::ldexp(1.0, -F), O);
}

// ---------------------------------------------------------------------------------
// Uniform INT8 key code: the comparison datapath of section III and section VI (an INT8
// multiply-accumulate kernel with the tiling of the shift kernel; Table II lists the uniform INT8
// quantiser as an accuracy baseline).  Per key vector: scale = largest magnitude (binary16),
// khat = clamp(round-half-even(K * 127 / amax), -127, 127), decided in binary32 exactly like
// the query quantiser; K ~ (scale / 127) * khat.  Scores are plain integer dot products
// A_ij = sum_m qhat_im * khat_jm; logits z = A * Delta * (scale / 127) * log2(e) / sqrt(d).
// ---------------------------------------------------------------------------------
void ora_encode_keys_int8(const uint16_t* K, int64_t n_vec, int d, int8_t* codes, uint16_t* scales) {
    for (int64_t v = 0; v < n_vec; ++v) {
        const uint16_t* row = K + v * d;
        uint16_t smax_bits = 0;
        for (int m = 0; m < d; ++m) {
            const uint16_t mag = row[m] & 0x7fff;
            if (mag > smax_bits) smax_bits = mag;
        }
        scales[v] = smax_bits;
        const float amax = static_cast<float>(half_bits_to_double(smax_bits));
        if (amax == 0.0f) {
            for (int m = 0; m < d; ++m) codes[v * d + m] = 0;
            continue;
        }
        const float inv = 127.0f / amax;
        for (int m = 0; m < d; ++m) {
            const float x = static_cast<float>(half_bits_to_double(row[m]));
            float r = std::nearbyintf(x * inv);
            if (r > 127.0f) r = 127.0f;
            if (r < -127.0f) r = -127.0f;
            codes[v * d + m] = static_cast<int8_t>(r);
        }
    }
}

void ora_scores_int8(const int8_t* qhat, const int8_t* codes, int64_t T, int Hq, int Hkv, int d, int64_t* A) {
    const int G = Hq / Hkv;
    for (int h = 0; h < Hq; ++h) {
        const int kv = h / G;
        for (int64_t t = 0; t < T; ++t) {
            const int8_t* c = codes + (t * Hkv + kv) * d;
            int64_t acc = 0;
            for (int m = 0; m < d; ++m) acc += static_cast<int64_t>(qhat[h * d + m]) * static_cast<int64_t>(c[m]);
            A[static_cast<int64_t>(h) * T + t] = acc;
        }
    }
}

void ora_attention_twopass_int8(const int64_t* A, const float* delta, const uint16_t* scales,
                                const int8_t* vhat, const int8_t* g, int64_t T, int Hq, int Hkv,
                                int d, double* O) {
    twopass_core(A, delta, scales, vhat, g, T, Hq, Hkv, d, 1.0 / 127.0, O);
}

// ---------------------------------------------------------------------------------
// Streaming softmax with an integer running maximum in the log2 domain, section
// II-E, plus the split over the key axis that the kernel grid has (section II-F).
// The keys are cut into `splits` contiguous ranges; each range is consumed in tiles
// of `tile` keys with state (M integer, l, O[d]):
//   M' = max(M, ceil(max over the tile of z));  p_j = 2^(z_j - M');
//   l  = l * 2^(M - M') + sum p;   O = O * 2^(M - M') + sum p_j * v_j.
// Every rescale factor is an exact power of two.  The ranges are merged with the
// same rule (M* = max M_s, factors 2^(M_s - M*)) and the result is O / l.
// The state is binary32, as in the kernel, to show that the streamed form agrees
// with the two-pass definition at that precision.  The weights are NOT quantised to
// powers of two here (the paper's default A.V path is floating point).
// ---------------------------------------------------------------------------------
void ora_attention_online(const int64_t* A, const float* delta, const uint16_t* scales,
                          const int8_t* vhat, const int8_t* g, int64_t T, int Hq, int Hkv,
                          int d, int F, int tile, int splits, float* O) {
    const int G = Hq / Hkv;
    const int kNone = INT32_MIN / 2;  // "no key seen yet"
    struct Part { int M; float l; std::vector<float> o; };
    for (int h = 0; h < Hq; ++h) {
        const int kv = h / G;
        const float qf = static_cast<float>(static_cast<double>(delta[h]) * std::ldexp(1.0, -F) *
                                            1.4426950408889634074 / std::sqrt(static_cast<double>(d)));
        std::vector<Part> parts;
        for (int s = 0; s < splits; ++s) {
            const int64_t t0 = T * s / splits, t1 = T * (s + 1) / splits;
            Part p{kNone, 0.0f, std::vector<float>(d, 0.0f)};
            for (int64_t tb = t0; tb < t1; tb += tile) {
                const int64_t te = (tb + tile < t1) ? tb + tile : t1;
                std::vector<float> z(static_cast<size_t>(te - tb));
                float zmax = -std::numeric_limits<float>::infinity();
                for (int64_t t = tb; t < te; ++t) {
                    z[t - tb] = static_cast<float>(A[static_cast<int64_t>(h) * T + t]) * qf *
                                static_cast<float>(half_bits_to_double(scales[t * Hkv + kv]));
                    zmax = std::fmax(zmax, z[t - tb]);
                }
                const int Mt = static_cast<int>(std::ceil(zmax));
                const int Mn = (Mt > p.M) ? Mt : p.M;
                const float resc = (p.M == kNone) ? 0.0f : std::ldexp(1.0f, p.M - Mn);
                p.l *= resc;
                for (int m = 0; m < d; ++m) p.o[m] *= resc;
                for (int64_t t = tb; t < te; ++t) {
                    const float w = std::exp2(z[t - tb] - static_cast<float>(Mn));
                    p.l += w;
                    const float vs = std::ldexp(1.0f, -g[t * Hkv + kv]);
                    const int8_t* vr = vhat + (t * Hkv + kv) * d;
                    for (int m = 0; m < d; ++m) p.o[m] += w * (static_cast<float>(vr[m]) * vs);
                }
                p.M = Mn;
            }
            parts.push_back(p);
        }
        int Ms = kNone;
        for (const Part& p : parts) if (p.M > Ms) Ms = p.M;
        float l = 0.0f;
        std::vector<float> o(d, 0.0f);
        for (const Part& p : parts) {
            if (p.M == kNone) continue;
            const float f = std::ldexp(1.0f, p.M - Ms);
            l += p.l * f;
            for (int m = 0; m < d; ++m) o[m] += p.o[m] * f;
        }
        for (int m = 0; m < d; ++m) O[static_cast<int64_t>(h) * d + m] = (l > 0.0f) ? o[m] / l : 0.0f;
    }
}

// ---------------------------------------------------------------------------------
// Log2-quantised attention weights and the shift-based A.V: section II-E, eq. (6) and
// eq. (7) — the paper's non-default option, in which the second product needs no multiplier either.
//
//   M      = ceil(max_j z_j)                      (integer, log2 domain, z = logit * log2 e)
//   k_j    = round(M - z_j) >= 0,  weight 2^-k_j                                   eq. (6)
//   g_ref  = min_j g_j                            (value scales 2^-g_j, INT8 values vhat_j)
//   O      = 2^(-N - g_ref) * sum_{j : k_j <= k_max} vhat_j << (N - k_j + g_ref - g_j)   eq. (7)
//            divided by the sum of the kept weights, sum_{j : k_j <= k_max} 2^-k_j.
//
// Readings (the paper gives neither N nor k_max, and writes eq. (7) without the
// normaliser and without saying what a negative shift index means):
//   * k_j is evaluated as M - round(z_j): for an integer M and round-half-to-even this is
//     the same number, and it makes the decision independent of M.  The rounding is an
//     integer decision taken on a floating-point logit, so the logit is formed in binary32
//     in one fixed order:  z_j = (float(A_j) (x) (Delta (x) c)) (x) s_j  with
//     c = binary32(log2(e) / sqrt(d) / 2^F) and (x) the binary32 product; it is clamped to
//     +-1e8 before ceil / round (as for the running maximum of the default path).
//   * M and g_ref are those of the whole key range (the definition; a streaming kernel's
//     running values converge to them).
//   * a key with k_j > k_max is dropped from numerator and normaliser alike (its weight is
//     below 2^-k_max); a key whose shift index N - k_j + g_ref - g_j is negative is dropped
//     from the numerator only (its value is below one unit 2^(-N - g_ref) of the accumulator).
//   * N and k_max are inputs; 0 <= k_max <= N.
// Everything after the rounding is exact integer arithmetic here (int64 numerator in units
// of 2^(-N - g_ref), int64 normaliser in units of 2^-N); the final division is fp64.
// Parity: the arithmetic is pinned (rational sums, softmax of the rounded logits, hand
// cases for both drop rules); the VALUES of N and k_max are not the paper's — "parity
// unpinned" for those two constants.
// A [Hq, T]; delta [Hq]; scales [T, Hkv] binary16 bits; vhat [T, Hkv, d]; g [T, Hkv];
// O [Hq, d]; zr_out (optional) [Hq, T] rounded logits; M_out (optional) [Hq].
// ---------------------------------------------------------------------------------
void ora_attention_shiftav(const int64_t* A, const float* delta, const uint16_t* scales,
                           const int8_t* vhat, const int8_t* g, int64_t T, int Hq, int Hkv,
                           int d, int F, int N, int k_max, double* O, int32_t* zr_out,
                           int32_t* M_out) {
    const int G = Hq / Hkv;
    const float c = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(d)) /
                                       static_cast<double>(1LL << F));
    std::vector<int32_t> zr(static_cast<size_t>(T));
    std::vector<int64_t> num(static_cast<size_t>(d));
    for (int h = 0; h < Hq; ++h) {
        const int kv = h / G;
        double* out = O + static_cast<int64_t>(h) * d;
        for (int m = 0; m < d; ++m) out[m] = 0.0;
        if (M_out) M_out[h] = 0;
        if (T == 0) continue;
        const float qscale = delta[h] * c;                       // binary32 product
        int32_t M = INT32_MIN;
        int g_ref = INT32_MAX;
        for (int64_t t = 0; t < T; ++t) {
            const float s_j = static_cast<float>(half_bits_to_double(scales[t * Hkv + kv]));
            float z = static_cast<float>(A[static_cast<int64_t>(h) * T + t]);   // int -> binary32, nearest-even
            z = z * qscale;
            z = z * s_j;
            z = std::fmin(std::fmax(z, -1.0e8f), 1.0e8f);
            const int32_t up = static_cast<int32_t>(std::ceil(z));
            zr[t] = static_cast<int32_t>(std::nearbyintf(z));    // round half to even
            if (up > M) M = up;
            const int gj = g[t * Hkv + kv];
            if (gj < g_ref) g_ref = gj;
            if (zr_out) zr_out[static_cast<int64_t>(h) * T + t] = zr[t];
        }
        if (M_out) M_out[h] = M;
        int64_t norm = 0;                                        // units of 2^-N
        for (int m = 0; m < d; ++m) num[m] = 0;                  // units of 2^(-N - g_ref)
        for (int64_t t = 0; t < T; ++t) {
            const int64_t k = static_cast<int64_t>(M) - zr[t];  // >= 0 because ceil >= round
            if (k > k_max) continue;
            norm += int64_t{1} << (N - k);
            const int64_t sh = N - k + g_ref - g[t * Hkv + kv];
            if (sh < 0) continue;
            const int8_t* vr = vhat + (t * Hkv + kv) * d;
            for (int m = 0; m < d; ++m) num[m] += static_cast<int64_t>(vr[m]) * (int64_t{1} << sh);
        }
        if (norm == 0) continue;
        for (int m = 0; m < d; ++m)
            out[m] = std::ldexp(static_cast<double>(num[m]), -g_ref) / static_cast<double>(norm);
    }
}

// ---------------------------------------------------------------------------------
// Textbook scaled dot-product attention, eq. (1), on the unquantised binary16
// inputs, in fp64.  Reference for the FP16 decode kernel.
// Q [Hq, d]; K, V [T, Hkv, d]; O [Hq, d].
// ---------------------------------------------------------------------------------
void ora_sdpa_fp16(const uint16_t* Q, const uint16_t* K, const uint16_t* V, int64_t T, int Hq,
                   int Hkv, int d, double* O) {
    const int G = Hq / Hkv;
    std::vector<double> s(static_cast<size_t>(T));
    for (int h = 0; h < Hq; ++h) {
        const int kv = h / G;
        double* out = O + static_cast<int64_t>(h) * d;
        for (int m = 0; m < d; ++m) out[m] = 0.0;
        if (T == 0) continue;
        double smax = -std::numeric_limits<double>::infinity();
        for (int64_t t = 0; t < T; ++t) {
            double acc = 0.0;
            for (int m = 0; m < d; ++m)
                acc += half_bits_to_double(Q[h * d + m]) * half_bits_to_double(K[(t * Hkv + kv) * d + m]);
            s[t] = acc / std::sqrt(static_cast<double>(d));
            smax = std::fmax(smax, s[t]);
        }
        double wsum = 0.0;
        for (int64_t t = 0; t < T; ++t) {
            const double w = std::exp(s[t] - smax);
            wsum += w;
            for (int m = 0; m < d; ++m) out[m] += w * half_bits_to_double(V[(t * Hkv + kv) * d + m]);
        }
        for (int m = 0; m < d; ++m) out[m] /= wsum;
    }
}

// ---------------------------------------------------------------------------------
// The whole decode step for a ragged batch, chaining the functions above in the
// paper's order: [optional rotation of Q and K] -> query quantise -> key encode ->
// value quantise -> integer scores -> two-pass softmax and A.V.  k = 8 selects the uniform INT8
// comparison code (F is then ignored).
// Q [B, Hq, d]; K, V [sum_b T_b, Hkv, d] with sequence b occupying rows
// cu_lens[b] .. cu_lens[b+1]; O [B, Hq, d] fp64; A_dbg (nullable) [B, Hq, max_T]
// receives the integer scores (row stride max_T).  The independent units
// (sequence, KV head) are dealt round-robin to n_threads host threads; each unit
// copies its KV head's rows out of the interleaved layout and then runs the plain
// single-head-group functions above.  There is no other parallelism.
// stage_seconds (nullable, 4 doubles): per-thread time summed over threads for
// {rotation + query quantise, key encode + value quantise, scores, softmax + A.V}.
// Returns the number of integer scores that did not fit INT32 (0 for a valid F).
// ---------------------------------------------------------------------------------
int64_t ora_decode_attention(const uint16_t* Q, const uint16_t* K, const uint16_t* V,
                             const int64_t* cu_lens, int B, int Hq, int Hkv, int d, int k, int F,
                             int hadamard, double* O, int64_t* A_dbg, int64_t max_T,
                             int n_threads, double* stage_seconds) {
    if (n_threads < 1) n_threads = 1;
    const int G = Hq / Hkv;
    std::vector<int64_t> overflow(n_threads, 0);
    std::vector<double> st(static_cast<size_t>(n_threads) * 4, 0.0);
    auto now = [] {
        timespec ts;
        clock_gettime(CLOCK_MONOTONIC, &ts);
        return ts.tv_sec + 1e-9 * ts.tv_nsec;
    };
    auto work = [&](int tid) {
        for (int u = tid; u < B * Hkv; u += n_threads) {
            const int b = u / Hkv, kv = u % Hkv;
            const int64_t t0 = cu_lens[b], T = cu_lens[b + 1] - cu_lens[b];
            double c0 = now();
            // the G query heads of this KV head, and this KV head's rows of K and V
            const uint16_t* qsrc = Q + (static_cast<int64_t>(b) * Hq + kv * G) * d;
            std::vector<uint16_t> q(qsrc, qsrc + static_cast<int64_t>(G) * d);
            std::vector<uint16_t> kk(static_cast<size_t>(T) * d), vv(static_cast<size_t>(T) * d);
            for (int64_t t = 0; t < T; ++t) {
                std::memcpy(&kk[t * d], K + ((t0 + t) * Hkv + kv) * d, sizeof(uint16_t) * d);
                std::memcpy(&vv[t * d], V + ((t0 + t) * Hkv + kv) * d, sizeof(uint16_t) * d);
            }
            if (hadamard) {
                ora_hadamard_fp16(q.data(), G, d);
                ora_hadamard_fp16(kk.data(), T, d);
            }
            std::vector<int8_t> qhat(static_cast<size_t>(G) * d);
            std::vector<float> delta(G);
            ora_quantise_query(q.data(), G, d, qhat.data(), delta.data());
            double c1 = now();
            std::vector<uint8_t> codes(static_cast<size_t>(T) * d);
            std::vector<uint16_t> scales(static_cast<size_t>(T));
            if (k == 8) ora_encode_keys_int8(kk.data(), T, d, reinterpret_cast<int8_t*>(codes.data()), scales.data());
            else ora_encode_keys(kk.data(), T, d, k, codes.data(), scales.data());
            std::vector<int8_t> vhat(static_cast<size_t>(T) * d), g(static_cast<size_t>(T));
            ora_quantise_value(vv.data(), T, d, vhat.data(), g.data());
            double c2 = now();
            std::vector<int64_t> A(static_cast<size_t>(G) * T);
            if (k == 8) ora_scores_int8(qhat.data(), reinterpret_cast<const int8_t*>(codes.data()), T, G, 1, d, A.data());
            else overflow[tid] += ora_scores(qhat.data(), codes.data(), T, G, 1, d, k, F, A.data());
            double c3 = now();
            double* Oh = O + (static_cast<int64_t>(b) * Hq + kv * G) * d;
            if (k == 8) ora_attention_twopass_int8(A.data(), delta.data(), scales.data(), vhat.data(), g.data(), T, G, 1, d, Oh);
            else ora_attention_twopass(A.data(), delta.data(), scales.data(), vhat.data(), g.data(), T, G, 1, d, F, Oh);
            double c4 = now();
            if (A_dbg)
                for (int h = 0; h < G; ++h)
                    for (int64_t t = 0; t < T; ++t)
                        A_dbg[(static_cast<int64_t>(b) * Hq + kv * G + h) * max_T + t] =
                            A[static_cast<int64_t>(h) * T + t];
            st[tid * 4 + 0] += c1 - c0;
            st[tid * 4 + 1] += c2 - c1;
            st[tid * 4 + 2] += c3 - c2;
            st[tid * 4 + 3] += c4 - c3;
        }
    };
    if (n_threads == 1) {
        work(0);
    } else {
        std::vector<std::thread> th;
        for (int i = 0; i < n_threads; ++i) th.emplace_back(work, i);
        for (auto& t : th) t.join();
    }
    int64_t ov = 0;
    for (int i = 0; i < n_threads; ++i) ov += overflow[i];
    if (stage_seconds)
        for (int s = 0; s < 4; ++s) {
            stage_seconds[s] = 0.0;
            for (int i = 0; i < n_threads; ++i) stage_seconds[s] += st[i * 4 + s];
        }
    return ov;
}

int ora_hardware_threads() { return static_cast<int>(std::thread::hardware_concurrency()); }

}  // extern "C"
