// Warp-level quantisers shared by the cache-write kernels and the decode kernel's prologue.
// A head vector of D = 32 * EPL elements is spread over a warp, lane l holding elements
// l * EPL .. l * EPL + EPL - 1.
#pragma once
#include "sa_common.cuh"

namespace sa {

template <int EPL>
SA_D void load_vec_bits(const uint16_t* row, int lane, uint32_t (&bits)[EPL]) {
    if constexpr (EPL == 2) {
        const uint32_t w = *reinterpret_cast<const uint32_t*>(row + lane * 2);
        bits[0] = w & 0xffffu;
        bits[1] = w >> 16;
    } else {
        static_assert(EPL == 4, "head_dim must be 64 or 128");
        const uint2 w = *reinterpret_cast<const uint2*>(row + lane * 4);
        bits[0] = w.x & 0xffffu;
        bits[1] = w.x >> 16;
        bits[2] = w.y & 0xffffu;
        bits[3] = w.y >> 16;
    }
}

template <int N>
SA_D void store_bytes(uint8_t* dst, const uint8_t (&c)[N]) {
    if constexpr (N == 1) {
        dst[0] = c[0];
    } else if constexpr (N == 2) {
        *reinterpret_cast<uint16_t*>(dst) = (uint16_t)(c[0] | (c[1] << 8));
    } else {
        static_assert(N == 4, "1, 2 or 4 bytes");
        *reinterpret_cast<uint32_t*>(dst) = (uint32_t)c[0] | ((uint32_t)c[1] << 8) | ((uint32_t)c[2] << 16) | ((uint32_t)c[3] << 24);
    }
}

// Key vector -> canonical code bytes; returns the scale's binary16 bits (the largest magnitude).
// Section II-A: per-key-vector scale; section II-D: nearest-in-log2 codeword.
template <int EPL, int K>
SA_D uint32_t encode_key_vec(uint32_t (&bits)[EPL], int lane, bool hadamard, uint8_t (&codes)[EPL]) {
    if (hadamard) {
        float x[EPL];
#pragma unroll
        for (int i = 0; i < EPL; ++i) x[i] = half_bits_to_float(bits[i]);
        hadamard_warp<EPL>(x, bits, lane);
    }
    uint32_t smax = 0;
#pragma unroll
    for (int i = 0; i < EPL; ++i) smax = max(smax, bits[i] & 0x7fffu);   // binary16 magnitudes order like their bits
    smax = warp_max_u32(smax);
#pragma unroll
    for (int i = 0; i < EPL; ++i) codes[i] = encode_element<K>(bits[i], smax);
    return smax;
}

// Key vector -> uniform INT8 codes (the comparison code of section III / VI); returns the scale's
// binary16 bits (the largest magnitude).  Same rounding rule as the query quantiser.
template <int EPL>
SA_D uint32_t encode_key_int8_vec(uint32_t (&bits)[EPL], int lane, bool hadamard, uint8_t (&codes)[EPL]) {
    float x[EPL];
#pragma unroll
    for (int i = 0; i < EPL; ++i) x[i] = half_bits_to_float(bits[i]);
    if (hadamard) {
        hadamard_warp<EPL>(x, bits, lane);
#pragma unroll
        for (int i = 0; i < EPL; ++i) x[i] = half_bits_to_float(bits[i]);
    }
    uint32_t smax = 0;
#pragma unroll
    for (int i = 0; i < EPL; ++i) smax = max(smax, bits[i] & 0x7fffu);
    smax = warp_max_u32(smax);
    const float amax = half_bits_to_float(smax);
    const float inv = (amax == 0.0f) ? 0.0f : __fdiv_rn(127.0f, amax);
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
        const int r = __float2int_rn(__fmul_rn(x[i], inv));
        codes[i] = (uint8_t)(int8_t)max(-127, min(127, r));
    }
    return smax;
}

// Query vector -> integers in [-127, 127]; returns the step Delta = amax / 127 (eq. (2)).
// The rounding decision is taken in FP32 with IEEE divide and multiply, no contraction.
template <int EPL>
SA_D float quantise_query_vec(uint32_t (&bits)[EPL], int lane, bool hadamard, int (&q)[EPL]) {
    float x[EPL];
#pragma unroll
    for (int i = 0; i < EPL; ++i) x[i] = half_bits_to_float(bits[i]);
    if (hadamard) {
        hadamard_warp<EPL>(x, bits, lane);
#pragma unroll
        for (int i = 0; i < EPL; ++i) x[i] = half_bits_to_float(bits[i]);
    }
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < EPL; ++i) amax = fmaxf(amax, fabsf(x[i]));
    amax = warp_max_f32(amax);
    if (amax == 0.0f) {
#pragma unroll
        for (int i = 0; i < EPL; ++i) q[i] = 0;
        return 0.0f;
    }
    const float inv = __fdiv_rn(127.0f, amax);
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
        int r = __float2int_rn(__fmul_rn(x[i], inv));
        q[i] = max(-127, min(127, r));
    }
    return __fdiv_rn(amax, 127.0f);
}

// Value vector -> INT8 bytes and the power-of-two exponent g (section II-E).
template <int EPL>
SA_D int quantise_value_vec(const uint32_t (&bits)[EPL], uint8_t (&v)[EPL]) {
    uint32_t amax = 0;
#pragma unroll
    for (int i = 0; i < EPL; ++i) amax = max(amax, bits[i] & 0x7fffu);
    amax = warp_max_u32(amax);
    const int g = value_exponent(amax);   // in [-10, 30]
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
        // scaling by 2^g is exact in FP32 for every binary16 input and every g that can occur
        const float s = __fmul_rn(half_bits_to_float(bits[i]), pow2i(g));
        v[i] = (uint8_t)(int8_t)__float2int_rn(s);
    }
    return g;
}

}  // namespace sa
