// The integer score datapath of the decode kernel, kept free of anything that only compiles for
// the device so that its arithmetic can also be exercised on the host by the unit tests.
#pragma once
#include "sa_common.cuh"

namespace sa {

// Left shift that returns 0 for amounts >= 32 (PTX shl.b32 semantics).
SA_HD uint32_t shl_clamp_hd(uint32_t x, uint32_t n) {
#ifdef __CUDA_ARCH__
    return shl_clamp(x, n);
#else
    return n >= 32u ? 0u : (x << n);
#endif
}
SA_HD int popc_hd(uint32_t x) {
#ifdef __CUDA_ARCH__
    return __popc(x);
#else
    return __builtin_popcount(x);
#endif
}

// -------------------------------------------------------------------------------------------
// Integer scores of one key against GT queries: shift / sign-flip / add only.
//
// With F0 = 6 + KB the term of element m is  sigma * (qhat << r) * (2^KB + j),  r = 6 - e >= 0.
// It is accumulated in KB + 1 "planes": plane KB takes sigma*(qhat << r) of every element, plane
// b < KB only of the elements whose mantissa bit b is set; the score is
// sum_b plane_b << b.  The sign flip is a bitwise complement (x ^ S, S = 0 or -1) and the
// missing "+1" of the two's complement is added per key from population counts of the sign
// bits, which all GT queries share.  The zero code gives r = 0xffffffff, for which the shift
// returns 0.
// -------------------------------------------------------------------------------------------
template <int KB, int GT>
struct Planes {
    int32_t acc[KB + 1][GT];
    int32_t corr[KB + 1];
    SA_HD void clear() {
#pragma unroll
        for (int b = 0; b <= KB; ++b) {
            corr[b] = 0;
#pragma unroll
            for (int g = 0; g < GT; ++g) acc[b][g] = 0;
        }
    }
    // one element: canonical code byte `cb` (only bits 7..(4-KB) are looked at), queries q[g]
    SA_HD void element(uint32_t cb, const int32_t (&q)[GT]) {
        const uint32_t r = 6u - ((cb >> 4) & 7u);
        const int32_t S = -(int32_t)((cb >> 7) & 1u);
        int32_t mask[KB > 0 ? KB : 1];
#pragma unroll
        for (int b = 0; b < KB; ++b) mask[b] = -(int32_t)((cb >> (4 - KB + b)) & 1u);
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            const int32_t xs = (int32_t)shl_clamp_hd((uint32_t)q[g], r) ^ S;
            acc[KB][g] += xs;
#pragma unroll
            for (int b = 0; b < KB; ++b) acc[b][g] += xs & mask[b];
        }
    }
    // four canonical bytes in one word: the +1 corrections of the complemented terms
    SA_HD void corrections_bytes(uint32_t w) {
        const uint32_t neg = w & 0x80808080u;
        corr[KB] += popc_hd(neg);
#pragma unroll
        for (int b = 0; b < KB; ++b) corr[b] += popc_hd(neg & (w << (3 + KB - b)));
    }
    // eight nibbles (sign << 3 | e) in one word (PoT-4 only)
    SA_HD void corrections_nibbles(uint32_t w) { corr[KB] += popc_hd(w & 0x88888888u); }
    SA_HD int32_t score(int g, int f_extra) const {
        // unsigned arithmetic: the shifts are exact modulo 2^32 and the true sum fits in INT32
        uint32_t a = (uint32_t)(acc[KB][g] + corr[KB]) << KB;
#pragma unroll
        for (int b = 0; b < KB; ++b) a += (uint32_t)(acc[b][g] + corr[b]) << b;
        return (int32_t)(a << f_extra);
    }
};

}  // namespace sa
