// Host-side harness for the unit tests: exposes the library's exact-arithmetic device functions
// (which are also compiled for the host) through a C interface, so that they can be checked
// against the CPU oracle without a GPU.  Built by tests/test_host_arith.py; not part of the library.
#include "../paper_2609_09208_b200/csrc/sa_datapath.cuh"

using namespace sa;

template <int K>
static int32_t score_one(const uint8_t* codes, const int8_t* q, int d, int f_extra, bool nibble_path) {
    Planes<K, 1> pl;
    pl.clear();
    for (int m0 = 0; m0 < d; m0 += 4) {
        uint32_t w = 0;
        for (int i = 0; i < 4; ++i) w |= (uint32_t)codes[m0 + i] << (8 * i);
        if (!nibble_path) pl.corrections_bytes(w);
        for (int i = 0; i < 4; ++i) {
            const int32_t qq[1] = {q[m0 + i]};
            pl.element((w >> (8 * i)) & 0xffu, qq);
        }
    }
    if (nibble_path) {  // eight sign/exponent nibbles per word
        for (int m0 = 0; m0 < d; m0 += 8) {
            uint32_t w = 0;
            for (int i = 0; i < 8; ++i) w |= (uint32_t)(codes[m0 + i] >> 4) << (4 * i);
            pl.corrections_nibbles(w);
        }
    }
    return pl.score(0, f_extra);
}

extern "C" {
int hh_encode_element(int k, unsigned a_bits, unsigned s_bits) {
    switch (k) {
        case 0: return encode_element<0>(a_bits, s_bits);
        case 1: return encode_element<1>(a_bits, s_bits);
        case 2: return encode_element<2>(a_bits, s_bits);
        default: return encode_element<4>(a_bits, s_bits);
    }
}
void hh_encode_many(int k, const uint16_t* a_bits, int64_t n, unsigned s_bits, uint8_t* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = (uint8_t)hh_encode_element(k, a_bits[i], s_bits);
}
int hh_value_exponent(unsigned amax_bits) { return value_exponent(amax_bits); }
int32_t hh_score(int k, const uint8_t* codes, const int8_t* q, int d, int f_extra, int nibble_path) {
    switch (k) {
        case 0: return score_one<0>(codes, q, d, f_extra, nibble_path != 0);
        case 1: return score_one<1>(codes, q, d, f_extra, false);
        case 2: return score_one<2>(codes, q, d, f_extra, false);
        default: return score_one<4>(codes, q, d, f_extra, false);
    }
}
}
