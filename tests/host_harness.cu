// Host-side harness for the unit tests: exposes the library's exact-arithmetic device functions
// (which are also compiled for the host) through a C interface, so that they can be checked
// against the CPU oracle without a GPU.  Built by tests/test_host_arith.py; not part of the library.
#include "../paper_2609_09208_b200/csrc/sa_datapath.cuh"

using namespace sa;

// Scores of one PoT-4 key (canonical code bytes) against 8 queries, through the same packed
// datapath and word decoders the decode kernel uses (byte container: phys_byte; nibbles: canonical nibble ^ 7).
template <bool ALU>
static void score8_packed(const uint8_t* canon, const int8_t* q8, int d, bool nibble_path, int32_t* out) {
    using ST = ShiftTable<4>;
    alignas(256) static uint8_t tab[128 * ST::kRowBytes];          // S[m][g][pair]: the shifted packed pairs
    for (int m = 0; m < d; ++m)
        for (int g = 0; g < 8; ++g)
            for (int p = 0; p < 4; ++p)
                reinterpret_cast<uint32_t*>(tab)[(m * 8 + g) * 4 + p] =
                    ST::entry(pack_pair(q8[(2 * p) * d + m], q8[(2 * p + 1) * d + m]), g);
    PackedShift<4, ALU> pl;
    pl.begin(1u);
    if (!nibble_path) {
        for (int m0 = 0; m0 < d; m0 += 16) {
            uint32_t w[4] = {0, 0, 0, 0};
            for (int i = 0; i < 16; ++i) w[i / 4] |= (uint32_t)phys_byte(canon[m0 + i]) << (8 * (i % 4));
            const uint8_t* grp = tab + m0 * ST::kRowBytes;
            accumulate_word_bytes_tab<4, 0>(pl, w[0], grp);
            accumulate_word_bytes_tab<4, 1>(pl, w[1], grp);
            accumulate_word_bytes_tab<4, 2>(pl, w[2], grp);
            accumulate_word_bytes_tab<4, 3>(pl, w[3], grp);
        }
    } else {
        for (int m0 = 0; m0 < d; m0 += 8) {
            uint32_t w = 0;
            for (int i = 0; i < 8; ++i) w |= (uint32_t)((canon[m0 + i] ^ 0x70) >> 4) << (4 * i);
            accumulate_word_nibbles_tab<4>(pl, w, (const uint8_t*)(tab + m0 * ST::kRowBytes));
        }
    }
    for (int g = 0; g < 8; ++g) out[g] = pl.score(g);
}

// The scores of a mantissa code (k = 1, 2, 4) through the table datapath.
// The same scores through the table datapath of the mantissa codes.
// VAR 0: the default datapath; 1: the shifts as multiplications by 2^r; 2: sign flips and adds on the ALU pipe only
template <int K, int VAR>
static void score8_table(const uint8_t* canon, const int8_t* q8, int d, int32_t* out) {
    using TS = TableScore<K, 4, VAR == 1, VAR == 2>;
    alignas(256) static uint8_t tab[128 * TS::kElemBytes];
    for (int m = 0; m < d; ++m)
        for (int gp = 0; gp < 4; ++gp)
            fill_table_row<K>(tab + m * TS::kElemBytes + gp * TS::kRowBytes, q8[(2 * gp) * d + m], q8[(2 * gp + 1) * d + m]);
    TS ts;
    ts.begin(1u);
    for (int m0 = 0; m0 < d; m0 += 16) {
        uint32_t w[4] = {0, 0, 0, 0};
        for (int i = 0; i < 16; ++i) w[i / 4] |= (uint32_t)phys_byte(canon[m0 + i]) << (8 * (i % 4));
        const uint8_t* grp = tab + m0 * TS::kElemBytes;
        ts.template accumulate_word<0>(w[0], grp);
        ts.template accumulate_word<1>(w[1], grp);
        ts.template accumulate_word<2>(w[2], grp);
        ts.template accumulate_word<3>(w[3], grp);
    }
    for (int g = 0; g < 8; ++g) out[g] = ts.score(g);
}

// The same through the dense planar container (k = 1, 2): sign/exponent nibbles, two per byte, and the
// mantissa bits in k separate bit planes.
template <int K, int VAR>
static void score8_planar(const uint8_t* canon, const int8_t* q8, int d, int32_t* out) {
    using TS = TableScore<K, 4, VAR == 1, VAR == 2>;
    alignas(256) static uint8_t tab[128 * TS::kElemBytes];
    for (int m = 0; m < d; ++m)
        for (int gp = 0; gp < 4; ++gp)
            fill_table_row<K>(tab + m * TS::kElemBytes + gp * TS::kRowBytes, q8[(2 * gp) * d + m], q8[(2 * gp + 1) * d + m]);
    TS ts;
    ts.begin(1u);
    for (int m0 = 0; m0 < d; m0 += 16) {
        const uint8_t* grp = tab + m0 * TS::kElemBytes;
        for (int half = 0; half < 2; ++half) {
            uint32_t w = 0, planes[K];
            for (int b = 0; b < K; ++b) planes[b] = 0;
            for (int i = 0; i < 8; ++i) {
                const uint8_t phys = canon[m0 + 8 * half + i] ^ 0x70;
                w |= (uint32_t)(phys >> 4) << (4 * i);
                for (int b = 0; b < K; ++b) planes[b] |= (uint32_t)((phys >> (4 - K + b)) & 1u) << i;
            }
            if (half == 0) ts.template accumulate_nibble_word<0>(w, planes, grp);
            else ts.template accumulate_nibble_word<1>(w, planes, grp);
        }
    }
    for (int g = 0; g < 8; ++g) out[g] = ts.score(g);
}

template <int VAR>
static void score8_any(int k, const uint8_t* canon, const int8_t* q8, int d, int path, int32_t* out) {
    // path 0: byte container (packed datapath for k = 0, table datapath otherwise); 1: nibble container
    // (k = 0) or dense planar container (k = 1, 2)
    if (k == 0) score8_packed<VAR == 2>(canon, q8, d, path != 0, out);  // PoT-4 has no multiply variant
    else if (path != 0 && k == 1) score8_planar<1, VAR>(canon, q8, d, out);
    else if (path != 0 && k == 2) score8_planar<2, VAR>(canon, q8, d, out);
    else if (k == 1) score8_table<1, VAR>(canon, q8, d, out);
    else if (k == 2) score8_table<2, VAR>(canon, q8, d, out);
    else score8_table<4, VAR>(canon, q8, d, out);
}

extern "C" {
void hh_score8_planar(int k, const uint8_t* canon, const int8_t* q8, int d, int32_t* out) { score8_any<0>(k, canon, q8, d, 1, out); }
void hh_score8_table(int k, const uint8_t* canon, const int8_t* q8, int d, int32_t* out) { score8_any<0>(k, canon, q8, d, 0, out); }
// the same datapaths with the shifts executed as multiplications by 2^r
void hh_score8_mul(int k, const uint8_t* canon, const int8_t* q8, int d, int path, int32_t* out) { score8_any<1>(k, canon, q8, d, path, out); }
// ... and with every sign flip and add on the ALU pipe (exclusive-or, subtract, add)
void hh_score8_alu(int k, const uint8_t* canon, const int8_t* q8, int d, int path, int32_t* out) { score8_any<2>(k, canon, q8, d, path, out); }
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
void hh_score8(int k, const uint8_t* canon, const int8_t* q8, int d, int nibble_path, int32_t* out) {
    score8_any<0>(k, canon, q8, d, k == 0 ? nibble_path : 0, out);
}
}
