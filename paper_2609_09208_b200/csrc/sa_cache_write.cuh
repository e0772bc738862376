// Writing one token of one KV head into its page block (the cache write of section II-F): used by the
// append / fill kernels and by the decode kernel when it appends the step's new token itself.
#pragma once
#include "sa_common.cuh"
#include "sa_quant.cuh"

namespace sa {

// -------------------------------------------------------------------------------------------
// Writing one token of one KV head into its page block.
// -------------------------------------------------------------------------------------------
struct CacheArgs {
    uint8_t* pages;
    const int32_t* page_table;
    int32_t* seq_lens;
    int batch, max_pages, n_pages, Hkv;
    size_t page_bytes, kcode_off, meta_off, v_off, plane_off;
    int hadamard;
};

template <int D, int K, bool NIB>
SA_D void write_token_quant(uint8_t* block, const CacheArgs& a, int t, int lane, const uint16_t* krow,
                            const uint16_t* vrow) {
    constexpr int EPL = D / 32;
    uint32_t kb[EPL], vb[EPL];
    load_vec_bits<EPL>(krow, lane, kb);
    load_vec_bits<EPL>(vrow, lane, vb);
    uint8_t kc[EPL], vc[EPL];
    uint32_t smax;
    if constexpr (K == 8) {
        smax = encode_key_int8_vec<EPL>(kb, lane, a.hadamard != 0, kc);      // uniform INT8: stored as is
    } else {
        smax = encode_key_vec<EPL, K>(kb, lane, a.hadamard != 0, kc);
        // byte container: the physical byte (phys_byte); the sub-byte containers below work on the canonical
        // byte with its exponent field replaced by g = 7 - e (0 for the zero code), i.e. canonical ^ 0x70
#pragma unroll
        for (int i = 0; i < EPL; ++i) kc[i] = NIB ? (uint8_t)(kc[i] ^ 0x70) : phys_byte(kc[i]);
    }
    const int gg = quantise_value_vec<EPL>(vb, vc);
    block += (size_t)(t >> 5) * (a.page_bytes >> 1);          // the token's half of the page; offsets are within a half
    t &= 31;
    uint8_t* kdst = block + a.kcode_off;
    if (!NIB) {
        const int m = lane * EPL;                   // first element of this lane
        store_bytes<EPL>(kdst + ((size_t)(m >> 4) * kTileTokens + t) * 16 + (m & 15), kc);
    } else {
        // two elements per byte: low nibble = even element, high nibble = odd element
        uint8_t nb[EPL / 2];
#pragma unroll
        for (int i = 0; i < EPL / 2; ++i) nb[i] = (uint8_t)((kc[2 * i] >> 4) | (kc[2 * i + 1] & 0xf0));
        const int m = lane * EPL;
        store_bytes<EPL / 2>(kdst + ((size_t)(m >> 5) * kTileTokens + t) * 16 + ((m & 31) >> 1), nb);
        if constexpr (K > 0 && K < 8) {
            // dense planar container: mantissa bit b of element m goes to bit m % 8 of byte m / 8 of plane b.
            // A lane holds EPL consecutive elements, so 8 / EPL lanes share a byte; lane B assembles byte B.
            constexpr int LPB = 8 / EPL;                      // lanes per plane byte
#pragma unroll
            for (int bit = 0; bit < K; ++bit) {
                uint32_t mask[EPL];
#pragma unroll
                for (int i = 0; i < EPL; ++i) mask[i] = __ballot_sync(0xffffffffu, (kc[i] >> (4 - K + bit)) & 1u);
                if (lane < D / 8) {
                    uint32_t byte = 0;
#pragma unroll
                    for (int l = 0; l < LPB; ++l)
#pragma unroll
                        for (int i = 0; i < EPL; ++i) byte |= ((mask[i] >> (LPB * lane + l)) & 1u) << (EPL * l + i);
                    block[a.plane_off + ((size_t)bit * kTileTokens + t) * (D / 8) + lane] = (uint8_t)byte;
                }
            }
        }
    }
    {
        const int mv = lane * EPL;                  // values: 16-dim chunks, chunk c of token t at (c * 32 + t) * 16 within the half
        store_bytes<EPL>(block + a.v_off + ((size_t)(mv >> 4) * kTileTokens + t) * 16 + (mv & 15), vc);
    }
    if (lane == 0)
        *reinterpret_cast<uint32_t*>(block + a.meta_off + (size_t)t * 4) = (smax & 0xffffu) | ((uint32_t)(uint8_t)(int8_t)gg << 16);
}

template <int D>
SA_D void write_token_fp16(uint8_t* block, const CacheArgs& a, int t, int lane, const uint16_t* krow,
                           const uint16_t* vrow) {
    constexpr int EPL = D / 32;
    uint32_t kb[EPL], vb[EPL];
    load_vec_bits<EPL>(krow, lane, kb);
    load_vec_bits<EPL>(vrow, lane, vb);
    const int m = lane * EPL;                        // K and V both in 16-byte chunks of 8 elements
    block += (size_t)(t >> 5) * (a.page_bytes >> 1);          // the token's half of the page
    t &= 31;
    const size_t off = ((size_t)(m >> 3) * kTileTokens + t) * 16 + (size_t)(m & 7) * 2;
    uint16_t* kdst = reinterpret_cast<uint16_t*>(block + a.kcode_off + off);
    uint16_t* vdst = reinterpret_cast<uint16_t*>(block + a.v_off + off);
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
        kdst[i] = (uint16_t)kb[i];
        vdst[i] = (uint16_t)vb[i];
    }
}

// block pointer of logical page `lp` of sequence b, KV head h; nullptr if unmapped / out of range
SA_D uint8_t* page_block(const CacheArgs& a, int b, int lp, int h) {
    if (lp < 0 || lp >= a.max_pages) return nullptr;
    const int pidx = a.page_table[(size_t)b * a.max_pages + lp];
    if (pidx < 0 || pidx >= a.n_pages) return nullptr;
    return a.pages + ((size_t)pidx * a.Hkv + h) * a.page_bytes;
}

// MODE: 0..4 = power-of-two code with K mantissa bits (byte container), 8 = PoT-4 nibble, 9 / 10 = PoT-M1 /
// PoT-M2 in the dense planar container, 16 = FP16, 32 = uniform INT8 comparison code
template <int D, int MODE>
SA_D void write_token(uint8_t* block, const CacheArgs& a, int t, int lane, const uint16_t* krow,
                      const uint16_t* vrow) {
    if constexpr (MODE == 16) write_token_fp16<D>(block, a, t, lane, krow, vrow);
    else if constexpr (MODE == 8) write_token_quant<D, 0, true>(block, a, t, lane, krow, vrow);
    else if constexpr (MODE == 9) write_token_quant<D, 1, true>(block, a, t, lane, krow, vrow);
    else if constexpr (MODE == 10) write_token_quant<D, 2, true>(block, a, t, lane, krow, vrow);
    else if constexpr (MODE == 32) write_token_quant<D, 8, false>(block, a, t, lane, krow, vrow);
    else write_token_quant<D, MODE, false>(block, a, t, lane, krow, vrow);
}

}  // namespace sa
