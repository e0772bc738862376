// The integer score datapath of the decode kernel (section II-B eq. (3), II-C eq. (4), II-D
// eq. (5)): shifts, sign flips and adds only.  Everything here also compiles for the host so
// that the unit tests can run the very same arithmetic against the CPU oracle without a GPU.
//
// Term of element m at head-room F0 = 6 + KB:  sigma * (qhat << r) * (2^KB + j),  r = 6 - e >= 0.
//
// PoT-4 (KB = 0), packed datapath:
// * Two queries share one 32-bit register: P = (q_hi << 16) + q_lo as a 32-bit integer (a negative
//   q_lo borrows from the upper half; all arithmetic below is plain integer arithmetic on P, so
//   the two halves stay exact as long as the lower half's running sum fits in 16 bits).  One
//   shift and one add then serve two (query, element) pairs.
// * The shift P << r depends on the key only through its exponent, so the block shifts every packed
//   pair by every r once (ShiftTable) and the key loop looks the shifted pair up.
// * The sign flip and the add are one multiply-add by sigma = +1 or -1 (the multiplier only ever
//   sees +1 or -1: magnitudes are shifted, never multiplied).  It issues on the FMA pipe while the
//   byte permutes issue on the ALU pipe: on sm_100a the two pipes run side by side
//   (64 + 64 thread-instructions per clock per SM).
// * A window of 4 elements (4 * 127 * 2^6 < 2^15) is accumulated in the packed register, whose
//   lower half is biased by 0x8000 so that it never borrows; then both halves are added into
//   32-bit totals.
// Mantissa codes (KB = 1, 2, 4): table datapath, see TableScore below.
//
// Physical code format inside a page: byte container  sign << 7 | mantissa field << 3 | g  (phys_byte in
// sa_common.cuh), nibble  sign << 3 | g,  with g = 7 - e for a non-zero element and 0 for the zero code.
// The shift amount is g - 1, which is 0xffffffff for the zero code, and a shift by 32 or more returns 0.
#pragma once
#include "sa_common.cuh"

namespace sa {

SA_HD uint32_t shl_clamp_hd(uint32_t x, uint32_t n) {
#ifdef __CUDA_ARCH__
    return shl_clamp(x, n);
#else
    return n >= 32u ? 0u : (x << n);
#endif
}
// Ablation only (SA_ABLATE_SIGNED_SHIFT): a shift whose direction is decided per term, as a datapath without
// head-room would need: amount r - 3, left when that is non-negative, else arithmetic right (dropping bits).
SA_HD uint32_t shl_signed_hd(uint32_t x, uint32_t r) {
    const int rs = (int)r - 3;
    const uint32_t left = shl_clamp_hd(x, (uint32_t)rs), right = (uint32_t)((int32_t)x >> ((-rs) & 31));
    return rs >= 0 ? left : right;
}
#ifdef SA_ABLATE_SIGNED_SHIFT
#define SA_TERM_SHIFT shl_signed_hd
#else
#define SA_TERM_SHIFT shl_clamp_hd
#endif
SA_HD int popc_hd(uint32_t x) {
#ifdef __CUDA_ARCH__
    return __popc(x);
#else
    return __builtin_popcount(x);
#endif
}
// Byte permute with the generic PTX semantics: selector nibble n picks byte (n & 7) of {a, b};
// with bit 3 set the byte's most significant bit is replicated over the result byte instead.
SA_HD uint32_t prmt_hd(uint32_t a, uint32_t b, uint32_t sel) {
#ifdef __CUDA_ARCH__
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
#else
    const unsigned long long ab = ((unsigned long long)b << 32) | a;
    uint32_t d = 0;
    for (int n = 0; n < 4; ++n) {
        const uint32_t s = (sel >> (4 * n)) & 0xfu;
        uint32_t byte = (uint32_t)(ab >> (8 * (s & 7u))) & 0xffu;
        if (s & 8u) byte = (byte & 0x80u) ? 0xffu : 0x00u;
        d |= byte << (8 * n);
    }
    return d;
#endif
}
// a + b, issued as a * one + b (one == 1 at run time) so that it executes on the FMA pipe.
SA_HD uint32_t add_fma(uint32_t a, uint32_t b, uint32_t one) {
#ifdef __CUDA_ARCH__
    uint32_t d;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(one), "r"(b));
    return d;
#else
    return a * one + b;
#endif
}

// NP consecutive 32-bit words (NP = 1, 2, 4 or 8; min(16, 4 * NP)-byte aligned) with vector loads.
template <int NP>
SA_HD void load_np(const uint32_t* src, uint32_t (&q)[NP]) {
    if constexpr (NP == 8) {
        const uint4 v0 = reinterpret_cast<const uint4*>(src)[0], v1 = reinterpret_cast<const uint4*>(src)[1];
        q[0] = v0.x; q[1] = v0.y; q[2] = v0.z; q[3] = v0.w;
        q[4] = v1.x; q[5] = v1.y; q[6] = v1.z; q[7] = v1.w;
    } else if constexpr (NP == 4) {
        const uint4 v = *reinterpret_cast<const uint4*>(src);
        q[0] = v.x; q[1] = v.y; q[2] = v.z; q[3] = v.w;
    } else if constexpr (NP == 2) {
        const uint2 v = *reinterpret_cast<const uint2*>(src);
        q[0] = v.x; q[1] = v.y;
    } else {
        q[0] = src[0];
    }
}

// a * w + c on the FMA pipe; w is either a power of two held in a register (a shift-and-add) or a
// sign +1 / -1 (a sign flip and an add).
SA_HD uint32_t mad_fma(uint32_t a, uint32_t w, uint32_t c) {
#ifdef __CUDA_ARCH__
    uint32_t d;
    asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(w), "r"(c));
    return d;
#else
    return a * w + c;
#endif
}

// c + x with the sign flip of x chosen by the mask s (0: +x, 0xffffffff: -x) done as exclusive-or and
// subtract: logic and add instructions only, no multiplier.
SA_HD uint32_t flip_add(uint32_t x, uint32_t s, uint32_t c) {
#ifdef __CUDA_ARCH__
    // one opaque unit, like the multiply-add it stands in for (left as plain C the three operations of the many
    // independent updates are interleaved so freely that the kernel spills)
    uint32_t d;
    asm("{\n\t.reg .b32 t;\n\txor.b32 t, %1, %2;\n\tsub.s32 t, t, %2;\n\tadd.s32 %0, t, %3;\n\t}" : "=r"(d) : "r"(x), "r"(s), "r"(c));
    return d;
#else
    return c + ((x ^ s) - s);
#endif
}

SA_HD uint32_t pack_pair(int q_lo, int q_hi) { return ((uint32_t)q_hi << 16) + (uint32_t)q_lo; }

// Accumulators for 2 * NP queries against one PoT-4 key.
//
// Flush of a window register W = h * 2^16 + l (l = biased lower half, 0 <= l < 2^16): instead of
// separating both halves, two totals are kept modulo 2^32,
//     tot += W        and        hit += h        (h = W >> 16, arithmetic),
// and at the end  lower-query sum = tot - (hit << 16) - bias  (exact: the true value is far below
// 2^32) and  upper-query sum = hit.  That is one ALU instruction and two FMA-pipe adds per window
// register.
// ALU (SA_FLAG_ADD_ON_ALU, not the default): sg is a sign MASK (0 / 0xffffffff) and every sign flip and add
// is an exclusive-or, a subtract and an add on the ALU pipe; the multiplier array is not used at all.
template <int NP, bool ALU = false>
struct PackedShift {
    uint32_t win[NP];           // window sums, lower half biased by 0x8000
    uint32_t tot[NP], hit[NP];  // running totals, see above
    uint32_t n_windows;
    uint32_t one;               // 1, as a run-time value (keeps the adds on the FMA pipe)

    SA_HD void begin(uint32_t one_) {
        one = one_;
        n_windows = 0;
#pragma unroll
        for (int p = 0; p < NP; ++p) tot[p] = hit[p] = 0;
    }
    // sg: +1 or -1 (ALU: the sign mask); x: the element's packed pairs, already shifted (an entry of ShiftTable)
    SA_HD void entry_first(uint32_t sg, const uint32_t (&x)[NP]) {
#pragma unroll
        for (int p = 0; p < NP; ++p) win[p] = ALU ? flip_add(x[p], sg, 0x8000u) : mad_fma(x[p], sg, 0x8000u);
    }
    SA_HD void entry_next(uint32_t sg, const uint32_t (&x)[NP]) {
#pragma unroll
        for (int p = 0; p < NP; ++p) win[p] = ALU ? flip_add(x[p], sg, win[p]) : mad_fma(x[p], sg, win[p]);
    }
    SA_HD void window_end() {
        ++n_windows;
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            const uint32_t h = (uint32_t)((int32_t)win[p] >> 16);      // exact upper half
            tot[p] = ALU ? win[p] + tot[p] : add_fma(win[p], tot[p], one);
            hit[p] = ALU ? h + hit[p] : add_fma(h, hit[p], one);
        }
    }
    // score of query g (g even: lower half of register g / 2), before the final head-room shift
    SA_HD int32_t score(int g) const {
        return (g & 1) ? (int32_t)hit[g >> 1] : (int32_t)(tot[g >> 1] - (hit[g >> 1] << 16) - n_windows * 0x8000u);
    }
};

// ---------------------------------------------------------------------------------------------
// PoT-4 with the shifts hoisted out of the key loop.
//
// The shifted query q << r does not depend on the key, only on its exponent field: the block prepares
// S[m][g][pair] = packed pair of element m shifted left by g - 1 (g = 1 .. 7; the entry of g = 0, the
// zero code, is 0) once, in shared memory, and the key loop fetches the entry of ITS key's g — all
// query pairs of the element with one vector load — and adds it with the sign (one multiply-add by
// sigma on the FMA pipe per packed pair).  Per key element the ALU pipe then only sees two byte
// permutes.  The row of one element holds 8 entries of 4 NP bytes: lanes with different g read
// different banks, lanes with the same g the same address.  The windows, the bias and the totals are
// those of PackedShift; the values added are bit for bit the ones it would have shifted itself.
// ---------------------------------------------------------------------------------------------
template <int NP>
struct ShiftTable {
    static constexpr int kEntryBytes = 4 * NP;             // the NP packed pairs of one (element, g)
    static constexpr int kRowBytes = 8 * kEntryBytes;      // g = 0 .. 7: one element
    static constexpr int kShift = NP == 4 ? 4 : NP == 2 ? 3 : 2;      // log2(kEntryBytes)
    static_assert(NP == 1 || NP == 2 || NP == 4, "one, two or four packed query pairs");
    // entry g of a packed pair
    static SA_HD uint32_t entry(uint32_t packed, int g) { return g == 0 ? 0u : packed << (g - 1); }
    // low address byte of element e (counted from a 256-byte aligned group start) before its g is added,
    // and the rest of its offset
    static SA_HD constexpr uint32_t low(int e) { return (uint32_t)(e * kRowBytes) & 0xffu; }
    static SA_HD constexpr int high(int e) { return (e * kRowBytes) & ~0xff; }
};

// The NP words at (base with its low byte replaced by byte i of offs) + IMM.
template <int NP, int IMM>
SA_HD void shift_gather(uint32_t base, uint32_t offs, int i, uint32_t (&x)[NP]) {
#ifdef __CUDA_ARCH__
    const uint32_t addr = prmt_hd(offs, base, 0x7650u | (uint32_t)i);
    if constexpr (NP == 4) asm("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4+%5];" : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3]) : "r"(addr), "n"(IMM));
    else if constexpr (NP == 2) asm("ld.shared.v2.u32 {%0, %1}, [%2+%3];" : "=r"(x[0]), "=r"(x[1]) : "r"(addr), "n"(IMM));
    else asm("ld.shared.u32 %0, [%1+%2];" : "=r"(x[0]) : "r"(addr), "n"(IMM));
#else
    (void)base; (void)offs; (void)i;
    for (int p = 0; p < NP; ++p) x[p] = 0u;      // shared-space addresses exist on the device only
#endif
}
template <int NP, int IMM>
SA_HD void shift_gather(const uint8_t* base, uint32_t offs, int i, uint32_t (&x)[NP]) {
    const uintptr_t addr = (reinterpret_cast<uintptr_t>(base) & ~(uintptr_t)0xff) | ((offs >> (8 * i)) & 0xffu);
    const uint32_t* e = reinterpret_cast<const uint32_t*>(addr + IMM);
    for (int p = 0; p < NP; ++p) x[p] = e[p];
}

// Elements I .. 3 of one window: element E0 + STEP * I of the group, byte I of offs and of sw (sign at the
// byte's top bit).
template <int NP, int E0, int STEP, int I, bool ALU, typename Base>
SA_HD void shift_window(PackedShift<NP, ALU>& pl, uint32_t sw, uint32_t offs, Base grp) {
    if constexpr (I < 4) {
        using ST = ShiftTable<NP>;
        constexpr int e = E0 + STEP * I;
        uint32_t x[NP];
        shift_gather<NP, ST::high(e)>(grp, offs, I, x);
        const uint32_t sm = prmt_hd(sw, 0u, 0x8888u | (0x1111u * I));                 // sign mask: 0 / 0xffffffff
        const uint32_t sg = ALU ? sm : mad_fma(sm, pl.one + pl.one, pl.one);          // +1 / -1
        if (I == 0) pl.entry_first(sg, x);
        else pl.entry_next(sg, x);
        shift_window<NP, E0, STEP, I + 1, ALU>(pl, sw, offs, grp);
    }
}

// One 32-bit word of the byte container = 4 elements: word W4 (0 .. 3) of a group of 16 elements whose
// table rows start at grp (256-byte aligned).
template <int NP, int W4, bool ALU, typename Base>
SA_HD void accumulate_word_bytes_tab(PackedShift<NP, ALU>& pl, uint32_t w, Base grp) {
    using ST = ShiftTable<NP>;
    constexpr uint32_t pattern = ST::low(W4 * 4) | (ST::low(W4 * 4 + 1) << 8) | (ST::low(W4 * 4 + 2) << 16) | (ST::low(W4 * 4 + 3) << 24);
    const uint32_t offs = ((w << ST::kShift) & (0x07070707u << ST::kShift)) | pattern;      // g * entry bytes + row
    shift_window<NP, W4 * 4, 1, 0, ALU>(pl, w, offs, grp);
    pl.window_end();
}

// One 32-bit word of the nibble container = 8 elements (low nibble = even element), two windows: the even
// and the odd elements (the order of the terms within the exact sum is free).  grp: the rows of the word's
// first element (256-byte aligned).
template <int NP, bool ALU, typename Base>
SA_HD void accumulate_word_nibbles_tab(PackedShift<NP, ALU>& pl, uint32_t w, Base grp) {
    using ST = ShiftTable<NP>;
    constexpr uint32_t pat_e = ST::low(0) | (ST::low(2) << 8) | (ST::low(4) << 16) | (ST::low(6) << 24);
    constexpr uint32_t pat_o = ST::low(1) | (ST::low(3) << 8) | (ST::low(5) << 16) | (ST::low(7) << 24);
    const uint32_t we = w << 4;                                          // even elements' sign at the byte's top bit
    const uint32_t offs_e = ((w << ST::kShift) & (0x07070707u << ST::kShift)) | pat_e;
    const uint32_t offs_o = ((w >> (4 - ST::kShift)) & (0x07070707u << ST::kShift)) | pat_o;
    shift_window<NP, 0, 2, 0, ALU>(pl, we, offs_e, grp);
    pl.window_end();
    shift_window<NP, 1, 2, 0, ALU>(pl, w, offs_o, grp);
    pl.window_end();
}

// ---------------------------------------------------------------------------------------------
// Table datapath for the mantissa codes (KB >= 1).
//
// The mantissa factor (2^KB + j) depends only on the key element, the query only on the block:
// the block prepares U[m][pair][mu] = {q_lo, q_hi}[m] * (2^KB + mu) for mu = 0 .. 2^KB - 1 once, by
// repeated addition (no multiplication), in shared memory.  The row of one (element, query pair)
// holds 2^KB entries of 8 bytes — 128 bytes for KB = 4, exactly the 32 banks — so the 32 lanes of
// a warp, each fetching the entry of ITS key's mantissa, never conflict (equal entries broadcast).
// Per (query, element) the work is then: half a 64-bit gather, one shift by r = 6 - e on the ALU
// pipe, and one multiply-add by sigma = +1 or -1 on the FMA pipe, which is the sign flip and the
// accumulation in one instruction (the multiplier only ever sees +1 or -1: magnitudes are shifted,
// never multiplied).  The term is at most 127 * 31 * 2^6 < 2^18, the sum of 128 of them fits
// INT32 (the host checks the bound with the head-room).
//
// Per key element, shared by all queries: one byte permute for the shift amount, one for the sign
// (turned into +1 / -1 on the FMA pipe), and one that drops the mantissa's byte offset into the low
// byte of the table address — which is why the table of a group of 16 elements starts on a
// 256-byte boundary and the rest of the address is an immediate.
// ---------------------------------------------------------------------------------------------
// Entry {x, y} at (base with its low byte replaced by byte i of offs) + IMM.  The kernel passes a
// shared-space address, the unit tests on the host a plain pointer.
template <int IMM>
SA_HD void table_gather(uint32_t base, uint32_t offs, int i, uint32_t& x, uint32_t& y) {
#ifdef __CUDA_ARCH__
    const uint32_t addr = prmt_hd(offs, base, 0x7650u | (uint32_t)i);
    asm("ld.shared.v2.u32 {%0, %1}, [%2+%3];" : "=r"(x), "=r"(y) : "r"(addr), "n"(IMM));
#else
    (void)base; (void)offs; (void)i;
    x = y = 0u;                      // shared-space addresses exist on the device only
#endif
}
template <int IMM>
SA_HD void table_gather(const uint8_t* base, uint32_t offs, int i, uint32_t& x, uint32_t& y) {
    const uintptr_t addr = (reinterpret_cast<uintptr_t>(base) & ~(uintptr_t)0xff) | ((offs >> (8 * i)) & 0xffu);
    const uint32_t* e = reinterpret_cast<const uint32_t*>(addr + IMM);
    x = e[0];
    y = e[1];
}

// MUL (SA_FLAG_SHIFT_BY_MULTIPLY, not the default): sigma * 2^r is formed once per key element and the
// update is one multiply-add of the table entry by it.
// ALU (SA_FLAG_ADD_ON_ALU, not the default): the sign flip and the add are an exclusive-or, a subtract and an
// add on the ALU pipe (sg is then the sign mask 0 / 0xffffffff); the multiplier array is not used at all.
template <int KB, int NGP, bool MUL = false, bool ALU = false>
struct TableScore {
    static_assert(!(MUL && ALU), "the two variants exclude one another");
    static constexpr int kRowBytes = 8 << KB;              // one (element, query pair) row
    static constexpr int kElemBytes = NGP * kRowBytes;     // all query pairs of one element
    static constexpr int kGroupBytes = 16 * kElemBytes;    // 16 elements = 4 code words; a multiple of 256
    uint32_t acc[2 * NGP];
    uint32_t one, two;                                     // 1 and 2 as run-time values (FMA-pipe arithmetic)
    SA_HD void begin(uint32_t one_) {
        one = one_;
        two = one_ + one_;
#pragma unroll
        for (int g = 0; g < 2 * NGP; ++g) acc[g] = 0;
    }
    // query pairs GP .. NGP - 1 of one element; IMM = byte offset of the element's rows within the group;
    // sg = sigma (with MUL: sigma * 2^r, and r is not used)
    template <int IMM, int GP, typename Base>
    SA_HD void element_pairs(Base grp, uint32_t offs, int i, uint32_t r, uint32_t sg) {
        if constexpr (GP < NGP) {
            uint32_t x, y;
            table_gather<IMM + GP * kRowBytes>(grp, offs, i, x, y);
            acc[2 * GP] = MUL ? mad_fma(x, sg, acc[2 * GP])
                          : ALU ? flip_add(SA_TERM_SHIFT(x, r), sg, acc[2 * GP]) : mad_fma(SA_TERM_SHIFT(x, r), sg, acc[2 * GP]);
            acc[2 * GP + 1] = MUL ? mad_fma(y, sg, acc[2 * GP + 1])
                              : ALU ? flip_add(SA_TERM_SHIFT(y, r), sg, acc[2 * GP + 1]) : mad_fma(SA_TERM_SHIFT(y, r), sg, acc[2 * GP + 1]);
            element_pairs<IMM, GP + 1>(grp, offs, i, r, sg);
        }
    }
    template <int W4, int I, typename Base>
    SA_HD void elements(uint32_t w, uint32_t rw, uint32_t offs, Base grp) {
        if constexpr (I < 4) {
            const uint32_t r = prmt_hd(rw, 0u, 0x4440u | I);
            const uint32_t sm = prmt_hd(w, 0u, 0x8888u | (0x1111u * I));                      // sign mask: 0 / 0xffffffff
            const uint32_t sg = ALU ? sm : mad_fma(sm, two, one);                             // sigma: +1 / -1
            element_pairs<(W4 * 4 + I) * kElemBytes, 0>(grp, offs, I, r, MUL ? shl_clamp_hd(sg, r) : sg);
            elements<W4, I + 1>(w, rw, offs, grp);
        }
    }
    // One 32-bit word of the byte container = 4 elements: word W4 (0..3) of a group of 16 elements
    // whose table starts at grp (256-byte aligned).
    template <int W4, typename Base>
    SA_HD void accumulate_word(uint32_t w, Base grp) {
        const uint32_t gw = w & 0x07070707u;
        const uint32_t rw = (gw + 0x7f7f7f7fu) ^ 0x80808080u;       // shift amounts g - 1; 0xff for the zero code
        // byte offsets mu * 8 of the mantissas' entries: the mantissa field (bits 3 .. 6) holds mu << (4 - KB)
        const uint32_t offs = KB == 4 ? w & 0x78787878u : KB == 2 ? (w >> 2) & 0x18181818u : (w >> 3) & 0x08080808u;
        elements<W4, 0>(w, rw, offs, grp);
    }
    // Dense planar container (PoT-M1 / PoT-M2 only): one 32-bit word of sign/exponent nibbles = 8
    // elements (low nibble = even element), with the elements' mantissa bits in KB separate bit
    // planes: bit ni of planes[b] is bit b of element ni's mantissa.  W8 = position of the word in
    // its group of 16 elements (0 or 1).
    template <int W8, int NI, typename Base>
    SA_HD void nibble_elements(uint32_t w, uint32_t we, uint32_t re, uint32_t ro, uint32_t offs_e, uint32_t offs_o, Base grp) {
        if constexpr (NI < 8) {
            constexpr int byte = NI >> 1;
            const uint32_t r = prmt_hd((NI & 1) ? ro : re, 0u, 0x4440u | byte);
            const uint32_t sm = prmt_hd((NI & 1) ? w : we, 0u, 0x8888u | (0x1111u * byte));
            const uint32_t sg = ALU ? sm : mad_fma(sm, two, one);
            element_pairs<(W8 * 8 + NI) * kElemBytes, 0>(grp, (NI & 1) ? offs_o : offs_e, byte, r, MUL ? shl_clamp_hd(sg, r) : sg);
            nibble_elements<W8, NI + 1>(w, we, re, ro, offs_e, offs_o, grp);
        }
    }
    template <int W8, typename Base>
    SA_HD void accumulate_nibble_word(uint32_t w, const uint32_t (&planes)[KB], Base grp) {
        static_assert(KB == 1 || KB == 2, "the planar container holds PoT-M1 and PoT-M2");
        const uint32_t ge = w & 0x07070707u, go = (w >> 4) & 0x07070707u;   // g of even / odd elements
        const uint32_t re = (ge + 0x7f7f7f7fu) ^ 0x80808080u, ro = (go + 0x7f7f7f7fu) ^ 0x80808080u;
        const uint32_t we = w << 4;                                         // even elements' sign at the byte's top bit
        // Byte offsets mu * 8 of the table entries, one byte per element: bit 2i of a plane byte goes
        // to bit 3 + b of byte i.  The product by 0x00208208 places copies of the byte at bit offsets
        // 3, 9, 15, 21; the mask keeps the wanted copy of each bit (a bit spread, not arithmetic on data).
        uint32_t offs_e = 0u, offs_o = 0u;
#pragma unroll
        for (int b = 0; b < KB; ++b) {
            offs_e |= (((planes[b] & 0x55u) * 0x00208208u) & 0x08080808u) << b;
            offs_o |= ((((planes[b] >> 1) & 0x55u) * 0x00208208u) & 0x08080808u) << b;
        }
        nibble_elements<W8, 0>(w, we, re, ro, offs_e, offs_o, grp);
    }
    SA_HD int32_t score(int g) const { return (int32_t)acc[g]; }
};

// Fill the table rows of element m for query pair gp: entry mu = {q_lo, q_hi} * (2^KB + mu).
template <int KB>
SA_HD void fill_table_row(uint8_t* row, int q_lo, int q_hi) {
    uint32_t a = (uint32_t)q_lo << KB, b = (uint32_t)q_hi << KB;
#pragma unroll
    for (int mu = 0; mu < (1 << KB); ++mu) {
        reinterpret_cast<uint32_t*>(row)[2 * mu] = a;
        reinterpret_cast<uint32_t*>(row)[2 * mu + 1] = b;
        a += (uint32_t)q_lo;
        b += (uint32_t)q_hi;
    }
}

}  // namespace sa
