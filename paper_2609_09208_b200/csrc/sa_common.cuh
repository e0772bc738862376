// Shared declarations of the CUDA library: host-side plan/validation helpers and the small
// exact-arithmetic device functions used by more than one kernel.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sa.h"

#define SA_HD __host__ __device__ __forceinline__
#define SA_D __device__ __forceinline__

namespace sa {

constexpr int kPageTokens = 64;
constexpr int kTileTokens = 32;           // a page block is two halves of 32 tokens, each laid out like one staged tile
// Bytes of one half of a (page, KV head) block: code chunks, mantissa bit planes (dense planar container),
// metadata, value chunks.  kb: mantissa bits (8 for the INT8 comparison code); nib: sub-byte container.
// The page plan (make_plan) and the kernels' stage plans are both checked against it.
constexpr int half_block_bytes(int d, int kb, bool nib) {
    return kTileTokens * (nib ? d / 2 : d) + ((nib && kb > 0) ? kb * kTileTokens * (d / 8) : 0) + kTileTokens * 4 + kTileTokens * d;
}
constexpr int half_block_bytes_fp16(int d) { return 2 * kTileTokens * d * 2; }
constexpr int kNumSMsB200 = 148;          // the split plan's SM count where no device can be asked (see sm_count())
constexpr int kEmax = 6;                  // largest exponent of the 3-bit field
constexpr int kMNone = -(1 << 29);        // running-maximum value meaning "no key seen yet"

// ---------------------------------------------------------------------------------------------
// Host-side description of a validated configuration.
// ---------------------------------------------------------------------------------------------
struct Plan {
    int d, Hq, Hkv, G, k;     // k = mantissa bits (0 for SA_KV_FP16)
    bool mulshift;            // SA_FLAG_SHIFT_BY_MULTIPLY: the scores' shifts run on the integer multiplier
    bool addalu;              // SA_FLAG_ADD_ON_ALU: sign flips and adds as logic/add instructions, no multiply-add
    bool fp16, nibble, hadamard, int8;   // nibble: 4-bit sign/exponent codes (PoT-4 nibble container, or with k = 1, 2
                                         // the dense planar container); int8: the uniform INT8 comparison code
    int F;                    // head-room actually used
    int f_extra;              // F - (6 + k): applied as one final left shift of the INT32 sum
    sa_layout lay;
    size_t plane_off;         // dense planar container: offset of the mantissa bit planes inside a block
};

sa_status make_plan(const sa_config* cfg, Plan* out);
// Warps per block and resident blocks per SM of the decode kernel that serves a code
// (kb: 0 PoT-4, 1 / 2 / 4 mantissa codes, 8 INT8; the kernels' launch bounds and shared-memory
// plans are sized for exactly this, and the split plan counts on it).  At d = 64 two blocks of ten
// warps (20 warps at 96 registers): for PoT-M4 the ten warps share one 32 KB table of query
// multiples, and for every code fewer, larger blocks mean fewer prologues and partials, which is
// most of the time of a batch-1 step.  PoT-M1 / M2 keep four blocks of four warps: their finer
// granularity serves the short and ragged batches those codes are specified for (measured: 16 %
// faster there, 6 % slower at T = 32768, batch 1).  At d = 128 (8 KB tiles, one stage buffer per
// warp) PoT-M4 runs two blocks of eight warps beside their 32 KB tables (16 warps at 128 registers;
// measured 3 - 22 % faster than three blocks of four); the other codes keep blocks of four warps
// (larger blocks measured 2 - 13 % slower for them from batch 8 on).
struct KernelShape {
    int warps, blocks_per_sm;
};
constexpr KernelShape decode_shape(int d, int kb) {
    return (kb == 1 || kb == 2) ? KernelShape{4, 4}
           : (d == 64)          ? KernelShape{10, 2}
           : (kb == 4)          ? KernelShape{8, 2}
                                : KernelShape{4, 5};
}
constexpr KernelShape kFp16Shape{4, 3};
// Streaming multiprocessors of the current device (cudaDevAttrMultiProcessorCount, asked once per device; 148,
// a B200, where no device answers, so that the size queries also work on a machine without a GPU).
int sm_count();
// number of splits of the key axis for a cache of this shape, and queries handled per block
void split_plan(const Plan& p, int batch, int max_pages, int* n_splits, int* gt);

// ---------------------------------------------------------------------------------------------
// Exact helpers (usable on host for unit tests of the arithmetic, and on device).
// ---------------------------------------------------------------------------------------------

// Byte container: physical byte of a canonical code byte (sign << 7 | e << 4 | mantissa << (4 - k)):
//   sign << 7 | mantissa field << 3 | g,   g = 7 - e for a non-zero element, 0 for the zero code.
// The exponent field sits in the low bits (g - 1 is the shift amount), the mantissa field at bits
// 3 .. 6 (times 8 it is the byte offset of a table entry), and zeroed memory reads as zero codes.
SA_HD uint8_t phys_byte(uint8_t canon) {
    return (uint8_t)((canon & 0x80u) | ((canon & 0x0fu) << 3) | (((canon >> 4) & 7u) ^ 7u));
}
SA_HD uint8_t canon_byte(uint8_t phys) {
    return (uint8_t)((phys & 0x80u) | (((phys & 7u) ^ 7u) << 4) | ((phys >> 3) & 0x0fu));
}

// Normalise a non-zero binary16 magnitude (15 bits) to M * 2^X with M in [1024, 2047].
SA_HD void half_normalise(uint32_t mag_bits, int* M, int* X) {
    const int ex = (int)(mag_bits >> 10);
    const int man = (int)(mag_bits & 0x3ff);
    if (ex != 0) {
        *M = 1024 + man;
        *X = ex - 25;
    } else {
#ifdef __CUDA_ARCH__
        const int sh = __clz(man) - 21;
#else
        int sh = 0;
        while (((man << sh) & 0x400) == 0) ++sh;
#endif
        *M = man << sh;
        *X = -24 - sh;
    }
}

// Code of one key element (section II-A, II-D): `a_bits` the element's binary16 bits, `s_bits`
// the magnitude bits of the vector's scale (the largest magnitude in the vector), K the number of
// mantissa bits.  Returns the canonical byte.  Integer arithmetic only, hence exact:
//   u = a/s = rho * 2^-e0 with rho in [1, 2);  j = floor((rho - 1) 2^K);  with n = 2^K + j the
//   neighbours on the grid are n and n + 1 (in units of 2^(-K-e0)), and the upper one is nearer
//   in log2 exactly when rho^2 4^K >= n (n + 1).
template <int K>
SA_HD uint8_t encode_element(uint32_t a_bits, uint32_t s_bits) {
    const uint32_t mag = a_bits & 0x7fffu;
    if (mag == 0) return 0x70;
    int Ma, Xa, Ms, Xs;
    half_normalise(mag, &Ma, &Xa);
    half_normalise(s_bits & 0x7fffu, &Ms, &Xs);
    int e0 = Xs - Xa;
    uint32_t num = (uint32_t)Ma;
    if (Ma < Ms) { e0 += 1; num <<= 1; }
    if (e0 > 8) return 0x70;                       // far below the grid; also keeps e0 small
    uint32_t j = ((num - (uint32_t)Ms) << K) / (uint32_t)Ms;
    const unsigned long long n = (1u << K) + j;
    const unsigned long long lhs = (unsigned long long)num * num << (2 * K);
    const unsigned long long rhs = n * (n + 1) * (unsigned long long)Ms * (unsigned long long)Ms;
    if (lhs >= rhs) {
        ++j;
        if (j == (1u << K)) { j = 0; --e0; }
    }
    if (e0 >= 7) return 0x70;
    return (uint8_t)(((a_bits >> 15) << 7) | ((uint32_t)e0 << 4) | (j << (4 - K)));
}

// Power-of-two exponent g of the value scale: the largest g with amax * 2^g <= 127
// (section II-E).  amax = M * 2^X, so amax * 2^g <= 127  <=>  M * 2^(X + g + 4) <= 2032.
SA_HD int value_exponent(uint32_t amax_bits) {
    if ((amax_bits & 0x7fffu) == 0) return 0;
    int M, X;
    half_normalise(amax_bits & 0x7fffu, &M, &X);
    return (M <= 2032) ? (-4 - X) : (-5 - X);
}

#ifdef __CUDACC__
// ---------------------------------------------------------------------------------------------
// Device-only helpers.
// ---------------------------------------------------------------------------------------------

// Left shift with the PTX guarantee that amounts >= 32 give 0.  The zero code (e = 7) yields
// the shift amount 6 - 7 = 0xffffffff, so a zero element contributes 0 without a branch.
SA_D uint32_t shl_clamp(uint32_t x, uint32_t n) {
    uint32_t r;
    asm("shl.b32 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(n));
    return r;
}

// Programmatic dependent launch: a kernel launched with the attribute may start while its
// predecessor in the stream is still draining; it must call pdl_wait() before it touches anything the
// predecessor wrote.  Both are no-ops in a kernel launched the ordinary way.
SA_D void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
SA_D void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

SA_D uint32_t warp_max_u32(uint32_t v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
SA_D float warp_max_f32(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
SA_D float warp_sum_f32(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

SA_D float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Packed FP32 pair multiply-add of sm_100: d = a * b + c on two lanes held in one 64-bit register.
SA_D unsigned long long ffma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
SA_D unsigned long long pack_f32x2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
SA_D void unpack_f32x2(unsigned long long v, float* lo, float* hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(*lo), "=f"(*hi) : "l"(v));
}

// Walsh-Hadamard rotation of one head vector spread over a warp: lane l holds elements
// l*EPL .. l*EPL+EPL-1 in x[].  Sylvester order, butterflies with strides 1, 2, ..., d/2, each
// (a, b) <- (a + b, a - b) in FP32 with one rounding per add (no contraction is possible: there
// is no multiply), then one multiply by 1/sqrt(d) and a round to binary16.  Returns the rotated
// elements as binary16 bit patterns.
template <int EPL>
SA_D void hadamard_warp(float (&x)[EPL], uint32_t (&bits)[EPL], int lane) {
#pragma unroll
    for (int h = 1; h < EPL; h <<= 1) {
#pragma unroll
        for (int i = 0; i < EPL; ++i)
            if ((i & h) == 0) {
                const float a = x[i], b = x[i + h];
                x[i] = __fadd_rn(a, b);
                x[i + h] = __fsub_rn(a, b);
            }
    }
#pragma unroll
    for (int hl = 1; hl < 32; hl <<= 1) {
#pragma unroll
        for (int i = 0; i < EPL; ++i) {
            const float other = __shfl_xor_sync(0xffffffffu, x[i], hl);
            x[i] = (lane & hl) ? __fsub_rn(other, x[i]) : __fadd_rn(x[i], other);
        }
    }
    const float scale = (EPL == 2) ? 0.125f : 0.088388346f;   // 1/sqrt(64), 1/sqrt(128)
#pragma unroll
    for (int i = 0; i < EPL; ++i) bits[i] = __half_as_ushort(__float2half_rn(__fmul_rn(x[i], scale)));
}

// First tile of split s when n_tiles tiles are cut into n_splits slices: floor(n_tiles * s / n_splits) in 32-bit
// unsigned arithmetic (a 64-bit division is a long software routine on the GPU, and this sits on the critical
// path of every block); the host refuses caches with max tiles * splits >= 2^31.
SA_D int split_begin(int n_tiles, int s, int n_splits) {
    return (int)((uint32_t)n_tiles * (uint32_t)s / (uint32_t)n_splits);
}
// 2^e as a float, built from the exponent field; e must lie in [-126, 127].
SA_D float pow2i(int e) { return __int_as_float((e + 127) << 23); }
// 2^e for e <= 0, flushing to 0 below the normal range (used for softmax rescales, which are
// exact power-of-two factors because the running maximum is an integer).
SA_D float pow2i_neg(int e) { return e < -126 ? 0.0f : __int_as_float((e + 127) << 23); }

SA_D float half_bits_to_float(uint32_t b) { return __half2float(__ushort_as_half((unsigned short)b)); }
#endif  // __CUDACC__

#ifdef __CUDACC__
// Launch with programmatic stream serialisation allowed (see pdl_wait above).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}
#endif

}  // namespace sa
