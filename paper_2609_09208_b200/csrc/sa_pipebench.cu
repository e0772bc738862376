// Instruction-throughput micro-benchmarks: timed chains of one instruction kind (or a fixed mix)
// on every SM.  They replace the paper's disassembly-based operation counts (Table V) with
// measured issue rates on this machine and provide the denominator of the integer-pipe roofline.
// Each thread keeps 8 independent chains so that latency does not limit the rate.
#include "sa_common.cuh"

namespace sa {

enum PipeKind {
    PK_SHL = 0,       // x = x << r (variable amount)
    PK_LOP3 = 1,      // x = (x ^ a) & b
    PK_IADD3 = 2,     // x = x + a + b
    PK_IMAD_ONE = 3,  // x = x * 1 + a, the 1 opaque to the compiler (an add issued as multiply-add)
    PK_PRMT = 4,      // byte permute
    PK_SHL_IMAD = 5,  // alternating variable shift and multiply-add by one
    PK_LOP3_IMAD = 6, // alternating logic op and multiply-add by one
    PK_FFMA = 7,
    PK_FFMA2 = 8,     // packed fma.rn.f32x2 (two FMAs per instruction)
    PK_IMAD = 9,      // x = x * m + a, general multiplier
    PK_DP4A = 10,     // four-way INT8 dot product accumulate
    PK_POPC = 11,
    PK_I2F = 12,      // int8 -> float conversion
    PK_SHL_LOP3_IMAD = 13,  // shift, logic, add-as-multiply-add in the ratio 1:1:1
    PK_VSHL_WRAP_ADD = 14,  // x = (x << r) + a as ONE scalar video instruction, shift amount taken modulo 32
    PK_VSHL_CLAMP_ADD = 15, // the same with the shift amount clamped to 32
    PK_SHL_ADD = 16,        // x = (x << r) + a as a plain shift followed by an add (two instructions)
    PK_LDS128_BCAST = 17,   // 128-bit shared-memory load, all lanes of a warp at the same address
    PK_LDS64_GATHER = 18,   // 64-bit shared-memory load, every lane its own entry of one 128-byte row
    PK_CVT_F32_S32 = 19,    // int32 -> float
    PK_CVT_S32_F32 = 20,    // float -> int32, rounding up (the ceiling of the softmax's running maximum)
    PK_EX2 = 21,            // ex2.approx
    PK_CVT_F32_S8 = 22,     // byte of a register -> float, no dependent add
    PK_PRMT_FADD = 23,      // the same conversion as a byte permute into a magic constant and one FP32 add
    PK_IMAD_HI = 24,        // mul.hi (an arithmetic right shift by a constant on the FMA pipe)
    PK_LDS64_SCATTERED = 25, // as PK_LDS64_GATHER, the lanes' entries drawn irregularly (repeats within and across the half-warps)
    PK_COUNT = 26
};

template <int KIND>
__global__ void __launch_bounds__(256) pipe_kernel(int iters, uint32_t one, uint32_t amount, uint32_t* sink) {
    __shared__ __align__(128) uint32_t tab_s[8 * 32];      // eight rows of 128 bytes (the shared-memory kinds)
    tab_s[threadIdx.x] = 0u;                                // zeros: a loaded value never moves the next address
    __syncthreads();
    const uint32_t tab = (uint32_t)__cvta_generic_to_shared(tab_s);
    uint32_t x[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = threadIdx.x * 2654435761u + i * 40503u + blockIdx.x;
    if (KIND == PK_LDS128_BCAST || KIND == PK_LDS64_GATHER || KIND == PK_LDS64_SCATTERED) {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = 0u;              // these chains carry an address offset, which stays 0
    }
    const uint32_t a = x[3] | 1u, b = ~x[5], r = amount & 7u, m = one * 3u;
    float f[8];
    unsigned long long f2[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        f[i] = (float)(x[i] & 1023u);
        f2[i] = pack_f32x2(f[i], f[i] + 1.0f);
    }
    const float fa = (float)(one) * 0.999f, fb = (float)amount * 1e-3f;
    const unsigned long long fa2 = pack_f32x2(fa, fa), fb2 = pack_f32x2(fb, fb);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (KIND == PK_SHL) {
                    asm volatile("shl.b32 %0, %0, %1;" : "+r"(x[i]) : "r"(r));
                } else if (KIND == PK_LOP3) {
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x60;" : "+r"(x[i]) : "r"(a), "r"(b));   // (x ^ a) & b
                } else if (KIND == PK_IADD3) {
                    asm volatile("{ .reg .u32 t; add.u32 t, %0, %1; add.u32 %0, t, %2; }" : "+r"(x[i]) : "r"(a), "r"(b));
                } else if (KIND == PK_IMAD_ONE) {
                    asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(one), "r"(a));
                } else if (KIND == PK_PRMT) {
                    asm volatile("prmt.b32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(a), "r"(amount));
                } else if (KIND == PK_SHL_IMAD) {
                    if (u & 1) asm volatile("shl.b32 %0, %0, %1;" : "+r"(x[i]) : "r"(r));
                    else asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(one), "r"(a));
                } else if (KIND == PK_LOP3_IMAD) {
                    if (u & 1) asm volatile("lop3.b32 %0, %0, %1, %2, 0x60;" : "+r"(x[i]) : "r"(a), "r"(b));
                    else asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(one), "r"(a));
                } else if (KIND == PK_FFMA) {
                    asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f[i]) : "f"(fa), "f"(fb));
                } else if (KIND == PK_FFMA2) {
                    asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(f2[i]) : "l"(fa2), "l"(fb2));
                } else if (KIND == PK_IMAD) {
                    asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(m), "r"(a));
                } else if (KIND == PK_DP4A) {
                    asm volatile("dp4a.s32.s32 %0, %1, %2, %0;" : "+r"(x[i]) : "r"(a), "r"(b));
                } else if (KIND == PK_POPC) {
                    asm volatile("{ .reg .u32 t; popc.b32 t, %0; add.u32 %0, %0, t; }" : "+r"(x[i]));
                } else if (KIND == PK_I2F) {
                    asm volatile("{ .reg .f32 t; cvt.rn.f32.s8 t, %1; add.f32 %0, %0, t; }" : "+f"(f[i]) : "r"(x[i]));
                } else if (KIND == PK_VSHL_WRAP_ADD) {
                    asm volatile("vshl.u32.u32.u32.wrap.add %0, %0, %1, %2;" : "+r"(x[i]) : "r"(r), "r"(a));
                } else if (KIND == PK_VSHL_CLAMP_ADD) {
                    asm volatile("vshl.u32.u32.u32.clamp.add %0, %0, %1, %2;" : "+r"(x[i]) : "r"(r), "r"(a));
                } else if (KIND == PK_SHL_ADD) {
                    asm volatile("{ .reg .u32 t; shl.b32 t, %0, %1; add.u32 %0, t, %2; }" : "+r"(x[i]) : "r"(r), "r"(a));
                } else if (KIND == PK_LDS128_BCAST) {
                    // the address depends on the value loaded before (always 0), all lanes read the same 16 bytes;
                    // volatile, here and below, so that the access keeps its width although only its first word is used
                    uint32_t y, z, w;
                    asm volatile("ld.volatile.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(x[i]), "=r"(y), "=r"(z), "=r"(w) : "r"(tab + i * 128 + x[i]));
                } else if (KIND == PK_LDS64_GATHER) {
                    uint32_t y;
                    asm volatile("ld.volatile.shared.v2.u32 {%0, %1}, [%2];" : "=r"(x[i]), "=r"(y) : "r"(tab + i * 128 + ((threadIdx.x * 5u) & 15u) * 8u + x[i]));
                } else if (KIND == PK_LDS64_SCATTERED) {
                    uint32_t y;
                    const uint32_t e = ((threadIdx.x * 2654435761u) >> 13) & 15u;      // 11 distinct entries per warp, unevenly spread
                    asm volatile("ld.volatile.shared.v2.u32 {%0, %1}, [%2];" : "=r"(x[i]), "=r"(y) : "r"(tab + i * 128 + e * 8u + x[i]));
                } else if (KIND == PK_CVT_F32_S32) {
                    asm volatile("{ .reg .f32 t; cvt.rn.f32.s32 t, %0; mov.b32 %0, t; }" : "+r"(x[i]));
                } else if (KIND == PK_CVT_S32_F32) {
                    asm volatile("{ .reg .s32 t; cvt.rpi.s32.f32 t, %0; mov.b32 %0, t; }" : "+f"(f[i]));
                } else if (KIND == PK_EX2) {
                    asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(f[i]));
                } else if (KIND == PK_CVT_F32_S8) {
                    asm volatile("{ .reg .f32 t; cvt.rn.f32.s8 t, %0; mov.b32 %0, t; }" : "+r"(x[i]));
                } else if (KIND == PK_PRMT_FADD) {
                    asm volatile("{ .reg .b32 t; .reg .f32 u; prmt.b32 t, %0, 0x4b000000, 0x7650; mov.b32 u, t; add.f32 u, u, 0fCB000080; mov.b32 %0, u; }" : "+r"(x[i]));
                } else if (KIND == PK_IMAD_HI) {
                    asm volatile("mul.hi.s32 %0, %0, %1;" : "+r"(x[i]) : "r"(m << 27));
                } else if (KIND == PK_SHL_LOP3_IMAD) {
                    const int k3 = (u * 8 + i) % 3;
                    if (k3 == 0) asm volatile("shl.b32 %0, %0, %1;" : "+r"(x[i]) : "r"(r));
                    else if (k3 == 1) asm volatile("lop3.b32 %0, %0, %1, %2, 0x60;" : "+r"(x[i]) : "r"(a), "r"(b));
                    else asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(one), "r"(a));
                }
            }
        }
    }
    uint32_t acc = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float lo, hi;
        unpack_f32x2(f2[i], &lo, &hi);
        acc += x[i] + __float_as_uint(f[i]) + __float_as_uint(lo) + __float_as_uint(hi);
    }
    if (acc == 0x12345678u) sink[0] = acc;     // practically never true; keeps the chains alive
}

}  // namespace sa

using namespace sa;

// Launches `blocks` blocks of 256 threads of micro-benchmark `kind`; every thread executes
// iters * 64 instructions of that kind (kinds named "a+b": 64 pairs of the two instructions).
// `sink` is a device word that is (almost) never written.  The paper has no counterpart: this
// stands in for its disassembly-based operation counts.
extern "C" sa_status sa_pipe_microbench(int kind, int iters, int blocks, uint32_t* sink, sa_stream stream) {
    if (kind < 0 || kind >= PK_COUNT || iters <= 0 || blocks <= 0 || !sink) return SA_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
#define CASE(K) case K: pipe_kernel<K><<<blocks, 256, 0, s>>>(iters, 1u, 3u, sink); break;
    switch (kind) {
        CASE(0) CASE(1) CASE(2) CASE(3) CASE(4) CASE(5) CASE(6) CASE(7) CASE(8) CASE(9) CASE(10) CASE(11) CASE(12) CASE(13)
        CASE(14) CASE(15) CASE(16) CASE(17) CASE(18) CASE(19) CASE(20) CASE(21) CASE(22) CASE(23) CASE(24) CASE(25)
    }
#undef CASE
    return cudaGetLastError() == cudaSuccess ? SA_OK : SA_ERR_CUDA;
}
