// Warp-level tensor-core primitives used by the decode kernels (legacy mma.sync shapes: the tiles of
// a decode step have n = 8 and are far too small for the asynchronous tcgen05 path to pay).
#pragma once
#include "sa_common.cuh"

namespace sa {

// D(16x8, f32) += A(16x16, f16, row) * B(16x8, f16, col)
SA_D void mma_f16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// D(16x8, f32) += A(16x8, tf32, row) * B(8x8, tf32, col).  Operands are FP32 bit patterns whose
// low 13 mantissa bits are zero (the callers make them so), i.e. exact tf32 values.
// Lane (g = lane / 4, t = lane % 4): a0 = A[g][t], a1 = A[g + 8][t], a2 = A[g][t + 4], a3 = A[g + 8][t + 4];
// b0 = B[t][g], b1 = B[t + 4][g]; d0 = D[g][2t], d1 = D[g][2t + 1], d2 = D[g + 8][2t], d3 = D[g + 8][2t + 1].
SA_D void mma_tf32_1688(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Four 8 x 8 matrices of 16-bit elements, transposed on the way: lane i supplies the address of
// row i % 8 of matrix i / 8 (16 bytes); lane (g, t) receives from matrix j the two elements
// M_j[2t][g] (low half of r[j]) and M_j[2t + 1][g] (high half).
SA_D void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr)
                 : "memory");
}
// maximum of a signed integer over the warp, one instruction
SA_D int warp_max_s32(int v) {
    int r;
    asm volatile("redux.sync.max.s32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(v));
    return r;
}

SA_D int warp_min_s32(int v) {
    int r;
    asm volatile("redux.sync.min.s32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(v));
    return r;
}

}  // namespace sa
