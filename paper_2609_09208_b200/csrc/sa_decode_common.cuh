// Pieces shared by the quantised and the FP16 decode kernels: kernel arguments, the merge of
// the four warps of a block, and the split-K merge (section II-F: the grid has a split
// dimension; the merge rule follows from the integer running maximum of section II-E:
// M* = max_s M_s, every partial is rescaled by the exact factor 2^(M_s - M*)).
#pragma once
#include "sa_common.cuh"

namespace sa {

struct DecodeArgs {
    const uint8_t* pages;
    const int32_t* page_table;
    const int32_t* seq_lens;
    const uint16_t* Q;
    float* O;
    float* partials;          // [n_splits][batch][Hq][D + 2]: {M (int bits), l, O[D]}
    int32_t* dbg_scores;
    size_t dbg_stride;
    int batch, Hq, Hkv, G, max_pages, n_pages, n_splits, f_extra, hadamard;
    size_t page_bytes, kcode_off, meta_off, v_off, plane_off;
    float zscale;
    uint32_t one;             // the value 1, opaque to the compiler (adds issued as multiply-add)
    // Shift-based A.V option (eq. (6), (7)); all null / 0 on the default path.
    int32_t* zr;              // [batch][Hq][dbg_stride] rounded logits, written by the score pass
    int32_t* stat_m;          // [n_splits][batch][Hq] ceil of the largest logit of the split
    int32_t* stat_g;          // [n_splits][batch][gridDim.y] smallest value exponent g of the split
    int n_bits, k_max;        // N and k_max of eq. (7)
    // Fused cache append (sa_decode_step); null on the plain decode path.
    const uint16_t* Knew;     // [batch][Hkv][D] binary16: the step's new token, written at position seq_lens[b]
    const uint16_t* Vnew;
};

// red_s[w][g] = {M (int bits), l, O[D]} of warp w (NW warps per block) -> the block's partial in the workspace.
template <int D, int GT, int NW = 4>
SA_D void block_combine_and_store(const DecodeArgs& a, float (*red_s)[GT][D + 2], int b, int h0, int split) {
    for (int idx = threadIdx.x; idx < GT * (D + 1); idx += 32 * NW) {
        const int g = idx / (D + 1), c = idx % (D + 1);       // c = 0: l, c >= 1: O[c - 1]
        int Ms = kMNone;
#pragma unroll
        for (int w = 0; w < NW; ++w) Ms = max(Ms, __float_as_int(red_s[w][g][0]));
        float v = 0.0f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const int Mw = __float_as_int(red_s[w][g][0]);
            if (Mw != kMNone) v += red_s[w][g][1 + c] * pow2i_neg(Mw - Ms);
        }
        float* dst = a.partials + (((size_t)split * a.batch + b) * a.Hq + h0 + g) * (D + 2);
        dst[1 + c] = v;
        if (c == 0) dst[0] = __int_as_float(Ms);
    }
}

// Per-warp states (M, l, O) -> one partial per block.  acc[mt] is the 16 x 8 tile (dims x queries)
// of O^T in the accumulator layout of mma.m16n8k8: lane (gq, t4) holds dims 16 mt + 2 gq (c0, c1)
// and 16 mt + 2 gq + 1 (c2, c3) of queries 2 t4 (c0, c2) and 2 t4 + 1 (c1, c3).
template <int D, int GT, int NW>
SA_D void block_merge_and_store(const DecodeArgs& a, float (*red_s)[GT][D + 2], const int (&M)[GT],
                                float (&l)[GT], float (&acc)[D / 16][4], int lane, int warp, int b, int h0,
                                int split) {
    const int gq = lane >> 2, t4 = lane & 3;
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        const float lsum = warp_sum_f32(l[g]);
        if (lane == 0) {
            red_s[warp][g][0] = __int_as_float(M[g]);
            red_s[warp][g][1] = lsum;
        }
    }
#pragma unroll
    for (int mt = 0; mt < D / 16; ++mt) {
        const int dim = 16 * mt + 2 * gq;
        if (2 * t4 < GT) {
            red_s[warp][2 * t4][2 + dim] = acc[mt][0];
            red_s[warp][2 * t4][2 + dim + 1] = acc[mt][2];
        }
        if (2 * t4 + 1 < GT) {
            red_s[warp][2 * t4 + 1][2 + dim] = acc[mt][1];
            red_s[warp][2 * t4 + 1][2 + dim + 1] = acc[mt][3];
        }
    }
    __syncthreads();
    block_combine_and_store<D, GT, NW>(a, red_s, b, h0, split);
}

// One block per (sequence, query head): kMergeGroups groups of D threads each take every
// kMergeGroups-th split (independent, unrolled loads), then the groups are combined in shared
// memory and the result is normalised.
constexpr int kMergeGroups = 8;

// A sequence's length grows by one when the decode kernel appended the step's token itself (the token's
// page must be mapped, exactly the condition the decode kernel used).
struct BumpArgs {
    int32_t* seq_lens;        // null: no fused append
    const int32_t* page_table;
    int max_pages, n_pages, Hq;
};

template <int D>
__global__ void __launch_bounds__(D * kMergeGroups) merge_kernel(const float* __restrict__ partials,
                                                                 float* __restrict__ O, int n_splits, int n_rows,
                                                                 BumpArgs bump) {
    __shared__ int m_s[D * kMergeGroups / 32];
    __shared__ float o_s[kMergeGroups][D + 1];
    pdl_wait();                                               // the partials come from the kernel before
    pdl_launch_dependents();
    const int row = blockIdx.x;                               // b * Hq + h
    if (bump.seq_lens && threadIdx.x == 0 && row % bump.Hq == 0) {
        // every block of the decode kernel has read the old length by now
        const int b = row / bump.Hq, len = bump.seq_lens[b], lp = len / kPageTokens;
        const int pidx = (len >= 0 && lp < bump.max_pages) ? bump.page_table[(size_t)b * bump.max_pages + lp] : -1;
        if (pidx >= 0 && pidx < bump.n_pages) bump.seq_lens[b] = len + 1;
    }
    const int dd = threadIdx.x % D, grp = threadIdx.x / D;
    const size_t stride = (size_t)n_rows * (D + 2);
    const float* base = partials + (size_t)row * (D + 2);
    float l = 0.0f, o = 0.0f;
    constexpr int kHeld = 16;                                 // splits per thread held in registers
    if (n_splits <= kHeld * kMergeGroups) {
        // Common case: every load of this thread is issued before anything waits on one of them (a single
        // round trip to L2), then the maximum of the integer running maxima, then the exact rescale.
        int Mv[kHeld];
        float lv[kHeld], ov[kHeld];
#pragma unroll
        for (int k = 0; k < kHeld; ++k) {
            const int s = grp + k * kMergeGroups;
            const float* p = base + (size_t)(s < n_splits ? s : 0) * stride;
            Mv[k] = (s < n_splits) ? __float_as_int(p[0]) : kMNone;
            lv[k] = p[1];
            ov[k] = p[2 + dd];
        }
        int Ms = kMNone;
#pragma unroll
        for (int k = 0; k < kHeld; ++k) Ms = max(Ms, Mv[k]);
        // the thread's splits are those of its whole group: one value per group is enough
        if (dd == 0) m_s[grp] = Ms;
        __syncthreads();
#pragma unroll
        for (int g = 0; g < kMergeGroups; ++g) Ms = max(Ms, m_s[g]);
#pragma unroll
        for (int k = 0; k < kHeld; ++k) {
            const float f = (Mv[k] == kMNone) ? 0.0f : pow2i_neg(Mv[k] - Ms);
            l += lv[k] * f;
            o += ov[k] * f;
        }
    } else {
        // global maximum of the integer running maxima
        int Ms = kMNone;
        for (int s = threadIdx.x; s < n_splits; s += D * kMergeGroups) Ms = max(Ms, __float_as_int(base[s * stride]));
#pragma unroll
        for (int o2 = 16; o2 > 0; o2 >>= 1) Ms = max(Ms, __shfl_xor_sync(0xffffffffu, Ms, o2));
        if ((threadIdx.x & 31) == 0) m_s[threadIdx.x >> 5] = Ms;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < D * kMergeGroups / 32; ++w) Ms = max(Ms, m_s[w]);
#pragma unroll 8
        for (int s = grp; s < n_splits; s += kMergeGroups) {
            const float* p = base + s * stride;
            const int M = __float_as_int(p[0]);
            const float f = (M == kMNone) ? 0.0f : pow2i_neg(M - Ms);
            l += p[1] * f;
            o += p[2 + dd] * f;
        }
    }
    o_s[grp][dd] = o;
    if (dd == 0) o_s[grp][D] = l;
    __syncthreads();
    if (grp == 0) {
#pragma unroll
        for (int g = 1; g < kMergeGroups; ++g) {
            o += o_s[g][dd];
            l += o_s[g][D];
        }
        // no key at all: zeros; a poisoned partial (a bounded wait gave up) stays visible as NaN
        O[(size_t)row * D + dd] = (l == 0.0f) ? 0.0f : o / l;
    }
}

inline sa_status make_decode_args(const Plan& p, const sa_cache* c, const uint16_t* Q, float* O,
                                  void* workspace, size_t workspace_bytes, DecodeArgs* a, int* gt) {
    if (!c || !c->pages || !c->page_table || !c->seq_lens || !Q || !O) return SA_ERR_INVALID_ARG;
    if (c->batch <= 0 || c->max_pages_per_seq <= 0 || c->n_pages <= 0) return SA_ERR_INVALID_ARG;
    if (c->batch > 65535) return SA_ERR_CAPACITY;
    auto mis = [](const void* ptr, size_t al) { return (reinterpret_cast<uintptr_t>(ptr) & (al - 1)) != 0; };
    if (mis(c->pages, p.lay.align) || mis(c->page_table, 4) || mis(c->seq_lens, 4) || mis(Q, 16) || mis(O, 16))
        return SA_ERR_ALIGNMENT;
    int S, GT;
    split_plan(p, c->batch, c->max_pages_per_seq, &S, &GT);
    const size_t need = (size_t)S * c->batch * p.Hq * (p.d + 2) * sizeof(float);
    if (!workspace || workspace_bytes < need) return SA_ERR_CAPACITY;
    if (mis(workspace, 16)) return SA_ERR_ALIGNMENT;
    a->pages = static_cast<const uint8_t*>(c->pages);
    a->page_table = c->page_table;
    a->seq_lens = c->seq_lens;
    a->Q = Q;
    a->O = O;
    a->partials = static_cast<float*>(workspace);
    a->dbg_scores = nullptr;
    a->dbg_stride = (size_t)c->max_pages_per_seq * kPageTokens;
    a->batch = c->batch;
    a->Hq = p.Hq;
    a->Hkv = p.Hkv;
    a->G = p.G;
    a->max_pages = c->max_pages_per_seq;
    a->n_pages = c->n_pages;
    a->n_splits = S;
    a->f_extra = p.f_extra;
    a->hadamard = p.hadamard ? 1 : 0;
    a->page_bytes = p.lay.page_bytes;
    a->kcode_off = p.lay.kcode_off;
    a->meta_off = p.lay.meta_off;
    a->v_off = p.lay.v_off;
    a->plane_off = p.plane_off;
    a->zscale = 0.0f;
    a->one = 1u;
    a->zr = nullptr;
    a->stat_m = nullptr;
    a->stat_g = nullptr;
    a->n_bits = 0;
    a->k_max = 0;
    a->Knew = nullptr;
    a->Vnew = nullptr;
    *gt = GT;
    return SA_OK;
}

inline sa_status launch_merge(const Plan& p, const DecodeArgs& a, cudaStream_t s) {
    const int rows = a.batch * a.Hq;
    BumpArgs bump{a.Knew ? const_cast<int32_t*>(a.seq_lens) : nullptr, a.page_table, a.max_pages, a.n_pages, a.Hq};
    cudaError_t err;
    if (p.d == 64) err = launch_pdl(merge_kernel<64>, dim3(rows), dim3(64 * kMergeGroups), 0, s,
                                    (const float*)a.partials, a.O, a.n_splits, rows, bump);
    else err = launch_pdl(merge_kernel<128>, dim3(rows), dim3(128 * kMergeGroups), 0, s,
                          (const float*)a.partials, a.O, a.n_splits, rows, bump);
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SA_OK : SA_ERR_CUDA;
}

}  // namespace sa
