// Pieces shared by the quantised and the FP16 decode kernels: kernel arguments, the merge of
// the warps of a block, and the split-K merge (section II-F: the grid has a split
// dimension; the merge rule follows from the integer running maximum of section II-E:
// M* = max_s M_s, every partial is rescaled by the exact factor 2^(M_s - M*)).
#pragma once
#include "sa_common.cuh"
#include "sa_mma.cuh"

namespace sa {

struct DecodeArgs {
    const uint8_t* pages;
    const int32_t* page_table;
    const int32_t* seq_lens;
    const uint16_t* Q;
    float* O;
    float* partials;          // [slot][Hq][D + 2]: {M (int bits), l, O[D]}; slot = split * batch + sequence, or, where
                              // `plan` is set, the block's place among the (sequence, split) pairs of its batch
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
    // Test hook (sa_debug_decode_lost_copy): the copy of this tile of this (sequence, KV head) is never issued.
    int lost_b, lost_kvh, lost_tile;
    // The block waits for the preceding kernels before it reads anything, Q included (set when the kernel before
    // this one writes Q and releases its dependents early: the host-buffer entry's staging kernel).
    int wait_first;
    // Batches of 2 .. kRankedBatchMax sequences (plan_block below): `plan` receives {first slot, splits} of every
    // sequence for the merge kernel; bal_target is the number of (sequence, split) blocks per grid row that a batch
    // of unequal lengths is cut into (0: every sequence keeps n_splits).  Null / 0 elsewhere.
    int32_t* plan;
    int bal_target;
};

// Batches of 2 .. kRankedBatchMax sequences: which (sequence, split) a block of the grid works on is decided on the
// device, from the cached lengths, by every block in the same way.
//   * The sequences are taken longest first (ties by index), so that the blocks of the long sequences are
//     dispatched first and the launch ends on the short ones.
//   * Sequences of equal tile counts keep the host's n_splits each.  Otherwise the grid's x * z blocks of a row are
//     dealt out in proportion to the lengths: the smallest tiles-per-block is searched for which the sequences'
//     split counts, ceil(tiles / tiles-per-block) and at least one each, fit into bal_target blocks (the host's
//     grid, rounded down to whole waves of resident blocks); a sequence's tiles are then cut evenly into its splits.
//     Blocks of about equal work fill the machine whatever the mix of lengths — with the same n_splits for all, the
//     blocks of a batch's longest sequences set the time of the launch while the others' slots idle.
// (Sequences of equal tile counts are simply taken in index order.)
// Block i = z * n_splits + x of a grid row takes the i-th (sequence, split) pair in that order; its partial goes to
// slot i (the kernels recompute i from their grid coordinates), and {first slot, splits} of every sequence is left in `plan` for the merge kernel.  Blocks beyond the last
// pair have nothing to do (b = -1).
// Every block must work from the same lengths, so the plan that counts is made after the wait on the preceding
// kernels; one made before that wait is a guess (lengths read past L1, so that it leaves nothing stale behind).
// `scratch` keeps the guess's lengths and counts: if the lengths read after the wait are the same, the guess stands.
constexpr int kRankedBatchMax = 128;
constexpr int kPlanScratchInts = 3 * kRankedBatchMax + 48;
SA_HD bool batch_is_ranked(int batch) { return batch > 1 && batch <= kRankedBatchMax; }
struct BlockPlan {
    int b, split, n_splits, len;      // sequence (-1: none), which of its n_splits parts, the length the plan was made from
};
// sum of v over the block (every thread gets it); red: 2 x 16 ints, phase alternates between calls
SA_D int plan_block_sum(int v, int* red, int& phase) {
    v = __reduce_add_sync(0xffffffffu, v);
    if ((threadIdx.x & 31) == 0) red[phase * 16 + (threadIdx.x >> 5)] = v;
    __syncthreads();
    int total = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) total += red[phase * 16 + w];
    phase ^= 1;
    return total;
}
// z, x: the block's grid coordinates (z may be falsified by a test hook's guess); recheck: a plan made from `scratch`
// earlier (prev) stands if the lengths have not changed; counts: this is the plan that counts (it is left for the merge)
struct PlanArgs {              // what plan_block reads of the kernel arguments (by value: the call takes no address of them)
    const int32_t* seq_lens;
    int32_t* plan;
    int batch, n_splits, bal_target, max_pages, Knew;
};
SA_D PlanArgs plan_args(const DecodeArgs& a) {
    return PlanArgs{a.seq_lens, a.plan, a.batch, a.n_splits, a.bal_target, a.max_pages, a.Knew ? 1 : 0};
}
SA_D BlockPlan plan_block(PlanArgs a, int z, int x, bool recheck, bool counts, BlockPlan prev, int* scratch) {
    const int B = a.batch, S = a.n_splits, j = threadIdx.x;     // one thread per sequence (a block has >= 128 threads)
    int* len_s = scratch;
    int* cnt_s = scratch + kRankedBatchMax;
    int* pre_s = scratch + 2 * kRankedBatchMax;
    int* red_s = scratch + 3 * kRankedBatchMax;                 // 32 ints
    int* out_s = red_s + 32;                                    // 4 ints
    const bool writer = counts && a.plan != nullptr && z == 0 && x == 0 && blockIdx.y == 0;
    const int len_now = (j < B) ? __ldcg(a.seq_lens + j) : 0;
    if (recheck) {
        // (the scratch is read before the barrier only: once the guess stands, the first copies may land on it)
        const int pre_old = (writer && j < B) ? pre_s[j] : 0, cnt_old = (writer && j < B) ? cnt_s[j] : 0;
        if (!__syncthreads_or((j < B && len_now != len_s[j]) ? 1 : 0)) {
            if (writer && j < B) {
                a.plan[2 * j] = pre_old;
                a.plan[2 * j + 1] = cnt_old;
            }
            return prev;
        }
    }
    if (j < B) len_s[j] = len_now;
    if (j == 0) out_s[0] = -1;
    const int cap = a.max_pages * kPageTokens;
    const int tiles = (j < B) ? (min(max(len_now + (a.Knew ? 1 : 0), 0), cap) + 31) >> 5 : 0;
    __syncthreads();
    const int tiles0 = (min(max(len_s[0] + (a.Knew ? 1 : 0), 0), cap) + 31) >> 5;
    int cnt = S;                                                // splits of sequence j
    const bool uniform = __syncthreads_and((j >= B || tiles == tiles0) ? 1 : 0) != 0;
    if (uniform) {
        // equal tile counts: the blocks are equal whatever the order, so sequence z keeps the grid's own blocks
        if (j < B) {
            cnt_s[j] = S;
            pre_s[j] = j * S;
            if (writer) {
                a.plan[2 * j] = j * S;
                a.plan[2 * j + 1] = S;
            }
        }
        BlockPlan r;
        r.b = z;
        r.split = x;
        r.n_splits = S;
        r.len = len_s[z];
        __syncthreads();                                        // (as at the end of the general case)
        return r;
    }
    if (a.bal_target > 0) {
        int phase = 0;
        const int G = a.bal_target, N = plan_block_sum(tiles, red_s, phase);
        int tpb = max(1, (N + G - 1) / G);
        for (int it = 0; it < 48; ++it) {                       // (the first guess is at most a few per cent short)
            cnt = (j < B) ? max(1, (tiles + tpb - 1) / tpb) : 0;
            const int total = plan_block_sum(cnt, red_s, phase);
            if (total <= G) break;
            tpb = max(tpb + 1, (int)(((long long)tpb * total + G - 1) / G));
            cnt = (j < B) ? S : 0;                              // (if the search ran out: the host's plan, which always fits)
        }
    }
    if (j < B) cnt_s[j] = cnt;
    __syncthreads();
    if (j < B) {
        int pre = 0;                                            // blocks of the sequences ahead of this one
        for (int k = 0; k < B; ++k) {
            const int lk = len_s[k];
            if (lk > len_now || (lk == len_now && k < j)) pre += cnt_s[k];
        }
        pre_s[j] = pre;
        const int i = z * S + x;
        if (i >= pre && i < pre + cnt) {
            out_s[0] = j;
            out_s[1] = i - pre;
            out_s[2] = cnt;
        }
        if (writer) {
            a.plan[2 * j] = pre;
            a.plan[2 * j + 1] = cnt;
        }
    }
    __syncthreads();
    BlockPlan r;
    r.b = out_s[0];
    r.split = out_s[1];
    r.n_splits = out_s[2];
    r.len = r.b >= 0 ? len_s[r.b] : 0;
    __syncthreads();                                            // out_s may be written again by a later call
    return r;
}

// red_s[w][g] = {M (int bits), l, O[D]} of warp w (NW warps per block) -> the block's partial in the workspace
// (used by the kernels whose warps write their states to shared memory themselves).
template <int D, int GT, int NW = 4>
SA_D void block_combine_and_store(const DecodeArgs& a, float (*red_s)[GT][D + 2], int slot, int h0) {
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
        float* dst = a.partials + ((size_t)slot * a.Hq + h0 + g) * (D + 2);
        dst[1 + c] = v;
        if (c == 0) dst[0] = __int_as_float(Ms);
    }
}

// Per-warp states (M, l, O) -> one partial per block, in three steps separated by two block barriers:
// the integer maxima of all warps go to shared memory and one thread per query takes their maximum Mb;
// every warp scales its own state by the exact factor 2^(M - Mb) in registers and writes it out; the
// threads of the block add the warps' rows in a fixed order (deterministic) and store the partial.
// red_s[w][g] = {unused, l, O[D]} of warp w; the maxima live in the first words of the rows:
// red_s[w][g][0] = M of warp w before the first barrier, red_s[0][g][0] = Mb after the second.
// acc[mt] is the 16 x 8 tile (dims x queries) of O^T in the accumulator layout of mma.m16n8k8: lane
// (gq, t4) holds dims 16 mt + 2 gq (c0, c1) and 16 mt + 2 gq + 1 (c2, c3) of queries 2 t4 (c0, c2) and
// 2 t4 + 1 (c1, c3).
template <int D, int GT, int NW>
SA_D void block_merge_and_store(const DecodeArgs& a, float (*red_s)[GT][D + 2], const int (&M)[GT],
                                float (&l)[GT], float (&acc)[D / 16][4], int lane, int warp, int slot, int h0,
                                bool failed = false) {
    const int gq = lane >> 2, t4 = lane & 3;
    float lsum[GT];
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        lsum[g] = warp_sum_f32(l[g]);
        if (lane == 0) red_s[warp][g][0] = __int_as_float(M[g]);
    }
    // A warp whose bounded wait for a copy expired makes the block's whole partial a marked one: l = NaN is
    // written below from a register, not through the scratch rows, which alias the stage buffers — a copy that
    // was merely late could still land in them.
    const bool poisoned = __syncthreads_or(failed ? 1 : 0) != 0;
    if (threadIdx.x < GT) {
        int Mb = kMNone;
#pragma unroll
        for (int w = 0; w < NW; ++w) Mb = max(Mb, __float_as_int(red_s[w][threadIdx.x][0]));
        red_s[0][threadIdx.x][0] = __int_as_float(Mb);       // (only this thread reads that column before the barrier)
    }
    __syncthreads();
    // a warp that saw no key (M = "none") has l = 0 and O = 0; its factor is 0 or, if no warp saw one, 1
    float f[GT];
#pragma unroll
    for (int g = 0; g < GT; ++g) f[g] = pow2i_neg(M[g] - __float_as_int(red_s[0][g][0]));
    float f0 = 0.0f, f1 = 0.0f;                              // factors of this lane's queries 2 t4, 2 t4 + 1
#pragma unroll
    for (int g = 0; g < GT; ++g)
        if (t4 == g / 2) {
            if (g & 1) f1 = f[g];
            else f0 = f[g];
        }
    if (lane == 0) {
#pragma unroll
        for (int g = 0; g < GT; ++g) red_s[warp][g][1] = lsum[g] * f[g];
    }
#pragma unroll
    for (int mt = 0; mt < D / 16; ++mt) {
        const int dim = 16 * mt + 2 * gq;
        if (2 * t4 < GT) {
            red_s[warp][2 * t4][2 + dim] = acc[mt][0] * f0;
            red_s[warp][2 * t4][2 + dim + 1] = acc[mt][2] * f0;
        }
        if (2 * t4 + 1 < GT) {
            red_s[warp][2 * t4 + 1][2 + dim] = acc[mt][1] * f1;
            red_s[warp][2 * t4 + 1][2 + dim + 1] = acc[mt][3] * f1;
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < GT * (D + 2); idx += 32 * NW) {
        const int g = idx / (D + 2), c = idx % (D + 2);       // c = 0: M, 1: l, c >= 2: O[c - 2]
        float v = red_s[0][g][c];
        if (c != 0) {
#pragma unroll
            for (int w = 1; w < NW; ++w) v += red_s[w][g][c];
        }
        if (poisoned && c <= 1) v = (c == 0) ? __int_as_float(0) : __int_as_float(0x7fc00000);   // M = 0, l = NaN
        a.partials[((size_t)slot * a.Hq + h0 + g) * (D + 2) + c] = v;
    }
}

// Split-K merge.  One block of 128 threads per (sequence, query head, 16 output dims): 4 lanes of four
// dims times 32 groups of splits; a thread's loads (three splits at a time) are all in flight
// together, so up to 96 splits cost one round trip to L2.  Each thread merges its splits with a local
// maximum, the block takes the maximum M* of those, every thread rescales its sum by the exact
// 2^(M_local - M*), and the groups are added in a fixed order, in two levels (deterministic).  The block is kept this
// small — 128 threads, at most 32 registers, 2.7 KB of shared memory — so that it fits on an SM beside
// two resident blocks of the decode kernel: the next decode kernel is launched while this one runs
// (programmatic dependent launch), and a merge block that took the place of one of its blocks would make
// that block, and with it the whole grid, finish late.
// With more than 96 splits (the FP16 kernel at batch 1: 111) the block has 256 threads = 64 groups instead, so that
// the partials are still fetched in one round trip; it then no longer fits beside the quantised kernels' two blocks,
// whose split counts stay below that.
constexpr int kMergeDims = 16;                                // output dims per block
constexpr int kMergeLanes = kMergeDims / 4;                   // float4 lanes
constexpr int kMergeChunk = 3;                                // splits per thread whose loads are in flight together
constexpr int kMergeSmallSplits = (128 / kMergeLanes) * kMergeChunk;   // most splits a 128-thread block takes in one pass

// A sequence's length grows by one when the decode kernel appended the step's token itself (the token's
// page must be mapped, exactly the condition the decode kernel used).
struct BumpArgs {
    int32_t* seq_lens;        // null: no fused append
    const int32_t* page_table;
    int max_pages, n_pages, Hq;
    int early_release;        // release the dependents of the merge kernel before its own wait (see merge_kernel)
    const int32_t* plan;      // {first slot, splits} per sequence (plan_block), or null: slots split * batch + sequence
};

template <int D, int kMergeThreads>
__global__ void __launch_bounds__(kMergeThreads, 2048 / kMergeThreads) merge_kernel(const float* __restrict__ partials,
                                                                                    float* __restrict__ O, int n_splits,
                                                                                    int n_rows, BumpArgs bump) {
    constexpr int kMergeGroups = kMergeThreads / kMergeLanes;     // groups of splits
    __shared__ int mw_s[kMergeThreads / 32];
    __shared__ float4 o_s[kMergeGroups][kMergeLanes];
    __shared__ float l_s[kMergeGroups];
    // With early_release the kernel after this one may be scheduled at once — while the decode kernel whose
    // partials this block is about to wait for is still running — so that its blocks move in as that kernel's
    // blocks retire and are already waiting when this one completes.  That is safe because every kernel of this
    // library reads, ahead of its own wait, nothing that this kernel or its predecessors write (the decode kernels:
    // only Q and hints).  It pays for the ten-warp decode kernels at batch 1 (3–6 % of a step); with the four-warp
    // kernels (PoT-M1 / M2, d = 128, FP16) the early arrivals slow the running kernel down by more than they gain.
    if (bump.early_release) pdl_launch_dependents();
    pdl_wait();                                               // the partials come from the kernel before
    if (!bump.early_release) pdl_launch_dependents();
    const int row = blockIdx.x / (D / kMergeDims);            // b * Hq + h
    const int part = blockIdx.x % (D / kMergeDims);           // which 16 dims
    if (bump.seq_lens && threadIdx.x == 0 && part == 0 && row % bump.Hq == 0) {
        // every block of the decode kernel has read the old length by now
        const int b = row / bump.Hq, len = bump.seq_lens[b], lp = len / kPageTokens;
        const int pidx = (len >= 0 && lp < bump.max_pages) ? bump.page_table[(size_t)b * bump.max_pages + lp] : -1;
        if (pidx >= 0 && pidx < bump.n_pages) bump.seq_lens[b] = len + 1;
    }
    size_t stride = (size_t)n_rows * (D + 2);
    const int ln = threadIdx.x % kMergeLanes, grp = threadIdx.x / kMergeLanes;
    const float* base = partials + (size_t)row * (D + 2);
    if (bump.plan) {                                          // the sequence's splits sit in consecutive slots
        const int b = row / bump.Hq;
        const int first = bump.plan[2 * b];
        n_splits = bump.plan[2 * b + 1];
        stride = (size_t)bump.Hq * (D + 2);
        base = partials + ((size_t)first * bump.Hq + row % bump.Hq) * (D + 2);
    }
    const float* obase = base + 2 + part * kMergeDims + ln * 4;
    int Ml = kMNone;                                          // this thread's splits: grp, grp + 32, ...
    float l = 0.0f;
    float4 o = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    for (int s0 = grp; s0 < n_splits; s0 += kMergeGroups * kMergeChunk) {
        float2 ml[kMergeChunk], v0[kMergeChunk], v1[kMergeChunk];
#pragma unroll
        for (int k = 0; k < kMergeChunk; ++k) {
            const int s = s0 + k * kMergeGroups;
            const size_t off = (size_t)(s < n_splits ? s : s0) * stride;
            ml[k] = *reinterpret_cast<const float2*>(base + off);
            v0[k] = reinterpret_cast<const float2*>(obase + off)[0];
            v1[k] = reinterpret_cast<const float2*>(obase + off)[1];
            if (s >= n_splits) ml[k].x = __int_as_float(kMNone);
        }
        int Mn = Ml;
#pragma unroll
        for (int k = 0; k < kMergeChunk; ++k) Mn = max(Mn, __float_as_int(ml[k].x));
        const float fo = pow2i_neg(Ml - Mn);                  // 1 if nothing changed; 0 on the first chunk (l and o are 0 then)
        l *= fo;
        o.x *= fo;
        o.y *= fo;
        o.z *= fo;
        o.w *= fo;
        Ml = Mn;
#pragma unroll
        for (int k = 0; k < kMergeChunk; ++k) {
            const int M = __float_as_int(ml[k].x);
            const float f = (M == kMNone) ? 0.0f : pow2i_neg(M - Mn);     // a split that saw no key carries zeros
            l += ml[k].y * f;
            o.x += v0[k].x * f;
            o.y += v0[k].y * f;
            o.z += v1[k].x * f;
            o.w += v1[k].y * f;
        }
    }
    int Ms = warp_max_s32(Ml);
    if ((threadIdx.x & 31) == 0) mw_s[threadIdx.x >> 5] = Ms;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kMergeThreads / 32; ++w) Ms = max(Ms, mw_s[w]);
    const float f = (Ml == kMNone) ? 0.0f : pow2i_neg(Ml - Ms);
    o_s[grp][ln] = make_float4(o.x * f, o.y * f, o.z * f, o.w * f);
    if (ln == 0) l_s[grp] = l * f;
    __syncthreads();
    // the groups are added in a fixed order, in two levels (eight groups per thread, then the eighths): the result
    // does not depend on the timing of anything
    constexpr int kFan = 8;
    if (grp < kMergeGroups / kFan) {
        o = o_s[grp * kFan][ln];
        l = l_s[grp * kFan];
#pragma unroll
        for (int g = 1; g < kFan; ++g) {
            const float4 t = o_s[grp * kFan + g][ln];
            o.x += t.x;
            o.y += t.y;
            o.z += t.z;
            o.w += t.w;
            l += l_s[grp * kFan + g];
        }
    }
    __syncthreads();                                          // every first-level read is done: the rows can be overwritten
    if (grp < kMergeGroups / kFan) {
        o_s[grp][ln] = o;
        if (ln == 0) l_s[grp] = l;
    }
    __syncthreads();
    if (grp == 0) {
        o = o_s[0][ln];
        l = l_s[0];
#pragma unroll
        for (int g = 1; g < kMergeGroups / kFan; ++g) {
            const float4 t = o_s[g][ln];
            o.x += t.x;
            o.y += t.y;
            o.z += t.z;
            o.w += t.w;
            l += l_s[g];
        }
        // no key at all: zeros; a poisoned partial (a bounded wait gave up) stays visible as NaN
        const float inv = 1.0f / l;
        float4 r = make_float4(o.x * inv, o.y * inv, o.z * inv, o.w * inv);
        if (l == 0.0f) r = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        *reinterpret_cast<float4*>(O + (size_t)row * D + part * kMergeDims + ln * 4) = r;
    }
}

sa_status decode_step_impl(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q, const uint16_t* K_new,
                           const uint16_t* V_new, float* O, void* workspace, size_t workspace_bytes, sa_stream stream,
                           bool q_after_wait);

// Bytes of the split-K workspace: the partials and, for the batches whose blocks are planned on the device, the plan.
inline size_t decode_workspace_bytes(const Plan& p, int batch, int S, bool with_plan = true) {
    const size_t partials = (size_t)S * batch * p.Hq * (p.d + 2) * sizeof(float);
    return partials + ((with_plan && batch_is_ranked(batch)) ? (((size_t)batch * 8 + 15) & ~(size_t)15) : 0);
}

// with_plan = false: the caller's kernels index the partials by (split, sequence) themselves (the shift-based A.V option)
inline sa_status make_decode_args(const Plan& p, const sa_cache* c, const uint16_t* Q, float* O,
                                  void* workspace, size_t workspace_bytes, DecodeArgs* a, int* gt, bool with_plan = true) {
    if (!c || !c->pages || !c->page_table || !c->seq_lens || !Q || !O) return SA_ERR_INVALID_ARG;
    if (c->batch <= 0 || c->max_pages_per_seq <= 0 || c->n_pages <= 0) return SA_ERR_INVALID_ARG;
    if (c->batch > 65535) return SA_ERR_CAPACITY;
    auto mis = [](const void* ptr, size_t al) { return (reinterpret_cast<uintptr_t>(ptr) & (al - 1)) != 0; };
    if (mis(c->pages, p.lay.align) || mis(c->page_table, 4) || mis(c->seq_lens, 4) || mis(Q, 16) || mis(O, 16))
        return SA_ERR_ALIGNMENT;
    int S, GT;
    split_plan(p, c->batch, c->max_pages_per_seq, &S, &GT);
    // the kernels place the splits with 32-bit arithmetic: tiles * (splits + 1) must stay below 2^31
    if ((long long)c->max_pages_per_seq * (kPageTokens / kTileTokens) * (S + 1) >= (1LL << 31)) return SA_ERR_CAPACITY;
    const size_t need = decode_workspace_bytes(p, c->batch, S, with_plan);
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
    a->lost_b = a->lost_kvh = a->lost_tile = -1;
    a->wait_first = 0;
    a->plan = nullptr;
    a->bal_target = 0;
    if (with_plan && batch_is_ranked(c->batch)) {
        a->plan = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + (size_t)S * c->batch * p.Hq * (p.d + 2) * sizeof(float));
        // blocks per grid row that a batch of unequal lengths is cut into: the grid, rounded down to whole waves of
        // resident blocks (equal blocks gain nothing from a last, partly filled wave)
        const KernelShape shape = p.fp16 ? kFp16Shape : decode_shape(p.d, p.int8 ? 8 : p.k);
        const long long rows = (long long)p.Hkv * (p.G / GT), slots = (long long)sm_count() * shape.blocks_per_sm;
        long long per_row = (long long)S * c->batch;
        if (per_row * rows > slots) per_row = ((per_row * rows) / slots) * slots / rows;
        a->bal_target = (int)(per_row < c->batch ? c->batch : per_row);
    }
    *gt = GT;
    return SA_OK;
}

inline sa_status launch_merge(const Plan& p, const DecodeArgs& a, cudaStream_t s) {
    const int rows = a.batch * a.Hq;
    const int early = (!p.fp16 && decode_shape(p.d, p.int8 ? 8 : p.k).warps >= 8) ? 1 : 0;
    BumpArgs bump{a.Knew ? const_cast<int32_t*>(a.seq_lens) : nullptr, a.page_table, a.max_pages, a.n_pages, a.Hq, early, a.plan};
    cudaError_t err;
    const bool small = a.n_splits <= kMergeSmallSplits;
    const dim3 grid(rows * (p.d / kMergeDims));
    const float* part = a.partials;
    if (p.d == 64) err = small ? launch_pdl(merge_kernel<64, 128>, grid, dim3(128), 0, s, part, a.O, a.n_splits, rows, bump)
                               : launch_pdl(merge_kernel<64, 256>, grid, dim3(256), 0, s, part, a.O, a.n_splits, rows, bump);
    else err = small ? launch_pdl(merge_kernel<128, 128>, grid, dim3(128), 0, s, part, a.O, a.n_splits, rows, bump)
                     : launch_pdl(merge_kernel<128, 256>, grid, dim3(256), 0, s, part, a.O, a.n_splits, rows, bump);
    return (err == cudaSuccess && cudaGetLastError() == cudaSuccess) ? SA_OK : SA_ERR_CUDA;
}

}  // namespace sa
