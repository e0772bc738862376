// The decode kernel template and its launcher; included by the translation units that instantiate it
// (sa_decode_k*.cu, one per key code so that they compile in parallel).
#pragma once
// Decode attention over the power-of-two key cache: the hot path.
//
// Grid (split, KV head x query chunk, sequence); 4, 8 or 10 warps per block (decode_shape).  A block
// quantises its GT query heads into shared memory (ahead of its wait on the preceding kernel),
// then each of its warps walks its own 32-key tiles of the block's slice of the key axis with a
// private online-softmax state, so the main loop has no block-wide barrier.  Per tile: lane = key
// for the integer scores (section II-B eq. (3) with the mantissa code of eq. (5)), warp-wide maxima
// and an integer running maximum in the log2 domain (section II-E); then the floating-point A.V
// over the INT8 values as small tensor-core products
// O^T[dims][queries] += V^T[dims][keys] P^T[keys][queries] (mma.m16n8k8, tf32 operands: the INT8
// values are exact, every weight is split into two tf32 terms, accumulation in FP32).  The warps'
// states and then the blocks' partial results are merged with exact power-of-two factors.
// For sa_decode_step the warp that owns the new token's tile writes the token first (section II-F).
//
// Compile-time switches for ablation measurements only (section V-F of the paper lists the three design choices;
// each switch removes one of them from every instantiation, `python -m paper_2609_09208_b200.build -DNAME`):
//   SA_ABLATE_WORD_STAGING   a warp stages its tile itself with 32-bit loads and stores instead of one 16-byte
//                            aligned bulk-async copy, and reads the key codes back 32 bits at a time instead of 128
//   SA_ABLATE_SIGNED_SHIFT   the mantissa codes' shift without head-room: a signed amount (here F = 3 instead of
//                            6 + k), the direction decided per term — a right shift drops bits, so the scores of
//                            such a build are NOT the exact ones and its tests fail by design
//   SA_ABLATE_NO_MIN_BLOCKS  __launch_bounds__ without the resident-blocks clause (the register cap)
#include "sa_common.cuh"
#include "sa_cache_write.cuh"
#include "sa_datapath.cuh"
#include "sa_decode_common.cuh"
#include "sa_mma.cuh"
#include "sa_quant.cuh"
#include "sa_stage.cuh"

namespace sa {

// Shared-memory plan of one block (dynamic shared memory, 1024-byte aligned):
//   [NW warps x NS stage buffers][mbarriers][packed queries or table][query scales]; the
//   block-merge scratch re-uses the stage buffers once every warp has left its tile loop.
template <int D, int KB, bool NIB, int GT>
struct DecodeSmem {
    static constexpr int NP = (GT + 1) / 2;        // query pairs
    static constexpr bool kTable = (KB == 1 || KB == 2 || KB == 4);   // mantissa codes: table datapath
    static constexpr int NW = decode_shape(D, KB).warps;
    static constexpr int CH = NIB ? D / 32 : D / 16;
    static constexpr int PLANES = (NIB && kTable) ? KB : 0;           // dense planar container: mantissa bit planes
    using Stage = TileStage<CH, true, D, PLANES, D / 8>;
    // Stage buffers per warp: two (the next tile is in flight while this one is computed), except where a
    // second buffer would cost resident warps — d = 128 (a tile is 8 KB) and PoT-M4 (32 KB table): there one,
    // and the other warps of the SM cover the copy instead.
    static constexpr int NS = (D == 128 || KB == 4) ? 1 : kStages;
    static constexpr int kStageOff = 0;
    static constexpr int kMbarOff = NW * NS * Stage::kBytes;
    // PoT-4: the shifted packed query pairs [D][8][NP]; INT8: D/4 x GT words of four queries; mantissa
    // codes: the table of query multiples [D][NP][2^KB] x 8 bytes
    static constexpr int kQpOff = (kMbarOff + 256 + 255) & ~255;   // the table datapaths want 256-byte alignment
    // (the prologue's scratch for the unpacked queries, D x GT words, uses the same space first)
    static constexpr int kQpData = kTable ? D * NP * (8 << KB) : KB == 0 ? D * 8 * NP * 4 : D * NP * 4;
    static constexpr int kQpBytes = kQpData > D * GT * 4 ? kQpData : D * GT * 4;
    static constexpr int kQscaleOff = kQpOff + kQpBytes;
    // (The softmax weights of a tile need no space of their own: they overwrite the tile's key
    // codes in the stage buffer, which are dead by then.)
    static constexpr int kBytes = kQscaleOff + 128;
    static constexpr int kBlocksPerSM = decode_shape(D, KB).blocks_per_sm;
    static_assert(NW * GT * (D + 2) * 4 <= NW * NS * Stage::kBytes && NW * NS * 8 <= 256, "merge scratch must fit in the stage buffers");
    static_assert(Stage::kCodeBytes >= 32 * 8 * 4, "the weights of a tile must fit in its code area");
    static_assert(NW * NS * Stage::kBytes >= kPlanScratchInts * 4, "the block plan's scratch must fit in the stage buffers");
    static_assert(Stage::kBytes == half_block_bytes(D, KB, NIB), "a stage buffer is a verbatim copy of half a page block");
};

template <int D, int KB, bool NIB, int GT, int MODE = 0>
#ifdef SA_ABLATE_NO_MIN_BLOCKS
__global__ void __launch_bounds__((32 * DecodeSmem<D, KB, NIB, GT>::NW)) decode_kernel(DecodeArgs a) {
#else
__global__ void __launch_bounds__((32 * DecodeSmem<D, KB, NIB, GT>::NW), (DecodeSmem<D, KB, NIB, GT>::kBlocksPerSM)) decode_kernel(DecodeArgs a) {
#endif
    // MODE 0: the decode kernel; 1: the same with SA_FLAG_SHIFT_BY_MULTIPLY; 2: the score pass of the shift-based
    // A.V option (a.zr set: rounded logits and statistics instead of softmax and A.V), kept out of the other two
    // 3: the same with SA_FLAG_ADD_ON_ALU; 4: the test hook that never issues one chosen tile's copy (sa_debug_decode_lost_copy)
    constexpr bool MUL = (MODE == 1), SP = (MODE == 2), ALUO = (MODE == 3), LOST = (MODE == 4);
    constexpr uint32_t kPolls = LOST ? (1u << 10) : kWaitLimit;
    // KB = 0: PoT-4 (packed shift datapath); KB = 1, 2, 4: mantissa codes (table datapath);
    // KB = 8: uniform INT8 comparison code (dp4a).  MUL: the shifts run on the integer multiplier
    // (SA_FLAG_SHIFT_BY_MULTIPLY; same scores, reported separately from the shift kernels).
    using SM = DecodeSmem<D, KB, NIB, GT>;
    using Stage = typename SM::Stage;
    constexpr int EPL = D / 32;
    constexpr int NP = SM::NP;
    constexpr int NW = SM::NW, NT = 32 * NW;       // warps and threads per block
    constexpr int NS = SM::NS;                     // stage buffers per warp
    constexpr int WORDS = NIB ? D / 8 : D / 4;     // 32-bit code words per key
    constexpr int MT = D / 16;                     // 16-dim row tiles of O^T in the A.V phase
    extern __shared__ __align__(1024) uint8_t smem[];
    float* qscale_s = reinterpret_cast<float*>(smem + SM::kQscaleOff);
    int32_t (*q_s)[GT] = reinterpret_cast<int32_t (*)[GT]>(smem + SM::kQpOff);     // prologue only
    float (*red_s)[GT][D + 2] = reinterpret_cast<float (*)[GT][D + 2]>(smem + SM::kStageOff);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chunks = a.G / GT;
    const int kvh = blockIdx.y / chunks;
    const int h0 = kvh * a.G + (blockIdx.y % chunks) * GT;     // first query head of this block
    // What this block works on: sequence z and split x of the host's n_splits, or (batches of 2 .. 128 sequences)
    // what plan_block deals it from the cached lengths.  The plan made here, from lengths the preceding kernel may be
    // about to change, is a guess that lets the query prologue run ahead of the dependency wait; the plan made after
    // the wait decides, and the prologue is repeated in the rare case that it names another sequence (a step adds
    // one token to every sequence, which keeps their order).  The test-hook instantiation guesses wrong on purpose, so
    // that its tests walk the repeat.
    const bool ranked = batch_is_ranked(a.batch);
    int* plan_scratch = reinterpret_cast<int*>(smem + SM::kStageOff);
    BlockPlan bp{(int)blockIdx.z, (int)blockIdx.x, a.n_splits, 0};
    if (a.wait_first) pdl_wait();
    if (__builtin_expect(ranked, 0))
        bp = plan_block(plan_args(a), LOST ? (blockIdx.z + 1) % a.batch : blockIdx.z, blockIdx.x, false, a.wait_first != 0, bp, plan_scratch);
    int b = bp.b;
    const uint32_t mbar0 = smem_addr(smem + SM::kMbarOff) + warp * NS * 8;
    const uint32_t stage0 = smem_addr(smem + SM::kStageOff) + warp * NS * Stage::kBytes;
    const uint8_t* stage_ptr0 = smem + SM::kStageOff + warp * NS * Stage::kBytes;

    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < NS; ++s) mbar_init(mbar0 + s * 8, 1u);
        fence_mbar_init();
        fence_proxy_async();
    }
    __syncwarp();
    pdl_launch_dependents();    // the split-K merge may be scheduled as soon as blocks of this grid retire
    // A guess at the warps' first tiles, from a length the preceding kernel may be about to change, only to ask
    // L2 for those tiles while that kernel drains (loads that bypass L1, so nothing stale can be read back later).
    // The length is fetched here, so that its latency hides behind the query quantisation; the dependent
    // page-table reads and the hints themselves are left to the last warp, after the prologue's last barrier,
    // so that no other warp waits for them.
    int len_g, tile_g, pidx_g;
    bool again;
#pragma unroll 1
    do {
        len_g = 0, tile_g = -1, pidx_g = -1;
        const int split_g = bp.split, nsp_g = bp.n_splits;         // what the hints below are computed for
        const int bq = b < 0 ? 0 : b;                              // (a block without work so far prepares sequence 0)
        if (ranked) len_g = bp.len;
        else if (lane == 0 || warp == NW - 1) len_g = __ldcg(a.seq_lens + bq);

        // ---- prologue: quantise the GT query heads (eq. (2)) and pack them two per register.  It reads
        // only Q, which no kernel of a decode step writes, so it runs BEFORE the wait on the preceding
        // kernel (the cache append) and overlaps it. ----
        for (int g = warp; g < GT; g += NW) {
            uint32_t bits[EPL];
            load_vec_bits<EPL>(a.Q + ((size_t)bq * a.Hq + h0 + g) * D, lane, bits);
            int q[EPL];
            const float delta = quantise_query_vec<EPL>(bits, lane, a.hadamard != 0, q);
#pragma unroll
            for (int i = 0; i < EPL; ++i) q_s[lane * EPL + i][g] = q[i];
            if (lane == 0) qscale_s[g] = delta * a.zscale;        // Delta * 2^-F * log2(e) / sqrt(d)
        }
        __syncthreads();
        if (lane == 0) {
            const int n_tiles_g = (min(max(len_g + (a.Knew ? 1 : 0), 0), a.max_pages * kPageTokens) + 31) >> 5;
            const int t_g = split_begin(n_tiles_g, bp.split, bp.n_splits) + warp;
            if (t_g < split_begin(n_tiles_g, (bp.split + 1), bp.n_splits)) tile_g = t_g;
        }
        if constexpr (SM::kTable) {
            // table of query multiples, built by repeated addition: row (m, pair) = {q_lo, q_hi} * (2^KB + mu)
            using TS = TableScore<KB, NP>;
            uint8_t* tab = smem + SM::kQpOff;
            // One thread per row (element, query pair) and pass; it walks the row's 2^KB entries by
            // repeated addition of the pair, starting at an entry that depends on its lane so that the
            // lanes of a half-warp always write different banks, and wraps around once.
            constexpr int ROWS = D * NP;
            constexpr int PASSES = (ROWS + NT - 1) / NT;
            constexpr uint32_t MASK = (1u << KB) - 1u;
            int qlo[PASSES], qhi[PASSES];
#pragma unroll
            for (int k = 0; k < PASSES; ++k) {
                const int row = threadIdx.x + k * NT;              // = m * NP + p
                const int m = row / NP, p = row % NP;
                qlo[k] = (row < ROWS) ? q_s[m][2 * p] : 0;
                qhi[k] = (row < ROWS && 2 * p + 1 < GT) ? q_s[m][2 * p + 1] : 0;
            }
            __syncthreads();                                       // q_s is about to be overwritten
            const uint32_t mu0 = ((uint32_t)lane >> (4 - KB)) & MASK;
#pragma unroll
            for (int k = 0; k < PASSES; ++k) {
                const int row = threadIdx.x + k * NT;
                if (row < ROWS) {
                    uint2* dst = reinterpret_cast<uint2*>(tab + (size_t)row * TS::kRowBytes);
                    const uint32_t lo = (uint32_t)qlo[k], hi = (uint32_t)qhi[k];
                    uint32_t x = lo << KB, y = hi << KB;           // entry mu0: (2^KB + mu0) times the pair, by shift-and-add
#pragma unroll
                    for (int bit = 0; bit < KB; ++bit)
                        if (mu0 & (1u << bit)) { x += lo << bit; y += hi << bit; }
#pragma unroll
                    for (uint32_t st = 0; st <= MASK; ++st) {
                        const uint32_t mu = (mu0 + st) & MASK;
                        if (mu == 0u) { x = lo << KB; y = hi << KB; }
                        dst[mu] = make_uint2(x, y);
                        x += lo;
                        y += hi;
                    }
                }
            }
        } else if constexpr (KB != 8) {
            uint32_t qp_reg[(D * NP + NT - 1) / NT];
#pragma unroll
            for (int k = 0; k < (D * NP + NT - 1) / NT; ++k) {
                const int idx = threadIdx.x + k * NT;
                const int m = idx / NP, p = idx % NP;
                qp_reg[k] = (idx < D * NP) ? pack_pair(q_s[m][2 * p], (2 * p + 1 < GT) ? q_s[m][2 * p + 1] : 0) : 0u;
            }
            __syncthreads();                                       // q_s is about to be overwritten
            // S[m][g][pair] = the packed pair shifted by g - 1 (0 for g = 0); the entries of one pair are written
            // starting at a g that depends on the element, so that the lanes of a warp use different banks
            uint32_t* tab = reinterpret_cast<uint32_t*>(smem + SM::kQpOff);
#pragma unroll
            for (int k = 0; k < (D * NP + NT - 1) / NT; ++k) {
                const int idx = threadIdx.x + k * NT;
                const int m = idx / NP, p = idx % NP;
                if (idx < D * NP) {
#pragma unroll
                    for (int st = 0; st < 8; ++st) {
                        const int g = (st + m) & 7;
                        tab[(m * 8 + g) * NP + p] = ShiftTable<NP>::entry(qp_reg[k], g);
                    }
                }
            }
        } else {
            // four consecutive elements of one query per word, in the byte order of the key words
            uint32_t* q4_s = reinterpret_cast<uint32_t*>(smem + SM::kQpOff);
            uint32_t q4_reg[(D / 4 * GT + NT - 1) / NT];
#pragma unroll
            for (int k = 0; k < (D / 4 * GT + NT - 1) / NT; ++k) {
                const int idx = threadIdx.x + k * NT;
                const int w = idx / GT, g = idx % GT;
                q4_reg[k] = 0u;
                if (idx < D / 4 * GT)
                    q4_reg[k] = (uint32_t)(q_s[4 * w][g] & 0xff) | ((uint32_t)(q_s[4 * w + 1][g] & 0xff) << 8) |
                                ((uint32_t)(q_s[4 * w + 2][g] & 0xff) << 16) | ((uint32_t)(q_s[4 * w + 3][g] & 0xff) << 24);
            }
            __syncthreads();                                       // q_s is about to be overwritten
#pragma unroll
            for (int k = 0; k < (D / 4 * GT + NT - 1) / NT; ++k) {
                const int idx = threadIdx.x + k * NT;
                if (idx < D / 4 * GT) q4_s[idx] = q4_reg[k];
            }
        }
        __syncthreads();

        if (warp == NW - 1 && lane < NW) {                        // lane w: the first tile of warp w
            const int n_tiles_g = (min(max(len_g + (a.Knew ? 1 : 0), 0), a.max_pages * kPageTokens) + 31) >> 5;
            const int t_g = split_begin(n_tiles_g, bp.split, bp.n_splits) + lane;
            if (t_g < split_begin(n_tiles_g, (bp.split + 1), bp.n_splits)) {
                const int p_g = __ldcg(a.page_table + (size_t)bq * a.max_pages + (t_g >> 1));
                if (p_g >= 0 && p_g < a.n_pages)
                    Stage::prefetch(a.pages + ((size_t)p_g * a.Hkv + kvh) * a.page_bytes, (t_g & 1) * 32, !SP);
            }
        }
        pdl_wait();                 // everything below reads what the preceding kernels in the stream wrote (the cache)
        // the page of the guessed first tile, read again now that it is valid, at the same time as the length(s)
        // (one round trip instead of two when the guess holds, which it does unless the length crossed a tile boundary)
        if (lane == 0 && tile_g >= 0) pidx_g = a.page_table[(size_t)bq * a.max_pages + (tile_g >> 1)];
        again = false;
        if (__builtin_expect(ranked && !a.wait_first, 0)) {       // the plan that counts; wait_first made it after the wait already
            // (the test hook's guess was made for another block's coordinates: it never stands)
            bp = plan_block(plan_args(a), blockIdx.z, blockIdx.x, !LOST, true, bp, plan_scratch);
            again = bp.b != bq && bp.b >= 0;
            if (bp.split != split_g || bp.n_splits != nsp_g) tile_g = -1;     // the hint was for other tiles
            b = bp.b;
        }
    } while (again);
    if (ranked && b < 0) return;                                  // more blocks than (sequence, split) pairs
    const int split = bp.split, n_splits = bp.n_splits;

    // ---- this warp's tiles; start the first copies ----
    int len = ranked ? bp.len : a.seq_lens[b];
    int tile_new = -1, pidx_new = -1;
    if (a.Knew) {
        // Fused append: the step's new token goes to position len (if its page is mapped) and is part of
        // this step's attention.  Every block takes the same decision; the split-K merge kernel bumps
        // seq_lens once all blocks have read it.
        const int lp = len / kPageTokens;
        pidx_new = (len >= 0 && lp < a.max_pages) ? a.page_table[(size_t)b * a.max_pages + lp] : -1;
        if (pidx_new >= 0 && pidx_new < a.n_pages) {
            tile_new = len >> 5;
            len += 1;
        }
    }
    const int n_tiles = (min(len, a.max_pages * kPageTokens) + 31) >> 5;
    const int tile0 = split_begin(n_tiles, split, n_splits);
    const int tile1 = split_begin(n_tiles, (split + 1), n_splits);
    const int first = tile0 + warp;
    const int n_my = first < tile1 ? (tile1 - first + NW - 1) / NW : 0;
    if (tile_new >= first && tile_new < tile1 && (tile_new - first) % NW == 0) {      // warp-uniform: this warp owns that tile
        // encode / quantise the token and write it into its page before the tile is copied to shared memory
        constexpr int WMODE = (KB == 8) ? 32 : (NIB ? 8 + KB : KB);
        CacheArgs ca{};
        ca.page_bytes = a.page_bytes;
        ca.kcode_off = a.kcode_off;
        ca.meta_off = a.meta_off;
        ca.v_off = a.v_off;
        ca.plane_off = a.plane_off;
        ca.hadamard = a.hadamard;
        uint8_t* block = const_cast<uint8_t*>(a.pages) + ((size_t)pidx_new * a.Hkv + kvh) * a.page_bytes;
        const size_t row = ((size_t)b * a.Hkv + kvh) * D;
        write_token<D, WMODE>(block, ca, (len - 1) % kPageTokens, lane, a.Knew + row, a.Vnew + row);
        fence_proxy_async_global();
        __syncwarp();
    }
    // Lane 0: start the copies of my i-th tile into stage i % NS.  A tile whose page is not
    // mapped gets a plain arrival instead (the phase completes, the tile is skipped below).
#ifndef SA_ABLATE_WORD_STAGING
    auto issue = [&](int i) {
        const int tile = first + NW * i;
        const int pidx = (tile == tile_g) ? pidx_g : a.page_table[(size_t)b * a.max_pages + (tile >> 1)];
        const int s = i % NS;
        if (LOST && tile == a.lost_tile && b == a.lost_b && kvh == a.lost_kvh) return;   // test hook: this copy never starts
        if (pidx < 0 || pidx >= a.n_pages) {
            mbar_arrive(mbar0 + s * 8);
        } else {
            const uint8_t* block = a.pages + ((size_t)pidx * a.Hkv + kvh) * a.page_bytes;
            Stage::issue(stage0 + s * Stage::kBytes, block, (tile & 1) * 32, mbar0 + s * 8, true,
                         !SP);                                    // the score pass of the shift-A.V option needs no values
        }
    };
    if (lane == 0)
        for (int i = 0; i < NS && i < n_my; ++i) issue(i);
#else
    // ablation: the whole warp copies the tile word by word; lane 0 then completes the stage's barrier phase
    auto issue = [&](int i) {
        const int tile = first + NW * i;
        const int pidx = a.page_table[(size_t)b * a.max_pages + (tile >> 1)];
        const int s = i % NS;
        if (pidx >= 0 && pidx < a.n_pages) {
            const uint32_t* src = reinterpret_cast<const uint32_t*>(a.pages + ((size_t)pidx * a.Hkv + kvh) * a.page_bytes +
                                                                    (size_t)(tile & 1) * Stage::kBytes);
            uint32_t* dst = reinterpret_cast<uint32_t*>(smem + SM::kStageOff + (warp * NS + s) * Stage::kBytes);
            for (int w = lane; w < Stage::kBytes / 4; w += 32) dst[w] = __ldcg(src + w);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(mbar0 + s * 8);
    };
    for (int i = 0; i < NS && i < n_my; ++i) issue(i);
#endif

    int M[GT];
    float Mf[GT];            // M as a float (exact below 2^24)
    float l[GT];
    float acc[MT][4];        // O^T tiles: lane (gq, t4) holds dims 16 mt + 2 gq (+1) of queries 2 t4 (+1)
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        M[g] = kMNone;
        Mf[g] = (float)kMNone;
        l[g] = 0.0f;
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[mt][c] = 0.0f;
    int g_min = 0x7fffffff;                        // shift-A.V score pass only
    const int gq = lane >> 2, t4 = lane & 3;
    // row of this lane's key in the weight buffer: within a group of 8 keys the even keys come first
    const int prow = (lane & 24) | ((lane & 1) << 2) | ((lane & 7) >> 1);
    bool failed = false;

    for (int i = 0; i < n_my; ++i) {
        const int tile = first + NW * i;
        const int s = i % NS;
        const uint32_t parity = (uint32_t)(i / NS) & 1u;
        // the decision is made warp-uniform: a lane must never leave the loop alone
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(mbar0 + s * 8, parity, kPolls))) {
            failed = true;
            // give the other stage's copy (already issued) a bounded chance to land before this
            // warp's buffers are re-used by the block merge
            if (NS > 1 && i + 1 < n_my) (void)mbar_wait_bounded(mbar0 + ((i + 1) % NS) * 8, (uint32_t)((i + 1) / NS) & 1u, kPolls);
            break;
        }
        const int pidx = a.page_table[(size_t)b * a.max_pages + (tile >> 1)];
        const bool mapped = pidx >= 0 && pidx < a.n_pages;     // warp-uniform
        const uint8_t* st = stage_ptr0 + s * Stage::kBytes;
        if (mapped) {
            const int n_valid = min(32, len - tile * 32);

            // ---- phase 1: integer scores, lane = key; one 32-bit code word (4 or 8 elements) per
            // iteration, kept rolled so that the loop body stays in the instruction cache ----
            int32_t A[GT];
            const uint32_t* cw = reinterpret_cast<const uint32_t*>(st) + lane * 4;
            if constexpr (SM::kTable) {
                using TS = TableScore<KB, NP, MUL, ALUO>;
                uint32_t grp = smem_addr(smem + SM::kQpOff);    // table of the next 16 elements (256-byte aligned)
                TS ts;
                ts.begin(a.one);
                if constexpr (!NIB) {
#pragma unroll 1
                    for (int c = 0; c < WORDS / 4; ++c, grp += TS::kGroupBytes) {
                        const uint4 w4 = load_code_chunk(cw + c * 128);
                        ts.template accumulate_word<0>(w4.x, grp);
                        ts.template accumulate_word<1>(w4.y, grp);
                        ts.template accumulate_word<2>(w4.z, grp);
                        ts.template accumulate_word<3>(w4.w, grp);
                    }
                } else {
                    // dense planar container: 4 nibble words (32 elements) per 16-byte chunk, and per plane one
                    // 32-bit word of mantissa bits for the same 32 elements
                    const uint32_t* pw = reinterpret_cast<const uint32_t*>(st + Stage::kPlaneOff) + lane * (D / 32);
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        const uint4 w4 = load_code_chunk(cw + c * 128);
                        uint32_t pb[KB];
#pragma unroll
                        for (int bit = 0; bit < KB; ++bit) pb[bit] = pw[bit * (Stage::kPlaneBytes / 4) + c];
                        uint32_t pl[KB];
#pragma unroll
                        for (int bit = 0; bit < KB; ++bit) pl[bit] = pb[bit] & 0xffu;
                        ts.template accumulate_nibble_word<0>(w4.x, pl, grp);
#pragma unroll
                        for (int bit = 0; bit < KB; ++bit) pl[bit] = (pb[bit] >> 8) & 0xffu;
                        ts.template accumulate_nibble_word<1>(w4.y, pl, grp);
                        grp += TS::kGroupBytes;
#pragma unroll
                        for (int bit = 0; bit < KB; ++bit) pl[bit] = (pb[bit] >> 16) & 0xffu;
                        ts.template accumulate_nibble_word<0>(w4.z, pl, grp);
#pragma unroll
                        for (int bit = 0; bit < KB; ++bit) pl[bit] = pb[bit] >> 24;
                        ts.template accumulate_nibble_word<1>(w4.w, pl, grp);
                        grp += TS::kGroupBytes;
                    }
                }
#pragma unroll
                for (int g = 0; g < GT; ++g) A[g] = (int32_t)((uint32_t)ts.score(g) << a.f_extra);   // exact: the true sum fits INT32
            } else if constexpr (KB != 8) {
                // PoT-4: the packed pairs, shifted ahead of the loop, are looked up by the key's exponent field
                using ST = ShiftTable<NP>;
                PackedShift<NP, ALUO> pl;
                pl.begin(a.one);
                uint32_t grp = smem_addr(smem + SM::kQpOff);     // rows of the next group of elements (256-byte aligned)
                if constexpr (!NIB) {
#pragma unroll 1
                    for (int c = 0; c < D / 16; ++c, grp += 16 * ST::kRowBytes) {
                        const uint4 w4 = load_code_chunk(cw + c * 128);
                        accumulate_word_bytes_tab<NP, 0>(pl, w4.x, grp);
                        accumulate_word_bytes_tab<NP, 1>(pl, w4.y, grp);
                        accumulate_word_bytes_tab<NP, 2>(pl, w4.z, grp);
                        accumulate_word_bytes_tab<NP, 3>(pl, w4.w, grp);
                    }
                } else {
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c, grp += 32 * ST::kRowBytes) {
                        const uint4 w4 = load_code_chunk(cw + c * 128);
                        accumulate_word_nibbles_tab<NP>(pl, w4.x, grp);
                        accumulate_word_nibbles_tab<NP>(pl, w4.y, grp + 8 * ST::kRowBytes);
                        accumulate_word_nibbles_tab<NP>(pl, w4.z, grp + 16 * ST::kRowBytes);
                        accumulate_word_nibbles_tab<NP>(pl, w4.w, grp + 24 * ST::kRowBytes);
                    }
                }
#pragma unroll
                for (int g = 0; g < GT; ++g) A[g] = (int32_t)((uint32_t)pl.score(g) << a.f_extra);   // exact: the true sum fits INT32
            } else {
                // comparison datapath: four INT8 multiply-accumulates per instruction
                const uint32_t* q4_s = reinterpret_cast<const uint32_t*>(smem + SM::kQpOff);
#pragma unroll
                for (int g = 0; g < GT; ++g) A[g] = 0;
#pragma unroll 4
                for (int wq = 0; wq < D / 4; ++wq) {
                    const uint32_t w = cw[(wq >> 2) * 128 + (wq & 3)];
                    uint32_t q4[GT];
                    load_np<GT>(q4_s + wq * GT, q4);
#pragma unroll
                    for (int g = 0; g < GT; ++g) A[g] = __dp4a((int)q4[g], (int)w, A[g]);
                }
            }
            const uint32_t meta = reinterpret_cast<const uint32_t*>(st + Stage::kMetaOff)[lane];

            // ---- phase 2: logits, integer running maximum, weights ----
            const bool valid = lane < n_valid;
            const float s_j = half_bits_to_float(meta & 0xffffu);
            const int g_j = (int)(int8_t)((meta >> 16) & 0xffu);
            const float vscale = valid ? pow2i(-g_j) : 0.0f;  // 2^-g_j; g_j in [-10, 30] for written tokens
            if constexpr (SP) {
                // Score pass of the shift-based A.V option (eq. (6)): store the rounded logits and keep
                // the ceiling of the largest one and the smallest value exponent; no softmax, no A.V here.
#pragma unroll
                for (int g = 0; g < GT; ++g) {
                    if (a.dbg_scores && valid)
                        a.dbg_scores[((size_t)b * a.Hq + h0 + g) * a.dbg_stride + (size_t)tile * 32 + lane] = A[g];
                    const float z = valid ? fminf(fmaxf((float)A[g] * qscale_s[g] * s_j, -1.0e8f), 1.0e8f) : -1.0e8f;
                    M[g] = max(M[g], warp_max_s32(__float2int_ru(z)));
                    if (valid) a.zr[((size_t)b * a.Hq + h0 + g) * a.dbg_stride + (size_t)tile * 32 + lane] = __float2int_rn(z);
                }
                g_min = min(g_min, valid ? g_j : 0x7fffffff);
                __syncwarp();
#ifndef SA_ABLATE_WORD_STAGING
                if (lane == 0 && i + NS < n_my) {
                    fence_proxy_async();
                    issue(i + NS);
                }
#else
                if (i + NS < n_my) issue(i + NS);
#endif
                continue;
            }
            // The weights go where the tile's key codes were (every lane is done with them): row =
            // key, 8 query columns of FP32.
            __syncwarp();
            float (*p_t)[8] = reinterpret_cast<float (*)[8]>(const_cast<uint8_t*>(st));
            const float s_v = valid ? s_j : 0.0f, z_bias = valid ? 0.0f : -INFINITY;
            float pv[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};        // unused query columns stay zero
            if (a.dbg_scores && valid) {                      // parity tests only: one branch around all the stores
#pragma unroll
                for (int g = 0; g < GT; ++g)
                    a.dbg_scores[((size_t)b * a.Hq + h0 + g) * a.dbg_stride + (size_t)tile * 32 + lane] = A[g];
            }
            float z[GT];
            bool above = false;
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                // a lane without a key gets z = -inf through the addend (the product is rounded once either way)
                z[g] = fmaf((float)A[g] * qscale_s[g], s_v, z_bias);
                above |= z[g] > Mf[g];
            }
            // The running maximum M is an integer that bounds every logit seen so far from above; it has to
            // move only when a logit of this tile exceeds it, which after the first tiles is rare.
            if (__any_sync(0xffffffffu, above)) {             // warp-uniform
                float r0 = 0.0f, r1 = 0.0f;                   // rescale factors of this lane's queries 2 t4, 2 t4 + 1
#pragma unroll
                for (int g = 0; g < GT; ++g) {
                    // ceiling of the tile's largest logit: ceil is monotone, so take the integer maximum (the
                    // conversion saturates; a lane without a key gives the smallest integer)
                    const int Mt = max(warp_max_s32(__float2int_ru(z[g])), -(1 << 28));
                    const int Mo = __float2int_rn(Mf[g]);     // exact: M is an integer below 2^29 in magnitude
                    const int Mn = max(Mo, Mt);
                    const float resc = pow2i_neg(Mo - Mn);    // exact power of two; 0 while M is still "no key seen" (-2^29)
                    l[g] *= resc;
                    Mf[g] = (float)Mn;
                    if (t4 == g / 2) {
                        if (g & 1) r1 = resc;
                        else r0 = resc;
                    }
                }
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    acc[mt][0] *= r0;
                    acc[mt][1] *= r1;
                    acc[mt][2] *= r0;
                    acc[mt][3] *= r1;
                }
            }
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                const float p = ex2_approx(z[g] - Mf[g]);     // at most 1; 2^-inf = 0 for a lane without a key
                l[g] += p;
                pv[g] = p * vscale;                           // weight times 2^-g_j
            }
            reinterpret_cast<float4*>(&p_t[prow][0])[0] = make_float4(pv[0], pv[1], pv[2], pv[3]);
            reinterpret_cast<float4*>(&p_t[prow][0])[1] = make_float4(pv[4], pv[5], pv[6], pv[7]);
            __syncwarp();

            // ---- phase 3: O^T += V^T P^T on the tensor cores.  One 8 x 8 block of 16-bit pairs
            // (8 keys x 16 dims of INT8), transposed by ldmatrix, is the A fragment of one product:
            // column t of the product is key 2t of the block, column t + 4 is key 2t + 1; row gq is
            // dim 2 gq, row gq + 8 is dim 2 gq + 1.  The weight rows are stored in the same key order.
            // Every weight is split here into two tf32 terms (low 13 mantissa bits zero). ----
            uint32_t bh[4][2], bl[4][2];
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const float pv = p_t[8 * j + 4 * c + t4][gq];
                    const float hi = __uint_as_float(__float_as_uint(pv) & 0xffffe000u);
                    bh[j][c] = __float_as_uint(hi);
                    bl[j][c] = __float_as_uint(pv - hi) & 0xffffe000u;
                }
            const uint32_t vaddr = stage0 + s * Stage::kBytes + Stage::kVOff + lane * 16;   // chunk mt of key row `lane`
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                uint32_t x[4];
                ldmatrix_x4_trans(x, vaddr + mt * 512);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t a0 = __float_as_uint((float)(int8_t)(x[j]));
                    const uint32_t a1 = __float_as_uint((float)(int8_t)(x[j] >> 8));
                    const uint32_t a2 = __float_as_uint((float)(int8_t)(x[j] >> 16));
                    const uint32_t a3 = __float_as_uint((float)(int8_t)(x[j] >> 24));
                    mma_tf32_1688(acc[mt], a0, a1, a2, a3, bh[j][0], bh[j][1]);
                    mma_tf32_1688(acc[mt], a0, a1, a2, a3, bl[j][0], bl[j][1]);
                }
            }
        }
        __syncwarp();                                         // every lane is done with this stage
#ifndef SA_ABLATE_WORD_STAGING
        if (lane == 0 && i + NS < n_my) {
            fence_proxy_async();
            issue(i + NS);
        }
#else
        if (i + NS < n_my) issue(i + NS);
#endif
    }
    if constexpr (!SP) {
#pragma unroll
        for (int g = 0; g < GT; ++g) M[g] = __float2int_rn(Mf[g]);      // exact: an integer of magnitude at most 2^29
    }
    if (failed) {
        // A bounded wait expired: make the failure visible in the output instead of returning a
        // plausible number (no copy of this warp can still be in flight into a buffer it re-uses).
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            l[g] = __int_as_float(0x7fc00000);
            M[g] = max(M[g], 0);                               // a state that "saw no key" would be skipped by the merges
        }
    }

    // ---- merge the warps of the block, write the block's partial ----
    __syncthreads();
    if constexpr (SP) {
        // score pass of the shift-A.V option: the block's statistics instead of a partial
        int* stat_s = reinterpret_cast<int*>(smem + SM::kStageOff);           // [NW][GT + 1]
        g_min = warp_min_s32(g_min);
        if (lane == 0) {
#pragma unroll
            for (int g = 0; g < GT; ++g) stat_s[warp * (GT + 1) + g] = failed ? 0x7fffffff : M[g];
            stat_s[warp * (GT + 1) + GT] = g_min;
        }
        __syncthreads();
        if (threadIdx.x <= GT) {
            int v = (threadIdx.x < GT) ? kMNone : 0x7fffffff;
            for (int w = 0; w < NW; ++w) {
                const int x = stat_s[w * (GT + 1) + threadIdx.x];
                v = (threadIdx.x < GT) ? max(v, x) : min(v, x);
            }
            if (threadIdx.x < GT) a.stat_m[((size_t)split * a.batch + b) * a.Hq + h0 + threadIdx.x] = v;
            else a.stat_g[((size_t)split * a.batch + b) * gridDim.y + blockIdx.y] = v;
        }
        return;
    }
    // the block's slot among the partials (recomputed here rather than carried through the tile loop)
    const int slot = ranked ? blockIdx.z * a.n_splits + blockIdx.x : blockIdx.x * a.batch + blockIdx.z;
    block_merge_and_store<D, GT, NW>(a, red_s, M, l, acc, lane, warp, slot, h0, failed);
}

template <int D, int KB, bool NIB, int GT, int MODE>
static void launch_one(const DecodeArgs& a, dim3 grid, cudaStream_t s) {
    constexpr int bytes = DecodeSmem<D, KB, NIB, GT>::kBytes;
    if (bytes > 48 * 1024) {
        // opt in to more than 48 KB of dynamic shared memory (an attribute of the function; no allocation)
        static const cudaError_t once = cudaFuncSetAttribute(decode_kernel<D, KB, NIB, GT, MODE>,
                                                             cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        (void)once;
    }
    (void)launch_pdl(decode_kernel<D, KB, NIB, GT, MODE>, grid, dim3(32 * DecodeSmem<D, KB, NIB, GT>::NW), (size_t)bytes, s, a);
}

template <int D, int KB, bool NIB, int MODE>
static void launch_gt(const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s) {
    switch (GT) {
        case 8: launch_one<D, KB, NIB, 8, MODE>(a, grid, s); break;
        case 4: launch_one<D, KB, NIB, 4, MODE>(a, grid, s); break;
        case 2: launch_one<D, KB, NIB, 2, MODE>(a, grid, s); break;
        default: launch_one<D, KB, NIB, 1, MODE>(a, grid, s); break;
    }
}

// All instantiations of one key code and container: head_dim 64 / 128, the queries per block, and the
// kernel's mode (0 decode; 1 the same with the shifts on the integer multiplier, mantissa codes only;
// 2 the score pass of the shift-based A.V option, 3 sign flips and adds on the ALU pipe: power-of-two codes only).
template <int KB, bool NIB>
static void launch_code(int d, int mode, const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s) {
    constexpr bool kPot = (KB != 8);
    constexpr bool kMul = (KB == 1 || KB == 2 || KB == 4);
    if (d == 64) {
        if (kPot && mode == 2) launch_gt<64, KB, NIB, kPot ? 2 : 0>(a, GT, grid, s);
        else if (kPot && mode == 3) launch_gt<64, KB, NIB, kPot ? 3 : 0>(a, GT, grid, s);
        else if (kMul && mode == 1) launch_gt<64, KB, NIB, kMul ? 1 : 0>(a, GT, grid, s);
        else launch_gt<64, KB, NIB, 0>(a, GT, grid, s);
    } else {
        if (kPot && mode == 2) launch_gt<128, KB, NIB, kPot ? 2 : 0>(a, GT, grid, s);
        else if (kPot && mode == 3) launch_gt<128, KB, NIB, kPot ? 3 : 0>(a, GT, grid, s);
        else if (kMul && mode == 1) launch_gt<128, KB, NIB, kMul ? 1 : 0>(a, GT, grid, s);
        else launch_gt<128, KB, NIB, 0>(a, GT, grid, s);
    }
}

// One translation unit per key code (they compile in parallel); nib: the sub-byte container of the code.
void launch_decode_pot4(bool nib, int d, int mode, const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s);
void launch_decode_potm1(bool nib, int d, int mode, const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s);
void launch_decode_potm2(bool nib, int d, int mode, const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s);
void launch_decode_potm4(int d, int mode, const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s);
void launch_decode_potm4_lost_copy(const DecodeArgs& a, dim3 grid, cudaStream_t s);   // test hook: head_dim 64, 8 queries per block
void launch_decode_int8(int d, const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s);

}  // namespace sa
