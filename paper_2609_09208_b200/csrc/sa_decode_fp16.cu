// Decode attention over an unquantised binary16 cache: softmax(Q K^T / sqrt(d)) V of eq. (1) with
// FP32 accumulation — the like-for-like baseline of the power-of-two kernels (the paper's three
// levels of comparison put FP16 attention on tensor cores, section III).
//
// Same grid, split and merge as the quantised kernel; each warp streams its own 32-key tiles
// through a two-stage shared-memory ring filled by bulk-async copies.  Per tile:
//   S^T = Q K^T   as  mma.m16n8k16: rows = the block's (up to 8) query heads padded to 16,
//                     k = head dims, n = 8 keys;  Q fragments live in registers for the whole kernel,
//                     K fragments are 32-bit shared-memory loads from the 16-byte chunk layout;
//   online softmax with an integer running maximum (the 4 lanes of a row share its 32 keys);
//   O += P V      as  mma.m16n8k16: the S^T accumulators, converted to binary16, are exactly the
//                     A fragments of P; V fragments come from ldmatrix.trans on 8 x 8 blocks
//                     (8 keys x one 16-byte chunk), which the chunk layout stores contiguously.
#include "sa_common.cuh"
#include "sa_cache_write.cuh"
#include "sa_decode_common.cuh"
#include "sa_mma.cuh"
#include "sa_quant.cuh"
#include "sa_stage.cuh"

namespace sa {

SA_D uint32_t pack_half2(float lo, float hi) {
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// Stage buffer of one 32-key tile = one half of a page block: K chunks [D/8][32 keys][16 B], then V chunks
// [D/8][32 keys][16 B].
template <int D>
struct Fp16Stage {
    static constexpr int kChunks = D / 8;
    static constexpr int kVOff = kChunks * 512;
    static constexpr int kBytes = 2 * kChunks * 512;
    static_assert(kBytes == half_block_bytes_fp16(D), "a stage buffer is a verbatim copy of half a page block");
    // tk0 = 0 or 32: the tile is that half of the (page, KV head) block, laid out like the stage buffer: one copy
    SA_D static void issue(uint32_t dst, const uint8_t* block, int tk0, uint32_t mbar) {
        mbar_arrive_expect_tx(mbar, (uint32_t)kBytes);
        bulk_g2s(dst, block + (size_t)(tk0 >> 5) * kBytes, (uint32_t)kBytes, mbar);
    }
    // the same range as an L2 prefetch hint
    SA_D static void prefetch(const uint8_t* block, int tk0) {
        bulk_prefetch_l2(block + (size_t)(tk0 >> 5) * kBytes, (uint32_t)kBytes);
    }
};

template <int D, int GT>
struct Fp16Smem {
    using Stage = Fp16Stage<D>;
    static constexpr int kStageOff = 0;
    static constexpr int kMbarOff = 4 * kStages * Stage::kBytes;
    static constexpr int kBytes = kMbarOff + 128;
    static_assert(4 * GT * (D + 2) * 4 <= 4 * kStages * Stage::kBytes, "merge scratch must fit in the stage buffers");
    static_assert(kPlanScratchInts * 4 <= 4 * kStages * Stage::kBytes, "the block plan's scratch must fit in the stage buffers");
};

template <int D, int GT>
__global__ void __launch_bounds__(128, 3) decode_fp16_kernel(DecodeArgs a) {
    using SM = Fp16Smem<D, GT>;
    using Stage = typename SM::Stage;
    constexpr int KB16 = D / 16;                   // 16-dim blocks of the QK product
    constexpr int NB8 = D / 8;                     // 8-dim blocks of the output
    extern __shared__ __align__(128) uint8_t smem[];
    float (*red_s)[GT][D + 2] = reinterpret_cast<float (*)[GT][D + 2]>(smem + SM::kStageOff);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row = lane >> 2, quad = lane & 3;    // fragment row (query) and column pair
    const int chunks = a.G / GT;
    const int kvh = blockIdx.y / chunks;
    const int h0 = kvh * a.G + (blockIdx.y % chunks) * GT;
    // batches of 2 .. 128 sequences: the block's (sequence, split) is dealt by plan_block from the cached lengths,
    // guessed ahead of the dependency wait and settled after it (see the quantised kernel)
    const bool ranked = batch_is_ranked(a.batch);
    int* plan_scratch = reinterpret_cast<int*>(smem + SM::kStageOff);
    BlockPlan bp{(int)blockIdx.z, (int)blockIdx.x, a.n_splits, 0};
    if (a.wait_first) pdl_wait();
    if (ranked) bp = plan_block(plan_args(a), blockIdx.z, blockIdx.x, false, a.wait_first != 0, bp, plan_scratch);
    int b = bp.b;
    const uint32_t mbar0 = smem_addr(smem + SM::kMbarOff) + warp * kStages * 8;
    const uint32_t stage0 = smem_addr(smem + SM::kStageOff) + warp * kStages * Stage::kBytes;
    const uint8_t* stage_ptr0 = smem + SM::kStageOff + warp * kStages * Stage::kBytes;

    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) mbar_init(mbar0 + s * 8, 1u);
        fence_mbar_init();
        fence_proxy_async();
    }
    __syncwarp();

    pdl_launch_dependents();    // the split-K merge may be scheduled as soon as blocks of this grid retire

    // Q fragments (A operand, rows = query heads; rows >= GT are zero): for 16-dim block kb the lane
    // holds dims 16kb + 2*quad + {0,1} and + 8 of query `row`.
    uint32_t qa[KB16][2];
    int tile_g, pidx_g;
    bool again;
#pragma unroll 1
    do {
        const int split_g = bp.split, nsp_g = bp.n_splits;         // what the hint below is computed for
        const int bq = b < 0 ? 0 : b;                              // (a block without work so far prepares sequence 0)
#pragma unroll
        for (int kb = 0; kb < KB16; ++kb) {
            qa[kb][0] = qa[kb][1] = 0u;
            if (row < GT) {
                const uint32_t* q32 = reinterpret_cast<const uint32_t*>(a.Q + ((size_t)bq * a.Hq + h0 + row) * D);
                qa[kb][0] = __ldg(q32 + kb * 8 + quad);
                qa[kb][1] = __ldg(q32 + kb * 8 + 4 + quad);
            }
        }

        // While the preceding kernel drains: ask L2 for this warp's first tile, guessed from a length that kernel
        // may be about to change (loads that bypass L1; a hint only).
        tile_g = -1, pidx_g = -1;
        if (lane == 0) {
            const int len_g = (ranked ? bp.len : __ldcg(a.seq_lens + bq)) + (a.Knew ? 1 : 0);
            const int n_tiles_g = (min(max(len_g, 0), a.max_pages * kPageTokens) + 31) >> 5;
            const int t_g = split_begin(n_tiles_g, bp.split, bp.n_splits) + warp;
            if (t_g < split_begin(n_tiles_g, (bp.split + 1), bp.n_splits)) {
                tile_g = t_g;
                const int p_g = __ldcg(a.page_table + (size_t)bq * a.max_pages + (t_g >> 1));
                if (p_g >= 0 && p_g < a.n_pages)
                    Stage::prefetch(a.pages + ((size_t)p_g * a.Hkv + kvh) * a.page_bytes, (t_g & 1) * 32);
            }
        }
        pdl_wait();                 // everything below reads what the preceding kernels in the stream wrote (the cache)
        // the page of the guessed first tile, read again now that it is valid, together with the length(s) (one round
        // trip instead of two when the guess holds)
        if (lane == 0 && tile_g >= 0) pidx_g = a.page_table[(size_t)bq * a.max_pages + (tile_g >> 1)];
        again = false;
        if (ranked && !a.wait_first) {
            bp = plan_block(plan_args(a), blockIdx.z, blockIdx.x, true, true, bp, plan_scratch);
            again = bp.b != bq && bp.b >= 0;
            if (bp.split != split_g || bp.n_splits != nsp_g) tile_g = -1;     // the hint was for other tiles
            b = bp.b;
        }
    } while (again);
    if (ranked && b < 0) return;                                  // more blocks than (sequence, split) pairs
    const int split = bp.split, n_splits = bp.n_splits;

    int len = ranked ? bp.len : a.seq_lens[b];
    int tile_new = -1, pidx_new = -1;
    if (a.Knew) {
        // fused append (see the quantised kernel): the step's new token goes to position len if its page is mapped
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
    const int n_my = first < tile1 ? (tile1 - first + 3) >> 2 : 0;
    if (tile_new >= first && tile_new < tile1 && (tile_new - first) % 4 == 0) {      // this warp owns that tile
        CacheArgs ca{};
        ca.page_bytes = a.page_bytes;
        ca.kcode_off = a.kcode_off;
        ca.v_off = a.v_off;
        uint8_t* block = const_cast<uint8_t*>(a.pages) + ((size_t)pidx_new * a.Hkv + kvh) * a.page_bytes;
        const size_t rown = ((size_t)b * a.Hkv + kvh) * D;
        write_token<D, 16>(block, ca, (len - 1) % kPageTokens, lane, a.Knew + rown, a.Vnew + rown);
        fence_proxy_async_global();
        __syncwarp();
    }
    auto issue = [&](int i) {
        const int tile = first + 4 * i;
        const int pidx = (tile == tile_g) ? pidx_g : a.page_table[(size_t)b * a.max_pages + (tile >> 1)];
        const int s = i % kStages;
        if (pidx < 0 || pidx >= a.n_pages) {
            mbar_arrive(mbar0 + s * 8);
        } else {
            const uint8_t* block = a.pages + ((size_t)pidx * a.Hkv + kvh) * a.page_bytes;
            Stage::issue(stage0 + s * Stage::kBytes, block, (tile & 1) * 32, mbar0 + s * 8);
        }
    };
    if (lane == 0)
        for (int i = 0; i < kStages && i < n_my; ++i) issue(i);

    int M = kMNone;                                // running maximum of this lane's query row
    float l = 0.0f;                                // this lane's share of the row's weight sum
    float o[NB8][4];
#pragma unroll
    for (int nb = 0; nb < NB8; ++nb) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.0f;
    bool failed = false;

    for (int i = 0; i < n_my; ++i) {
        const int tile = first + 4 * i;
        const int s = i % kStages;
        const uint32_t parity = (uint32_t)(i / kStages) & 1u;
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(mbar0 + s * 8, parity))) {
            failed = true;
            if (i + 1 < n_my) (void)mbar_wait_bounded(mbar0 + ((i + 1) % kStages) * 8, (uint32_t)((i + 1) / kStages) & 1u);
            break;
        }
        const int pidx = a.page_table[(size_t)b * a.max_pages + (tile >> 1)];
        if (pidx >= 0 && pidx < a.n_pages) {
            const int n_valid = min(32, len - tile * 32);
            const uint8_t* st = stage_ptr0 + s * Stage::kBytes;
            const uint32_t st_addr = stage0 + s * Stage::kBytes;

            // ---- S^T = Q K^T: four 8-key blocks ----
            float sc[4][4];
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) {
                sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.0f;
                // key nb*8 + row, dims 2*quad + {0,1} of every 16-byte chunk
                const uint32_t* kw = reinterpret_cast<const uint32_t*>(st) + (nb * 8 + row) * 4 + quad;
#pragma unroll
                for (int kb = 0; kb < KB16; ++kb) {
                    const uint32_t b0 = kw[(2 * kb) * 128];          // chunk 2kb: dims 16kb + 2*quad + {0,1}
                    const uint32_t b1 = kw[(2 * kb + 1) * 128];      // chunk 2kb+1: dims 16kb + 8 + ...
                    mma_f16_16816(sc[nb], qa[kb][0], 0u, qa[kb][1], 0u, b0, b1);
                }
            }

            // ---- online softmax, integer running maximum; this lane: row `row`, keys nb*8 + 2*quad + {0,1} ----
            float zmax = -INFINITY;
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int key = nb * 8 + 2 * quad + e;
                    sc[nb][e] = (key < n_valid) ? sc[nb][e] * a.zscale : -INFINITY;
                    zmax = fmaxf(zmax, sc[nb][e]);
                }
            }
            zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, 1));
            zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, 2));
            const int Mt = (int)ceilf(fminf(fmaxf(zmax, -1.0e8f), 1.0e8f));
            const int Mn = max(M, Mt);
            const float resc = (M == kMNone) ? 0.0f : pow2i_neg(M - Mn);
            if (Mn != M) {
#pragma unroll
                for (int nb = 0; nb < NB8; ++nb) { o[nb][0] *= resc; o[nb][1] *= resc; }
            }
            M = Mn;
            l *= resc;
            uint32_t pa[4];                                          // P as A fragments, one per 8-key block
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) {
                const float p0 = ex2_approx(sc[nb][0] - (float)Mn);  // exp2(-inf) = 0 for masked keys
                const float p1 = ex2_approx(sc[nb][1] - (float)Mn);
                // the weights enter the product rounded to binary16; the normaliser sums the same rounded
                // values, so that the result stays an exact weighted mean of the value rows
                const __half2 ph = __floats2half2_rn(p0, p1);
                const float2 pr = __half22float2(ph);
                l += pr.x + pr.y;
                pa[nb] = *reinterpret_cast<const uint32_t*>(&ph);
            }

            // ---- O += P V: two 16-key blocks x D/8 output blocks ----
#pragma unroll
            for (int nb = 0; nb < NB8; ++nb) {
                uint32_t vb[4];                                      // V^T fragments of chunk nb: keys 0-7, 8-15, 16-23, 24-31
                ldmatrix_x4_trans(vb, st_addr + Stage::kVOff + (nb * 32 + lane) * 16);
                if (n_valid < 32) {
                    // slots past the sequence end may hold anything (even NaN patterns): their weight is
                    // zero, but 0 * NaN is not, so the value halves of those keys are cleared
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int key = j * 8 + 2 * quad;
                        if (key >= n_valid) vb[j] = 0u;
                        else if (key + 1 >= n_valid) vb[j] &= 0x0000ffffu;
                    }
                }
                mma_f16_16816(o[nb], pa[0], 0u, pa[1], 0u, vb[0], vb[1]);
                mma_f16_16816(o[nb], pa[2], 0u, pa[3], 0u, vb[2], vb[3]);
            }
        }
        __syncwarp();
        if (lane == 0 && i + kStages < n_my) {
            fence_proxy_async();
            issue(i + kStages);
        }
    }
    if (failed) {                                  // a bounded wait expired: make it visible in the output
        l = __int_as_float(0x7fc00000);
        M = max(M, 0);                             // a state that "saw no key" would be skipped by the merges
    }

    // ---- per-warp state -> shared memory, merge the four warps, write the block's partial ----
    __syncthreads();                               // the merge scratch re-uses the stage buffers
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if (row < GT) {
#pragma unroll
        for (int nb = 0; nb < NB8; ++nb) {
            red_s[warp][row][2 + nb * 8 + 2 * quad] = o[nb][0];
            red_s[warp][row][2 + nb * 8 + 2 * quad + 1] = o[nb][1];
        }
        if (quad == 0) {
            red_s[warp][row][0] = __int_as_float(M);
            red_s[warp][row][1] = l;
        }
    }
    __syncthreads();
    const int slot = ranked ? blockIdx.z * a.n_splits + blockIdx.x : blockIdx.x * a.batch + blockIdx.z;
    block_combine_and_store<D, GT>(a, red_s, slot, h0);
}

}  // namespace sa

using namespace sa;

template <int D, int GT>
static void launch_fp16_one(const DecodeArgs& a, dim3 grid, cudaStream_t s) {
    constexpr int bytes = Fp16Smem<D, GT>::kBytes;
    if (bytes > 48 * 1024) {
        // opt in to more than 48 KB of dynamic shared memory (an attribute of the function; no allocation)
        static const cudaError_t once = cudaFuncSetAttribute(decode_fp16_kernel<D, GT>,
                                                             cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        (void)once;
    }
    (void)launch_pdl(decode_fp16_kernel<D, GT>, grid, dim3(128), (size_t)bytes, s, a);
}

template <int D>
static void launch_fp16(const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s) {
    switch (GT) {
        case 8: launch_fp16_one<D, 8>(a, grid, s); break;
        case 4: launch_fp16_one<D, 4>(a, grid, s); break;
        case 2: launch_fp16_one<D, 2>(a, grid, s); break;
        default: launch_fp16_one<D, 1>(a, grid, s); break;
    }
}

namespace sa {
// the binary16 decode kernel for these arguments (used by sa_decode_step as well)
void launch_decode_fp16_main(const Plan& p, const DecodeArgs& a, int GT, cudaStream_t s) {
    const dim3 grid((unsigned)a.n_splits, (unsigned)(p.Hkv * (p.G / GT)), (unsigned)a.batch);
    if (p.d == 64) launch_fp16<64>(a, GT, grid, s);
    else launch_fp16<128>(a, GT, grid, s);
}
}  // namespace sa

extern "C" sa_status sa_decode_attention_fp16_stages(const sa_config* cfg, const sa_cache* cache,
                                                     const uint16_t* Q, float* O, void* workspace,
                                                     size_t workspace_bytes, int stages, sa_stream stream) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (!p.fp16) return SA_ERR_UNSUPPORTED;
    if ((stages & ~3) || stages == 0) return SA_ERR_INVALID_ARG;
    DecodeArgs a;
    int GT;
    st = make_decode_args(p, cache, Q, O, workspace, workspace_bytes, &a, &GT);
    if (st != SA_OK) return st;
    a.zscale = (float)(1.4426950408889634 / sqrt((double)p.d));
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (stages & 1) {
        launch_decode_fp16_main(p, a, GT, s);
        if (cudaGetLastError() != cudaSuccess) return SA_ERR_CUDA;
    }
    return (stages & 2) ? launch_merge(p, a, s) : SA_OK;
}

extern "C" sa_status sa_decode_attention_fp16(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q,
                                              float* O, void* workspace, size_t workspace_bytes,
                                              sa_stream stream) {
    return sa_decode_attention_fp16_stages(cfg, cache, Q, O, workspace, workspace_bytes, 3, stream);
}
