// The paper's non-default option: attention weights quantised to powers of two and the
// shift-based A.V (section II-E eq. (6), (7); section V-G "Both products, and why only one by
// default").
//
//   M = ceil(max_j z_j),  k_j = M - round(z_j) >= 0,  weight 2^-k_j                       eq. (6)
//   O = 2^(-N - g_ref) * sum_{j : k_j <= k_max} vhat_j << (N - k_j + g_ref - g_j)         eq. (7)
//       divided by sum_{j : k_j <= k_max} 2^-k_j;   g_ref = min_j g_j.
//
// Both M and g_ref are those of the whole sequence, so the option runs as two passes over the
// key axis instead of one streaming pass with running values (whose truncations would depend on
// the order of the tiles):
//   pass 1  the decode kernel's score phase (sa_decode_kernel.cuh, DecodeArgs::zr != null): integer
//           scores, rounded logits to memory, per block the ceiling of its largest logit and its
//           smallest value exponent;
//   pass 2  shiftav_kernel below: reduces those statistics to M and g_ref, then per 32-key tile
//           forms the shift indices (lane = key), accumulates vhat << index in INT32 (lane =
//           output dims; the paper notes that an INT32 accumulator per tile is enough) and adds the tile's sum to FP32
//           running sums; a key with k_j > k_max is dropped everywhere, one with a negative shift
//           index from the numerator only;
//   merge   the ordinary split-K merge (all partials share the reference M, so its factors are 1).
// Integer decisions (round, ceil) are taken on the binary32 logit formed exactly as in the default
// path; everything after them is exact integer arithmetic up to the FP32 sums over tiles.
#include "sa_common.cuh"
#include "sa_decode_common.cuh"
#include "sa_mma.cuh"
#include "sa_stage.cuh"

namespace sa {

template <int D, int GT>
struct ShiftAvSmem {
    using Stage = TileStage<0, true, D>;           // metadata and value rows only
    static constexpr int kStageOff = 0;
    static constexpr int kMbarOff = 4 * kStages * Stage::kBytes;
    static constexpr int kShOff = kMbarOff + 128;  // shift indices [4 warps][32 keys][8 queries] bytes
    static constexpr int kStatOff = kShOff + 4 * 32 * 8;
    static constexpr int kBytes = kStatOff + 64;   // M[8] and g_ref
    static_assert(4 * GT * (D + 2) * 4 <= 4 * kStages * Stage::kBytes, "merge scratch must fit in the stage buffers");
};

template <int D, int GT>
__global__ void __launch_bounds__(128) shiftav_kernel(DecodeArgs a) {
    using SM = ShiftAvSmem<D, GT>;
    using Stage = typename SM::Stage;
    constexpr int DPL = D / 32;                    // output dims per lane
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t (*sh_s)[32][8] = reinterpret_cast<uint8_t (*)[32][8]>(smem + SM::kShOff);
    int* stat_s = reinterpret_cast<int*>(smem + SM::kStatOff);
    float (*red_s)[GT][D + 2] = reinterpret_cast<float (*)[GT][D + 2]>(smem + SM::kStageOff);

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chunks = a.G / GT;
    const int kvh = blockIdx.y / chunks;
    const int h0 = kvh * a.G + (blockIdx.y % chunks) * GT;
    const int b = blockIdx.z;
    const int split = blockIdx.x;
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
    pdl_wait();
    pdl_launch_dependents();

    const int len = a.seq_lens[b];
    const int n_tiles = (min(len, a.max_pages * kPageTokens) + 31) >> 5;
    const int tile0 = split_begin(n_tiles, split, a.n_splits);
    const int tile1 = split_begin(n_tiles, (split + 1), a.n_splits);
    const int first = tile0 + warp;
    const int n_my = first < tile1 ? (tile1 - first + 3) >> 2 : 0;
    auto issue = [&](int i) {
        const int tile = first + 4 * i;
        const int pidx = a.page_table[(size_t)b * a.max_pages + (tile >> 1)];
        const int s = i % kStages;
        if (pidx < 0 || pidx >= a.n_pages) {
            mbar_arrive(mbar0 + s * 8);
        } else {
            const uint8_t* block = a.pages + ((size_t)pidx * a.Hkv + kvh) * a.page_bytes;
            Stage::issue_values(stage0 + s * Stage::kBytes, block, a.page_bytes, a.meta_off, (tile & 1) * 32, mbar0 + s * 8);
        }
    };
    if (lane == 0)
        for (int i = 0; i < kStages && i < n_my; ++i) issue(i);

    // ---- M per query head and g_ref, from the statistics of pass 1 (every split of this sequence) ----
    if (warp <= GT && warp < 4) {
        for (int q = warp; q <= GT; q += 4) {          // q < GT: a query's maximum; q == GT: the minimum exponent
            int v = (q < GT) ? kMNone : 0x7fffffff;
            for (int s = lane; s < a.n_splits; s += 32) {
                if (q < GT) v = max(v, a.stat_m[((size_t)s * a.batch + b) * a.Hq + h0 + q]);
                else v = min(v, a.stat_g[((size_t)s * a.batch + b) * gridDim.y + blockIdx.y]);
            }
            v = (q < GT) ? warp_max_s32(v) : warp_min_s32(v);
            if (lane == 0) stat_s[q] = v;
        }
    }
    __syncthreads();
    int Mq[GT];
    bool poisoned = false;
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        Mq[g] = stat_s[g];
        poisoned |= (Mq[g] == 0x7fffffff);            // pass 1 gave up on a bounded wait
    }
    const int g_ref = (stat_s[GT] == 0x7fffffff) ? 0 : stat_s[GT];
    const int N = a.n_bits, k_max = a.k_max;

    float l[GT];
    float O[GT][DPL];
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        l[g] = 0.0f;
#pragma unroll
        for (int c = 0; c < DPL; ++c) O[g][c] = 0.0f;
    }
    bool failed = false;

    for (int i = 0; i < n_my; ++i) {
        const int tile = first + 4 * i;
        const int s = i % kStages;
        const uint32_t parity = (uint32_t)(i / kStages) & 1u;
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(mbar0 + s * 8, parity))) {   // warp-uniform
            failed = true;
            if (i + 1 < n_my) (void)mbar_wait_bounded(mbar0 + ((i + 1) % kStages) * 8, (uint32_t)((i + 1) / kStages) & 1u);
            break;
        }
        const int pidx = a.page_table[(size_t)b * a.max_pages + (tile >> 1)];
        const bool mapped = pidx >= 0 && pidx < a.n_pages;
        const uint8_t* st = stage_ptr0 + s * Stage::kBytes;
        if (mapped) {
            // ---- shift indices, lane = key ----
            const bool valid = lane < min(32, len - tile * 32);
            const uint32_t meta = reinterpret_cast<const uint32_t*>(st + Stage::kMetaOff)[lane];
            const int g_j = (int)(int8_t)((meta >> 16) & 0xffu);
            uint32_t idx[2] = {0x20202020u, 0x20202020u};        // 32: "shift everything out"
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                const int zr = valid ? a.zr[((size_t)b * a.Hq + h0 + g) * a.dbg_stride + (size_t)tile * 32 + lane] : 0;
                const long long k = (long long)Mq[g] - zr;       // >= 0
                const bool keep = valid && k <= k_max;
                l[g] += keep ? (float)(1u << (N - (int)k)) : 0.0f;   // 2^(N - k), exact
                const long long sh = (long long)N - k + g_ref - g_j;
                const uint32_t code = (keep && sh >= 0) ? (uint32_t)sh : 32u;
                idx[g >> 2] = (idx[g >> 2] & ~(0xffu << (8 * (g & 3)))) | (code << (8 * (g & 3)));
            }
            *reinterpret_cast<uint2*>(&sh_s[warp][lane][0]) = make_uint2(idx[0], idx[1]);
            __syncwarp();

            // ---- per-tile INT32 accumulation of vhat << index, lane = DPL output dims ----
            uint32_t acc[GT][DPL];
#pragma unroll
            for (int g = 0; g < GT; ++g)
#pragma unroll
                for (int c = 0; c < DPL; ++c) acc[g][c] = 0u;
            // values are staged in 16-dim chunks of 512 bytes: this lane's dims sit in chunk (lane * DPL) / 16
            const uint8_t* vbase = st + Stage::kVOff + ((lane * DPL) >> 4) * 512 + ((lane * DPL) & 15);
#pragma unroll 4
            for (int t = 0; t < 32; ++t) {
                uint32_t v[DPL];
                if constexpr (DPL == 2) {
                    const uint32_t vv = *reinterpret_cast<const uint16_t*>(vbase + t * 16);
                    v[0] = (uint32_t)(int32_t)(int8_t)(vv);
                    v[1] = (uint32_t)(int32_t)(int8_t)(vv >> 8);
                } else {
                    const uint32_t vv = *reinterpret_cast<const uint32_t*>(vbase + t * 16);
#pragma unroll
                    for (int c = 0; c < DPL; ++c) v[c] = (uint32_t)(int32_t)(int8_t)(vv >> (8 * c));
                }
                const uint2 ix = *reinterpret_cast<const uint2*>(&sh_s[warp][t][0]);
#pragma unroll
                for (int g = 0; g < GT; ++g) {
                    const uint32_t shift = ((g < 4 ? ix.x : ix.y) >> (8 * (g & 3))) & 0xffu;
#pragma unroll
                    for (int c = 0; c < DPL; ++c) acc[g][c] += shl_clamp(v[c], shift);   // two's complement: exact modulo 2^32
                }
            }
#pragma unroll
            for (int g = 0; g < GT; ++g)
#pragma unroll
                for (int c = 0; c < DPL; ++c) O[g][c] += (float)(int32_t)acc[g][c];
        }
        __syncwarp();
        if (lane == 0 && i + kStages < n_my) {
            fence_proxy_async();
            issue(i + kStages);
        }
    }
    if (failed || poisoned) {
#pragma unroll
        for (int g = 0; g < GT; ++g) l[g] = __int_as_float(0x7fc00000);
    }

    // ---- block partial: {M = 0, l in units of 2^-N, O in units of 2^-N (scaled by 2^-g_ref)} ----
    __syncthreads();
    const float vs = pow2i(-g_ref);
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        const float lsum = warp_sum_f32(l[g]);
        if (lane == 0) {
            red_s[warp][g][0] = __int_as_float(0);
            red_s[warp][g][1] = lsum;
        }
#pragma unroll
        for (int c = 0; c < DPL; ++c) red_s[warp][g][2 + lane * DPL + c] = O[g][c] * vs;
    }
    __syncthreads();
    block_combine_and_store<D, GT, 4>(a, red_s, split * a.batch + b, h0);
}

template <int D, int GT>
static void launch_shiftav(const DecodeArgs& a, dim3 grid, cudaStream_t s) {
    constexpr int bytes = ShiftAvSmem<D, GT>::kBytes;
    (void)launch_pdl(shiftav_kernel<D, GT>, grid, dim3(128), (size_t)bytes, s, a);
}

template <int D>
static void launch_shiftav_gt(const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s) {
    switch (GT) {
        case 8: launch_shiftav<D, 8>(a, grid, s); break;
        case 4: launch_shiftav<D, 4>(a, grid, s); break;
        case 2: launch_shiftav<D, 2>(a, grid, s); break;
        default: launch_shiftav<D, 1>(a, grid, s); break;
    }
}

// defined in sa_decode.cu: launches the decode kernel for these arguments (score pass when a.zr is set)
void launch_decode_main(const Plan& p, const DecodeArgs& a, int GT, cudaStream_t s);

static size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

// workspace: [split-K partials][rounded logits][stat_m][stat_g]
static void shiftav_layout(const Plan& p, int batch, int max_pages, int S, int GT, size_t* zr_off, size_t* m_off,
                           size_t* g_off, size_t* total) {
    const size_t partials = (size_t)S * batch * p.Hq * (p.d + 2) * sizeof(float);
    const size_t zr = (size_t)batch * p.Hq * max_pages * kPageTokens * sizeof(int32_t);
    const size_t sm = (size_t)S * batch * p.Hq * sizeof(int32_t);
    const size_t sg = (size_t)S * batch * p.Hkv * (p.G / GT) * sizeof(int32_t);
    *zr_off = align_up(partials);
    *m_off = *zr_off + align_up(zr);
    *g_off = *m_off + align_up(sm);
    *total = *g_off + align_up(sg);
}

}  // namespace sa

using namespace sa;

extern "C" sa_status sa_shiftav_workspace_bytes(const sa_config* cfg, int batch, int max_pages_per_seq, size_t* out) {
    if (!out || batch <= 0 || max_pages_per_seq <= 0) return SA_ERR_INVALID_ARG;
    Plan p;
    const sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (p.fp16 || p.int8) return SA_ERR_UNSUPPORTED;
    int S, GT;
    split_plan(p, batch, max_pages_per_seq, &S, &GT);
    size_t zo, mo, go;
    shiftav_layout(p, batch, max_pages_per_seq, S, GT, &zo, &mo, &go, out);
    return SA_OK;
}

extern "C" sa_status sa_decode_attention_shiftav(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q,
                                                 float* O, void* workspace, size_t workspace_bytes, int n_bits,
                                                 int k_max, int32_t* dbg_scores, int32_t* dbg_rounded,
                                                 sa_stream stream) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (p.fp16 || p.int8) return SA_ERR_UNSUPPORTED;
    // INT32 tile accumulator: 32 keys x 128 x 2^N < 2^31
    if (n_bits < 1 || n_bits > 18 || k_max < 0 || k_max > n_bits) return SA_ERR_INVALID_ARG;
    DecodeArgs a;
    int GT;
    st = make_decode_args(p, cache, Q, O, workspace, workspace_bytes, &a, &GT, false);   // statistics per (split, sequence)
    if (st != SA_OK) return st;
    size_t zo, mo, go, total;
    shiftav_layout(p, cache->batch, cache->max_pages_per_seq, a.n_splits, GT, &zo, &mo, &go, &total);
    if (workspace_bytes < total) return SA_ERR_CAPACITY;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return SA_ERR_ALIGNMENT;
    auto mis4 = [](const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 3) != 0; };
    if ((dbg_scores && mis4(dbg_scores)) || (dbg_rounded && mis4(dbg_rounded))) return SA_ERR_ALIGNMENT;
    char* ws = static_cast<char*>(workspace);
    a.dbg_scores = dbg_scores;
    a.zr = dbg_rounded ? dbg_rounded : reinterpret_cast<int32_t*>(ws + zo);
    a.stat_m = reinterpret_cast<int32_t*>(ws + mo);
    a.stat_g = reinterpret_cast<int32_t*>(ws + go);
    a.n_bits = n_bits;
    a.k_max = k_max;
    a.zscale = (float)(1.4426950408889634 / sqrt((double)p.d) / (double)(1LL << p.F));
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    launch_decode_main(p, a, GT, s);                             // pass 1: scores, rounded logits, statistics
    if (cudaGetLastError() != cudaSuccess) return SA_ERR_CUDA;
    const dim3 grid((unsigned)a.n_splits, (unsigned)(p.Hkv * (p.G / GT)), (unsigned)a.batch);
    if (p.d == 64) launch_shiftav_gt<64>(a, GT, grid, s);        // pass 2: shift-based A.V
    else launch_shiftav_gt<128>(a, GT, grid, s);
    if (cudaGetLastError() != cudaSuccess) return SA_ERR_CUDA;
    return launch_merge(p, a, s);
}
