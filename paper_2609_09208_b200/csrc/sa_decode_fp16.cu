// Decode attention over an unquantised binary16 cache: softmax(Q K^T / sqrt(d)) V of eq. (1)
// with FP32 accumulation.  Same grid, tiling, online softmax and merges as the quantised kernel,
// so that the throughput ratio between the two isolates the key/value representation.
#include "sa_common.cuh"
#include "sa_decode_common.cuh"
#include "sa_quant.cuh"

namespace sa {

template <int D, int GT>
__global__ void __launch_bounds__(128) decode_fp16_kernel(DecodeArgs a) {
    constexpr int EPL = D / 32;
    constexpr int CH = D / 8;                      // 16-byte chunks (8 binary16) per key
    constexpr int LPT = D / 8;
    constexpr int TS = 32 / LPT;
    constexpr int TPL = 32 / TS;
    __shared__ __align__(16) float q_s[D][GT];     // query times log2(e) / sqrt(d)
    __shared__ __align__(16) float2 p_s[4][32][GT];
    __shared__ __align__(16) float red_s[4][GT][D + 2];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chunks = a.G / GT;
    const int kvh = blockIdx.y / chunks;
    const int h0 = kvh * a.G + (blockIdx.y % chunks) * GT;
    const int b = blockIdx.z;
    const int split = blockIdx.x;

    for (int g = warp; g < GT; g += 4) {
        uint32_t bits[EPL];
        load_vec_bits<EPL>(a.Q + ((size_t)b * a.Hq + h0 + g) * D, lane, bits);
#pragma unroll
        for (int i = 0; i < EPL; ++i) q_s[lane * EPL + i][g] = half_bits_to_float(bits[i]) * a.zscale;
    }
    __syncthreads();

    const int len = a.seq_lens[b];
    const int n_tiles = (min(len, a.max_pages * kPageTokens) + 31) >> 5;
    const int tile0 = (int)((long long)n_tiles * split / a.n_splits);
    const int tile1 = (int)((long long)n_tiles * (split + 1) / a.n_splits);

    int M[GT];
    float l[GT];
    unsigned long long acc[GT][4];
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        M[g] = kMNone;
        l[g] = 0.0f;
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[g][j] = 0ull;
    }
    const int ts = lane / LPT, dc = lane % LPT;

    for (int tile = tile0 + warp; tile < tile1; tile += 4) {
        const int lp = tile >> 1;
        const int tk0 = (tile & 1) * 32;
        const int n_valid = min(32, len - tile * 32);
        const int pidx = a.page_table[(size_t)b * a.max_pages + lp];
        if (pidx < 0 || pidx >= a.n_pages) continue;
        const uint8_t* block = a.pages + ((size_t)pidx * a.Hkv + kvh) * a.page_bytes;

        // ---- scores, lane = key ----
        float z[GT];
#pragma unroll
        for (int g = 0; g < GT; ++g) z[g] = 0.0f;
#pragma unroll 4
        for (int c = 0; c < CH; ++c) {
            const uint4 w = __ldg(reinterpret_cast<const uint4*>(block + a.kcode_off + ((size_t)c * kPageTokens + tk0 + lane) * 16));
            const uint32_t w4[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int wi = 0; wi < 4; ++wi) {
                const float2 kf = __half22float2(*reinterpret_cast<const __half2*>(&w4[wi]));
                const int m = c * 8 + wi * 2;
                const float4* q0 = reinterpret_cast<const float4*>(&q_s[m][0]);
                const float4* q1 = reinterpret_cast<const float4*>(&q_s[m + 1][0]);
                if constexpr (GT >= 4) {
#pragma unroll
                    for (int i = 0; i < GT / 4; ++i) {
                        const float4 a0 = q0[i], a1 = q1[i];
                        z[4 * i + 0] = fmaf(a0.x, kf.x, z[4 * i + 0]); z[4 * i + 0] = fmaf(a1.x, kf.y, z[4 * i + 0]);
                        z[4 * i + 1] = fmaf(a0.y, kf.x, z[4 * i + 1]); z[4 * i + 1] = fmaf(a1.y, kf.y, z[4 * i + 1]);
                        z[4 * i + 2] = fmaf(a0.z, kf.x, z[4 * i + 2]); z[4 * i + 2] = fmaf(a1.z, kf.y, z[4 * i + 2]);
                        z[4 * i + 3] = fmaf(a0.w, kf.x, z[4 * i + 3]); z[4 * i + 3] = fmaf(a1.w, kf.y, z[4 * i + 3]);
                    }
                } else {
#pragma unroll
                    for (int g = 0; g < GT; ++g) {
                        z[g] = fmaf(q_s[m][g], kf.x, z[g]);
                        z[g] = fmaf(q_s[m + 1][g], kf.y, z[g]);
                    }
                }
            }
        }

        // ---- online softmax with an integer running maximum ----
        const bool valid = lane < n_valid;
        bool changed = false;
        float resc[GT];
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            const float zz = valid ? z[g] : -INFINITY;
            const float zmax = warp_max_f32(zz);
            const int Mt = (int)ceilf(fminf(fmaxf(zmax, -1.0e8f), 1.0e8f));
            const int Mn = max(M[g], Mt);
            resc[g] = (M[g] == kMNone) ? 0.0f : pow2i_neg(M[g] - Mn);
            changed |= (Mn != M[g]);
            M[g] = Mn;
            const float p = valid ? ex2_approx(zz - (float)Mn) : 0.0f;
            l[g] = l[g] * resc[g] + p;
            p_s[warp][lane][g] = make_float2(p, p);
        }
        if (changed) {
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                const unsigned long long r2 = pack_f32x2(resc[g], resc[g]);
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[g][j] = ffma2(acc[g][j], r2, 0ull);
            }
        }
        __syncwarp();

        // ---- O += p * V, lane = (token group, 8 dims) ----
        const uint8_t* vbase = block + a.v_off + ((size_t)tk0 * D + dc * 8) * 2;
#pragma unroll 4
        for (int i = 0; i < TPL; ++i) {
            const int t = ts + TS * i;
            uint4 vv = __ldg(reinterpret_cast<const uint4*>(vbase + (size_t)t * D * 2));
            if (t >= n_valid) vv = make_uint4(0u, 0u, 0u, 0u);   // unwritten slots may hold non-finite bit patterns
            const uint32_t v4[4] = {vv.x, vv.y, vv.z, vv.w};
            unsigned long long v2[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&v4[j]));
                v2[j] = pack_f32x2(f.x, f.y);
            }
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                const unsigned long long pp = *reinterpret_cast<const unsigned long long*>(&p_s[warp][t][g]);
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[g][j] = ffma2(v2[j], pp, acc[g][j]);
            }
        }
        __syncwarp();
    }

    block_merge_and_store<D, GT, 4>(a, red_s, M, l, acc, lane, warp, ts, dc, LPT, b, h0, split);
}

}  // namespace sa

using namespace sa;

template <int D>
static void launch_fp16(const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s) {
    switch (GT) {
        case 8: decode_fp16_kernel<D, 8><<<grid, 128, 0, s>>>(a); break;
        case 4: decode_fp16_kernel<D, 4><<<grid, 128, 0, s>>>(a); break;
        case 2: decode_fp16_kernel<D, 2><<<grid, 128, 0, s>>>(a); break;
        default: decode_fp16_kernel<D, 1><<<grid, 128, 0, s>>>(a); break;
    }
}

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
        const dim3 grid((unsigned)a.n_splits, (unsigned)(p.Hkv * (p.G / GT)), (unsigned)a.batch);
        if (p.d == 64) launch_fp16<64>(a, GT, grid, s);
        else launch_fp16<128>(a, GT, grid, s);
        if (cudaGetLastError() != cudaSuccess) return SA_ERR_CUDA;
    }
    return (stages & 2) ? launch_merge(p, a, s) : SA_OK;
}

extern "C" sa_status sa_decode_attention_fp16(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q,
                                              float* O, void* workspace, size_t workspace_bytes,
                                              sa_stream stream) {
    return sa_decode_attention_fp16_stages(cfg, cache, Q, O, workspace, workspace_bytes, 3, stream);
}
