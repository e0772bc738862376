// Host side of the C ABI: configuration validation, page layout, split plan, and the
// host-buffer convenience entry.  No kernels live here.
#include "sa_decode_common.cuh"
#include <cmath>

namespace sa {

sa_status make_plan(const sa_config* cfg, Plan* out) {
    if (!cfg || !out) return SA_ERR_INVALID_ARG;
    Plan p{};
    if (cfg->n_q_heads <= 0 || cfg->n_kv_heads <= 0 || cfg->n_q_heads % cfg->n_kv_heads != 0)
        return SA_ERR_INVALID_ARG;
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return SA_ERR_UNSUPPORTED;
    if (cfg->page_tokens != kPageTokens) return SA_ERR_UNSUPPORTED;
    if (cfg->flags & ~(SA_FLAG_HADAMARD | SA_FLAG_SHIFT_BY_MULTIPLY | SA_FLAG_ADD_ON_ALU)) return SA_ERR_INVALID_ARG;
    p.mulshift = (cfg->flags & SA_FLAG_SHIFT_BY_MULTIPLY) != 0;
    p.addalu = (cfg->flags & SA_FLAG_ADD_ON_ALU) != 0;
    if (p.mulshift && p.addalu) return SA_ERR_INVALID_ARG;
    if (p.addalu && (cfg->code == SA_KV_FP16 || cfg->code == SA_INT8)) return SA_ERR_UNSUPPORTED;   // no shift-and-add datapath there
    // no shift in the key loop to move: FP16 and INT8 have none, PoT-4 looks its shifted queries up
    if (p.mulshift && (cfg->code == SA_KV_FP16 || cfg->code == SA_INT8 || cfg->code == SA_POT4)) return SA_ERR_UNSUPPORTED;
    p.d = cfg->head_dim;
    p.Hq = cfg->n_q_heads;
    p.Hkv = cfg->n_kv_heads;
    p.G = p.Hq / p.Hkv;
    p.hadamard = (cfg->flags & SA_FLAG_HADAMARD) != 0;
    p.fp16 = (cfg->code == SA_KV_FP16);
    if (p.fp16) {
        if (cfg->klayout != SA_KLAYOUT_BYTE) return SA_ERR_UNSUPPORTED;
        if (p.hadamard) return SA_ERR_UNSUPPORTED;   // the rotation is a pre-quantisation transform
        p.k = 0;
        p.nibble = false;
        p.F = 0;
        p.f_extra = 0;
        p.lay.kcode_off = 0;
        p.lay.meta_off = (size_t)kTileTokens * p.d * 2;   // empty metadata block
        p.lay.v_off = p.lay.meta_off;
        p.lay.page_bytes = 2 * (p.lay.v_off + (size_t)kTileTokens * p.d * 2);
        if (p.lay.page_bytes != 2 * (size_t)half_block_bytes_fp16(p.d)) return SA_ERR_UNSUPPORTED;
        p.lay.align = 256;
        *out = p;
        return SA_OK;
    }
    if (cfg->code == SA_INT8) {
        if (cfg->klayout != SA_KLAYOUT_BYTE || cfg->headroom_F != 0) return SA_ERR_UNSUPPORTED;
        p.int8 = true;
        p.k = 0;
        p.F = 0;
        p.f_extra = 0;
        p.lay.kcode_off = 0;
        p.lay.meta_off = (size_t)kTileTokens * p.d;
        p.lay.v_off = p.lay.meta_off + (size_t)kTileTokens * 4;
        p.lay.page_bytes = 2 * (p.lay.v_off + (size_t)kTileTokens * p.d);
        if (p.lay.page_bytes != 2 * (size_t)half_block_bytes(p.d, 8, false)) return SA_ERR_UNSUPPORTED;
        p.lay.align = 256;
        *out = p;
        return SA_OK;
    }
    if (cfg->code != SA_POT4 && cfg->code != SA_POTM1 && cfg->code != SA_POTM2 && cfg->code != SA_POTM4)
        return SA_ERR_UNSUPPORTED;
    p.k = cfg->code;
    if (cfg->klayout == SA_KLAYOUT_NIBBLE) {
        if (p.k != 0) return SA_ERR_UNSUPPORTED;
        p.nibble = true;
    } else if (cfg->klayout == SA_KLAYOUT_PLANAR) {
        if (p.k != 1 && p.k != 2) return SA_ERR_UNSUPPORTED;    // 5 and 6 bits per element; 4 and 8 are dense already
        p.nibble = true;
    } else if (cfg->klayout != SA_KLAYOUT_BYTE) {
        return SA_ERR_UNSUPPORTED;
    }
    p.F = cfg->headroom_F == 0 ? kEmax + p.k : cfg->headroom_F;
    if (p.F < kEmax + p.k) return SA_ERR_UNSUPPORTED;           // eq. (4): left shifts only
    if (p.F - p.k > 24) return SA_ERR_UNSUPPORTED;
    // INT32 accumulator bound: d * 127 * (2^(k+1) - 1) * 2^(F - k) < 2^31
    const long long bound = (long long)p.d * 127 * ((1LL << (p.k + 1)) - 1) * (1LL << (p.F - p.k));
    if (bound >= (1LL << 31)) return SA_ERR_UNSUPPORTED;
    p.f_extra = p.F - p.k - kEmax;
    const size_t kbytes = p.nibble ? (size_t)p.d / 2 : (size_t)p.d;
    // offsets within one 32-token half of the block; the second half follows the first
    p.lay.kcode_off = 0;
    p.plane_off = (size_t)kTileTokens * kbytes;                 // k bit planes of d / 8 bytes per token (planar only)
    p.lay.meta_off = p.plane_off + (p.nibble ? (size_t)p.k * kTileTokens * (p.d / 8) : 0);
    p.lay.v_off = p.lay.meta_off + (size_t)kTileTokens * 4;
    p.lay.page_bytes = 2 * (p.lay.v_off + (size_t)kTileTokens * p.d);
    if (p.lay.page_bytes != 2 * (size_t)half_block_bytes(p.d, p.k, p.nibble)) return SA_ERR_UNSUPPORTED;   // the kernels' stage plans
    p.lay.align = 256;
    *out = p;
    return SA_OK;
}

int sm_count() {
    static int cached[64] = {};                               // 0: not asked yet (benign race: every thread stores the same value)
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        (void)cudaGetLastError();
        return kNumSMsB200;
    }
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            n = kNumSMsB200;
        }
        cached[dev] = n;
    }
    return cached[dev];
}

void split_plan(const Plan& p, int batch, int max_pages, int* n_splits, int* gt) {
    int GT = 1;
    for (int c = 8; c >= 1; c >>= 1)
        if (p.G % c == 0) { GT = c; break; }
    // One thread block per (split, KV head x query chunk, sequence); its warps take the 32-key
    // tiles of the block's slice in turn.  S is chosen by a small cost model of the
    // launch, fitted to measured sweeps over S, in units of one tile per warp on a full SM:
    //   * a block lasts about  r + c_fix  with r between tiles / (warps S) and its ceiling (warps that
    //     run out of tiles leave their issue slots to the others, but not all of the time), and
    //     c_fix for the prologue (query quantisation, table) and the block merge;
    //   * blocks run in waves of (SMs of the current device) x resident-blocks-per-SM; a last wave whose SMs hold only the
    //     fraction f of that takes 0.1 + 0.9 f of a full wave's time, a single partial wave f^0.2
    //     (an SM's throughput falls almost in proportion to its resident warps).
    // The sequence lengths live on the device, so the model uses the cache's capacity.
    const long long units = (long long)batch * p.Hkv * (p.G / GT);
    const KernelShape shape = p.fp16 ? kFp16Shape : decode_shape(p.d, p.int8 ? 8 : p.k);
    const int bps = shape.blocks_per_sm, nw = shape.warps;
    const int n_sms = sm_count();
    const long long slots = (long long)n_sms * bps;
    const long long tiles = (long long)max_pages * (kPageTokens / 32);
    long long cap = tiles / 2;                      // at least two tiles per block (short caches: spread them over the SMs)
    if (cap < 1) cap = 1;
    if (cap > 512) cap = 512;
    const double c_fix = 0.5;
    double best = 0.0;
    long long best_S = 1;
    for (long long S = 1; S <= cap; ++S) {
        const long long blocks = units * S;
        const double per_warp = (double)tiles / (double)(nw * S);
        const double block_time = 0.5 * (per_warp + (double)(((tiles + S - 1) / S + nw - 1) / nw)) + c_fix;
        const long long full = blocks / slots, rest = blocks % slots;
        double cost = (double)full * block_time;
        if (rest) {
            const double fill = (double)((rest + n_sms - 1) / n_sms) / (double)bps;
            // behind full waves a partial one overlaps their stragglers; on its own it does not
            cost += block_time * (full ? 0.1 + 0.9 * fill : pow(fill, 0.2));
        }
        if (S == 1 || cost < best * 0.999) {        // ties go to the smaller S (less merge work)
            best = cost;
            best_S = S;
        }
        if (blocks > 16 * slots) break;             // more waves than this never pay
    }
    *n_splits = (int)best_S;
    *gt = GT;
}

// Inputs of one decode step from device-addressable pinned host memory into the staging buffer.
__global__ void __launch_bounds__(256) stage_in_kernel(const uint4* __restrict__ q, const uint4* __restrict__ k,
                                                       const uint4* __restrict__ v, uint4* __restrict__ dq,
                                                       uint4* __restrict__ dk, uint4* __restrict__ dv, int nq, int nkv) {
    // The inputs sit in host memory that no kernel writes, so they are fetched before the wait and the trip over the
    // bus runs beside the step before; that step may still read the staging buffer, so the stores come after the
    // wait.  The kernel after this one (the decode kernel in its wait-first form, or the append kernel, which waits
    // before anything else) may be scheduled at once: neither reads the staging buffer before its own wait.
    pdl_launch_dependents();
    const int i = blockIdx.x * 256 + threadIdx.x;
    const uint4* src = nullptr;
    uint4* dst = nullptr;
    if (i < nq) {
        src = q + i;
        dst = dq + i;
    } else if (i < nq + nkv) {
        src = k + (i - nq);
        dst = dk + (i - nq);
    } else if (i < nq + 2 * nkv) {
        src = v + (i - nq - nkv);
        dst = dv + (i - nq - nkv);
    }
    uint4 x = make_uint4(0u, 0u, 0u, 0u);
    if (src) x = __ldcv(src);             // host memory: never from a cache line of an earlier step
    pdl_wait();
    if (dst) *dst = x;
}

}  // namespace sa

using namespace sa;

extern "C" {

int sa_version(void) { return 1; }

const char* sa_status_string(sa_status s) {
    switch (s) {
        case SA_OK: return "ok";
        case SA_ERR_INVALID_ARG: return "invalid argument";
        case SA_ERR_UNSUPPORTED: return "unsupported configuration";
        case SA_ERR_ALIGNMENT: return "misaligned pointer";
        case SA_ERR_CAPACITY: return "buffer too small";
        case SA_ERR_CUDA: return "CUDA runtime error";
    }
    return "unknown status";
}

sa_status sa_get_layout(const sa_config* cfg, sa_layout* out) {
    if (!out) return SA_ERR_INVALID_ARG;
    Plan p;
    const sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    *out = p.lay;
    return SA_OK;
}

sa_status sa_workspace_bytes(const sa_config* cfg, int batch, int max_pages_per_seq, size_t* out) {
    if (!out || batch <= 0 || max_pages_per_seq <= 0) return SA_ERR_INVALID_ARG;
    Plan p;
    const sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    int S, GT;
    split_plan(p, batch, max_pages_per_seq, &S, &GT);
    *out = decode_workspace_bytes(p, batch, S);
    return SA_OK;
}

sa_status sa_staging_bytes(const sa_config* cfg, int batch, size_t* out) {
    if (!out || batch <= 0) return SA_ERR_INVALID_ARG;
    Plan p;
    const sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    const size_t q = (size_t)batch * p.Hq * p.d * 2;
    const size_t kv = (size_t)batch * p.Hkv * p.d * 2;
    const size_t o = (size_t)batch * p.Hq * p.d * 4;
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    *out = up(q) + 2 * up(kv) + up(o);
    return SA_OK;
}

sa_status sa_decode_step_host(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q_host,
                              const uint16_t* K_new_host, const uint16_t* V_new_host, float* O_host,
                              void* staging, size_t staging_bytes, void* workspace,
                              size_t workspace_bytes, sa_stream stream) {
    if (!cache || !Q_host || !K_new_host || !V_new_host || !O_host || !staging) return SA_ERR_INVALID_ARG;
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (cache->batch <= 0) return SA_ERR_INVALID_ARG;
    size_t need;
    st = sa_staging_bytes(cfg, cache->batch, &need);
    if (st != SA_OK) return st;
    if (staging_bytes < need) return SA_ERR_CAPACITY;
    if (reinterpret_cast<uintptr_t>(staging) & 255) return SA_ERR_ALIGNMENT;
    size_t ws_need;
    st = sa_workspace_bytes(cfg, cache->batch, cache->max_pages_per_seq, &ws_need);
    if (st != SA_OK) return st;
    if (!workspace || workspace_bytes < ws_need) return SA_ERR_CAPACITY;
    const size_t q = (size_t)cache->batch * p.Hq * p.d * 2;
    const size_t kv = (size_t)cache->batch * p.Hkv * p.d * 2;
    const size_t o = (size_t)cache->batch * p.Hq * p.d * 4;
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    char* base = static_cast<char*>(staging);
    uint16_t* dQ = reinterpret_cast<uint16_t*>(base);
    uint16_t* dK = reinterpret_cast<uint16_t*>(base + up(q));
    uint16_t* dV = reinterpret_cast<uint16_t*>(base + up(q) + up(kv));
    float* dO = reinterpret_cast<float*>(base + up(q) + 2 * up(kv));
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // Pinned host buffers that the device can address directly need no copy engine at all: a small kernel
    // fetches the inputs (a few KB) and the merge kernel stores O straight into host memory.  A copy node
    // costs several microseconds of stream time, which is most of such a step at batch 1.
    void *mq = nullptr, *mk = nullptr, *mv = nullptr, *mo = nullptr;
    const bool mapped = cudaHostGetDevicePointer(&mq, const_cast<uint16_t*>(Q_host), 0) == cudaSuccess &&
                        cudaHostGetDevicePointer(&mk, const_cast<uint16_t*>(K_new_host), 0) == cudaSuccess &&
                        cudaHostGetDevicePointer(&mv, const_cast<uint16_t*>(V_new_host), 0) == cudaSuccess &&
                        cudaHostGetDevicePointer(&mo, O_host, 0) == cudaSuccess;
    (void)cudaGetLastError();                                    // a pageable buffer is not an error here
    auto al16 = [](const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15) == 0; };
    const bool direct = mapped && al16(mq) && al16(mk) && al16(mv) && al16(mo) && q % 16 == 0 && kv % 16 == 0;
    {
        // everything sa_decode_step will check, checked before a kernel or a copy is enqueued: a call that
        // returns an error has launched nothing
        DecodeArgs probe;
        int gt_probe;
        st = make_decode_args(p, cache, dQ, direct ? static_cast<float*>(mo) : dO, workspace, workspace_bytes, &probe, &gt_probe);
        if (st != SA_OK) return st;
    }
    if (direct) {
        const int nq = (int)(q / 16), nkv = (int)(kv / 16);
        const unsigned blocks = (unsigned)((nq + 2 * nkv + 255) / 256);
        if (launch_pdl(stage_in_kernel, dim3(blocks), dim3(256), 0, s, (const uint4*)mq, (const uint4*)mk, (const uint4*)mv,
                       (uint4*)dQ, (uint4*)dK, (uint4*)dV, nq, nkv) != cudaSuccess || cudaGetLastError() != cudaSuccess)
            return SA_ERR_CUDA;
        return decode_step_impl(cfg, cache, dQ, dK, dV, static_cast<float*>(mo), workspace, workspace_bytes, stream, true);
    }
    const char* hq = reinterpret_cast<const char*>(Q_host);
    if (up(q) == q && up(kv) == kv && reinterpret_cast<const char*>(K_new_host) == hq + q &&
        reinterpret_cast<const char*>(V_new_host) == hq + q + kv) {
        // the three inputs follow one another on the host exactly as in the staging buffer: one copy
        if (cudaMemcpyAsync(dQ, Q_host, q + 2 * kv, cudaMemcpyHostToDevice, s) != cudaSuccess) return SA_ERR_CUDA;
    } else {
        if (cudaMemcpyAsync(dQ, Q_host, q, cudaMemcpyHostToDevice, s) != cudaSuccess) return SA_ERR_CUDA;
        if (cudaMemcpyAsync(dK, K_new_host, kv, cudaMemcpyHostToDevice, s) != cudaSuccess) return SA_ERR_CUDA;
        if (cudaMemcpyAsync(dV, V_new_host, kv, cudaMemcpyHostToDevice, s) != cudaSuccess) return SA_ERR_CUDA;
    }
    st = sa_decode_step(cfg, cache, dQ, dK, dV, dO, workspace, workspace_bytes, stream);
    if (st != SA_OK) return st;
    if (cudaMemcpyAsync(O_host, dO, o, cudaMemcpyDeviceToHost, s) != cudaSuccess) return SA_ERR_CUDA;
    return SA_OK;
}

}  // extern "C"
