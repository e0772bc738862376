// Cache-write side of the library: key encode, query and value quantisation, append, bulk
// fill and the unpack test hook.  One warp handles one head vector; lane l owns the
// head_dim / 32 consecutive elements starting at l * (head_dim / 32).
#include "sa_common.cuh"
#include "sa_cache_write.cuh"
#include "sa_quant.cuh"

namespace sa {

// -------------------------------------------------------------------------------------------
// sa_encode_keys: canonical bytes + scales.
// -------------------------------------------------------------------------------------------
template <int D, int K>
__global__ void __launch_bounds__(128) encode_keys_kernel(const uint16_t* __restrict__ Kin, int64_t n_vec,
                                                          uint8_t* __restrict__ codes,
                                                          uint16_t* __restrict__ scales, int hadamard) {
    constexpr int EPL = D / 32;
    const int lane = threadIdx.x & 31;
    const int64_t v = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (v >= n_vec) return;
    uint32_t bits[EPL];
    load_vec_bits<EPL>(Kin + v * D, lane, bits);
    uint8_t c[EPL];
    uint32_t smax;
    if constexpr (K == 8) smax = encode_key_int8_vec<EPL>(bits, lane, hadamard != 0, c);
    else smax = encode_key_vec<EPL, K>(bits, lane, hadamard != 0, c);
    store_bytes<EPL>(codes + v * D + lane * EPL, c);
    if (lane == 0) scales[v] = (uint16_t)smax;
}

// -------------------------------------------------------------------------------------------
// sa_quantise_query
// -------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(128) quantise_query_kernel(const uint16_t* __restrict__ Q, int64_t n_vec,
                                                             int8_t* __restrict__ qhat,
                                                             float* __restrict__ delta, int hadamard) {
    constexpr int EPL = D / 32;
    const int lane = threadIdx.x & 31;
    const int64_t v = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (v >= n_vec) return;
    uint32_t bits[EPL];
    load_vec_bits<EPL>(Q + v * D, lane, bits);
    int q[EPL];
    const float dl = quantise_query_vec<EPL>(bits, lane, hadamard != 0, q);
    uint8_t c[EPL];
#pragma unroll
    for (int i = 0; i < EPL; ++i) c[i] = (uint8_t)(int8_t)q[i];
    store_bytes<EPL>(reinterpret_cast<uint8_t*>(qhat) + v * D + lane * EPL, c);
    if (lane == 0) delta[v] = dl;
}

// -------------------------------------------------------------------------------------------
// sa_quantise_values
// -------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(128) quantise_values_kernel(const uint16_t* __restrict__ V, int64_t n_vec,
                                                              int8_t* __restrict__ vhat,
                                                              int8_t* __restrict__ g) {
    constexpr int EPL = D / 32;
    const int lane = threadIdx.x & 31;
    const int64_t v = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (v >= n_vec) return;
    uint32_t bits[EPL];
    load_vec_bits<EPL>(V + v * D, lane, bits);
    uint8_t c[EPL];
    const int gg = quantise_value_vec<EPL>(bits, c);
    store_bytes<EPL>(reinterpret_cast<uint8_t*>(vhat) + v * D + lane * EPL, c);
    if (lane == 0) g[v] = (int8_t)gg;
}

// sa_append_kv: one block per sequence; warps loop over the KV heads.
template <int D, int MODE>
__global__ void __launch_bounds__(128) append_kernel(CacheArgs a, const uint16_t* __restrict__ Knew,
                                                     const uint16_t* __restrict__ Vnew, int bump) {
    pdl_wait();                 // earlier kernels in the stream may still be reading this cache
    pdl_launch_dependents();
    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int len = a.seq_lens[b];
    const bool ok = len >= 0 && page_block(a, b, len / kPageTokens, 0) != nullptr;
    if (ok) {
        for (int h = warp; h < a.Hkv; h += 4) {
            uint8_t* block = page_block(a, b, len / kPageTokens, h);
            const size_t row = ((size_t)b * a.Hkv + h) * D;
            write_token<D, MODE>(block, a, len % kPageTokens, lane, Knew + row, Vnew + row);
        }
    }
    __syncthreads();   // every warp has read seq_lens[b] before it changes
    if (ok && bump && threadIdx.x == 0) a.seq_lens[b] = len + 1;
}

// sa_fill_kv: tokens row0 .. row0 + T - 1 of the flat K/V arrays are sequence b's tokens 0 .. T-1.
template <int D, int MODE>
__global__ void __launch_bounds__(128) fill_kernel(CacheArgs a, const uint16_t* __restrict__ Kin,
                                                   const uint16_t* __restrict__ Vin, int b, int64_t row0,
                                                   int T) {
    const int lane = threadIdx.x & 31;
    const int64_t v = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);   // (token, head) vector index
    if (v >= (int64_t)T * a.Hkv) return;
    const int t = (int)(v / a.Hkv), h = (int)(v % a.Hkv);
    uint8_t* block = page_block(a, b, t / kPageTokens, h);
    if (!block) return;
    const size_t row = ((size_t)(row0 + t) * a.Hkv + h) * D;
    write_token<D, MODE>(block, a, t % kPageTokens, lane, Kin + row, Vin + row);
}

// sa_debug_unpack
template <int D, bool NIB>
__global__ void __launch_bounds__(128) unpack_kernel(CacheArgs a, int b, int T, uint8_t xor_mask, int planes, uint8_t* __restrict__ codes,
                                                     uint16_t* __restrict__ scales, int8_t* __restrict__ vhat,
                                                     int8_t* __restrict__ g) {
    constexpr int EPL = D / 32;
    const int lane = threadIdx.x & 31;
    const int64_t v = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (v >= (int64_t)T * a.Hkv) return;
    const int tt = (int)(v / a.Hkv), h = (int)(v % a.Hkv);
    const uint8_t* block = page_block(a, b, tt / kPageTokens, h);
    if (!block) return;
    block += (size_t)((tt % kPageTokens) >> 5) * (a.page_bytes >> 1);      // the token's half of the page
    const int t = tt & 31;
    const int m = lane * EPL;
    if (codes) {
        uint8_t c[EPL];
        if (!NIB) {
            const uint8_t* src = block + a.kcode_off + ((size_t)(m >> 4) * kTileTokens + t) * 16 + (m & 15);
#pragma unroll
            for (int i = 0; i < EPL; ++i) c[i] = xor_mask ? canon_byte(src[i]) : src[i];   // power-of-two codes / INT8 stored as is
        } else {
            const uint8_t* src = block + a.kcode_off + ((size_t)(m >> 5) * kTileTokens + t) * 16 + ((m & 31) >> 1);
#pragma unroll
            for (int i = 0; i < EPL / 2; ++i) {
                c[2 * i] = (uint8_t)((src[i] << 4) ^ 0x70);
                c[2 * i + 1] = (uint8_t)((src[i] & 0xf0) ^ 0x70);
            }
            // dense planar container: the canonical mantissa is left-aligned in the low nibble
            for (int bit = 0; bit < planes; ++bit) {
                const uint8_t* pl = block + a.plane_off + ((size_t)bit * kTileTokens + t) * (D / 8);
#pragma unroll
                for (int i = 0; i < EPL; ++i) c[i] |= (uint8_t)(((pl[(m + i) >> 3] >> ((m + i) & 7)) & 1u) << (4 - planes + bit));
            }
        }
        store_bytes<EPL>(codes + (size_t)v * D + m, c);
    }
    if (vhat) {
        const uint8_t* src = block + a.v_off + ((size_t)(m >> 4) * kTileTokens + t) * 16 + (m & 15);
        uint8_t c[EPL];
#pragma unroll
        for (int i = 0; i < EPL; ++i) c[i] = src[i];
        store_bytes<EPL>(reinterpret_cast<uint8_t*>(vhat) + (size_t)v * D + m, c);
    }
    if (lane == 0) {
        const uint32_t meta = *reinterpret_cast<const uint32_t*>(block + a.meta_off + (size_t)t * 4);
        if (scales) scales[v] = (uint16_t)(meta & 0xffffu);
        if (g) g[v] = (int8_t)((meta >> 16) & 0xff);
    }
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

static sa_status check_cache(const Plan& p, const sa_cache* c, CacheArgs* a) {
    if (!c || !c->pages || !c->page_table || !c->seq_lens) return SA_ERR_INVALID_ARG;
    if (c->batch <= 0 || c->max_pages_per_seq <= 0 || c->n_pages <= 0) return SA_ERR_INVALID_ARG;
    if (!aligned(c->pages, p.lay.align) || !aligned(c->page_table, 4) || !aligned(c->seq_lens, 4))
        return SA_ERR_ALIGNMENT;
    a->pages = static_cast<uint8_t*>(c->pages);
    a->page_table = c->page_table;
    a->seq_lens = c->seq_lens;
    a->batch = c->batch;
    a->max_pages = c->max_pages_per_seq;
    a->n_pages = c->n_pages;
    a->Hkv = p.Hkv;
    a->page_bytes = p.lay.page_bytes;
    a->kcode_off = p.lay.kcode_off;
    a->meta_off = p.lay.meta_off;
    a->v_off = p.lay.v_off;
    a->plane_off = p.plane_off;
    a->hadamard = p.hadamard ? 1 : 0;
    return SA_OK;
}

static int mode_of(const Plan& p) { return p.fp16 ? 16 : (p.int8 ? 32 : (p.nibble ? 8 + p.k : p.k)); }

#define SA_LAUNCH_CHECK() (cudaGetLastError() == cudaSuccess ? SA_OK : SA_ERR_CUDA)

// Dispatch over (head_dim, storage mode).
#define SA_DISPATCH_D_MODE(p, CALL)                                                     \
    do {                                                                                \
        const int mode_ = mode_of(p);                                                   \
        if ((p).d == 64) {                                                              \
            switch (mode_) {                                                            \
                case 0: CALL(64, 0); break;                                             \
                case 1: CALL(64, 1); break;                                             \
                case 2: CALL(64, 2); break;                                             \
                case 4: CALL(64, 4); break;                                             \
                case 8: CALL(64, 8); break;                                             \
                case 9: CALL(64, 9); break;                                             \
                case 10: CALL(64, 10); break;                                           \
                case 32: CALL(64, 32); break;                                           \
                default: CALL(64, 16); break;                                           \
            }                                                                           \
        } else {                                                                        \
            switch (mode_) {                                                            \
                case 0: CALL(128, 0); break;                                            \
                case 1: CALL(128, 1); break;                                            \
                case 2: CALL(128, 2); break;                                            \
                case 4: CALL(128, 4); break;                                            \
                case 8: CALL(128, 8); break;                                            \
                case 9: CALL(128, 9); break;                                            \
                case 10: CALL(128, 10); break;                                          \
                case 32: CALL(128, 32); break;                                          \
                default: CALL(128, 16); break;                                          \
            }                                                                           \
        }                                                                               \
    } while (0)

}  // namespace sa

using namespace sa;

extern "C" {

sa_status sa_encode_keys(const sa_config* cfg, const uint16_t* K, int64_t n, uint8_t* codes,
                         uint16_t* scales, sa_stream stream) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (p.fp16) return SA_ERR_UNSUPPORTED;
    if (!K || !codes || !scales || n < 0) return SA_ERR_INVALID_ARG;
    if (!aligned(K, 16) || !aligned(codes, 16) || !aligned(scales, 2)) return SA_ERR_ALIGNMENT;
    const int64_t n_vec = n * p.Hkv;
    if (n_vec == 0) return SA_OK;
    if ((n_vec + 3) / 4 > 0x7fffffffLL) return SA_ERR_CAPACITY;
    const unsigned grid = (unsigned)((n_vec + 3) / 4);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int had = p.hadamard ? 1 : 0;
#define CALL(D, KK) encode_keys_kernel<D, KK><<<grid, 128, 0, s>>>(K, n_vec, codes, scales, had)
    if (p.int8) {
        if (p.d == 64) CALL(64, 8);
        else CALL(128, 8);
    } else if (p.d == 64) {
        switch (p.k) { case 0: CALL(64, 0); break; case 1: CALL(64, 1); break; case 2: CALL(64, 2); break; default: CALL(64, 4); }
    } else {
        switch (p.k) { case 0: CALL(128, 0); break; case 1: CALL(128, 1); break; case 2: CALL(128, 2); break; default: CALL(128, 4); }
    }
#undef CALL
    return SA_LAUNCH_CHECK();
}

sa_status sa_quantise_query(const sa_config* cfg, const uint16_t* Q, int batch, int8_t* q_hat,
                            float* delta, sa_stream stream) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (!Q || !q_hat || !delta || batch < 0) return SA_ERR_INVALID_ARG;
    if (!aligned(Q, 16) || !aligned(q_hat, 16) || !aligned(delta, 4)) return SA_ERR_ALIGNMENT;
    const int64_t n_vec = (int64_t)batch * p.Hq;
    if (n_vec == 0) return SA_OK;
    const unsigned grid = (unsigned)((n_vec + 3) / 4);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int had = (p.hadamard && !p.fp16) ? 1 : 0;
    if (p.d == 64) quantise_query_kernel<64><<<grid, 128, 0, s>>>(Q, n_vec, q_hat, delta, had);
    else quantise_query_kernel<128><<<grid, 128, 0, s>>>(Q, n_vec, q_hat, delta, had);
    return SA_LAUNCH_CHECK();
}

sa_status sa_quantise_values(const sa_config* cfg, const uint16_t* V, int64_t n, int8_t* v_hat,
                             int8_t* g, sa_stream stream) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (!V || !v_hat || !g || n < 0) return SA_ERR_INVALID_ARG;
    if (!aligned(V, 16) || !aligned(v_hat, 16)) return SA_ERR_ALIGNMENT;
    const int64_t n_vec = n * p.Hkv;
    if (n_vec == 0) return SA_OK;
    if ((n_vec + 3) / 4 > 0x7fffffffLL) return SA_ERR_CAPACITY;
    const unsigned grid = (unsigned)((n_vec + 3) / 4);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (p.d == 64) quantise_values_kernel<64><<<grid, 128, 0, s>>>(V, n_vec, v_hat, g);
    else quantise_values_kernel<128><<<grid, 128, 0, s>>>(V, n_vec, v_hat, g);
    return SA_LAUNCH_CHECK();
}

sa_status sa_append_kv(const sa_config* cfg, const sa_cache* cache, const uint16_t* K_new,
                       const uint16_t* V_new, int bump_lens, sa_stream stream) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    CacheArgs a;
    st = check_cache(p, cache, &a);
    if (st != SA_OK) return st;
    if (!K_new || !V_new) return SA_ERR_INVALID_ARG;
    if (!aligned(K_new, 16) || !aligned(V_new, 16)) return SA_ERR_ALIGNMENT;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
#define CALL(D, M) (void)launch_pdl(append_kernel<D, M>, dim3(a.batch), dim3(128), 0, s, a, K_new, V_new, bump_lens)
    SA_DISPATCH_D_MODE(p, CALL);
#undef CALL
    return SA_LAUNCH_CHECK();
}

sa_status sa_fill_kv(const sa_config* cfg, const sa_cache* cache, const uint16_t* K, const uint16_t* V,
                     const int64_t* cu_lens_host, sa_stream stream) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    CacheArgs a;
    st = check_cache(p, cache, &a);
    if (st != SA_OK) return st;
    if (!cu_lens_host) return SA_ERR_INVALID_ARG;
    for (int b = 0; b < a.batch; ++b) {
        const int64_t T = cu_lens_host[b + 1] - cu_lens_host[b];
        if (T < 0 || cu_lens_host[b] < 0) return SA_ERR_INVALID_ARG;
        if (T > (int64_t)a.max_pages * kPageTokens) return SA_ERR_CAPACITY;
    }
    if (cu_lens_host[a.batch] == cu_lens_host[0]) return SA_OK;   // nothing to write
    if (!K || !V) return SA_ERR_INVALID_ARG;
    if (!aligned(K, 16) || !aligned(V, 16)) return SA_ERR_ALIGNMENT;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    for (int b = 0; b < a.batch; ++b) {
        const int64_t row0 = cu_lens_host[b];
        const int T = (int)(cu_lens_host[b + 1] - row0);
        if (T == 0) continue;
        const unsigned grid = (unsigned)(((int64_t)T * a.Hkv + 3) / 4);
#define CALL(D, M) fill_kernel<D, M><<<grid, 128, 0, s>>>(a, K, V, b, row0, T)
        SA_DISPATCH_D_MODE(p, CALL);
#undef CALL
        if (cudaGetLastError() != cudaSuccess) return SA_ERR_CUDA;
    }
    return SA_OK;
}

sa_status sa_debug_unpack(const sa_config* cfg, const sa_cache* cache, int b, int n_tokens,
                          uint8_t* codes, uint16_t* scales, int8_t* v_hat, int8_t* g, sa_stream stream) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (p.fp16) return SA_ERR_UNSUPPORTED;
    CacheArgs a;
    st = check_cache(p, cache, &a);
    if (st != SA_OK) return st;
    if (b < 0 || b >= a.batch || n_tokens < 0) return SA_ERR_INVALID_ARG;
    if (n_tokens > a.max_pages * kPageTokens) return SA_ERR_CAPACITY;
    if ((codes && !aligned(codes, 16)) || (v_hat && !aligned(v_hat, 16))) return SA_ERR_ALIGNMENT;
    if (n_tokens == 0) return SA_OK;
    const unsigned grid = (unsigned)(((int64_t)n_tokens * a.Hkv + 3) / 4);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const uint8_t xm = p.int8 ? 0x00 : 0x70;
    const int pl = p.nibble ? p.k : 0;                         // mantissa bit planes of the dense planar container
    if (p.d == 64) {
        if (p.nibble) unpack_kernel<64, true><<<grid, 128, 0, s>>>(a, b, n_tokens, xm, pl, codes, scales, v_hat, g);
        else unpack_kernel<64, false><<<grid, 128, 0, s>>>(a, b, n_tokens, xm, pl, codes, scales, v_hat, g);
    } else {
        if (p.nibble) unpack_kernel<128, true><<<grid, 128, 0, s>>>(a, b, n_tokens, xm, pl, codes, scales, v_hat, g);
        else unpack_kernel<128, false><<<grid, 128, 0, s>>>(a, b, n_tokens, xm, pl, codes, scales, v_hat, g);
    }
    return SA_LAUNCH_CHECK();
}

}  // extern "C"
