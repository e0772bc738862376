// Entry points of the decode path: argument checks, the split plan, and the dispatch to the decode
// kernel's instantiations (sa_decode_kernel.cuh; one translation unit per key code) and the split-K merge.
#include "sa_decode_kernel.cuh"

using namespace sa;

namespace sa {
void launch_decode_fp16_main(const Plan& p, const DecodeArgs& a, int GT, cudaStream_t s);   // sa_decode_fp16.cu
// The decode kernel for these arguments (the score pass of the shift-A.V option when a.zr is set).
void launch_decode_main(const Plan& p, const DecodeArgs& a, int GT, cudaStream_t s) {
    const dim3 grid((unsigned)a.n_splits, (unsigned)(p.Hkv * (p.G / GT)), (unsigned)a.batch);
    const int mode = a.zr ? 2 : (p.mulshift ? 1 : (p.addalu ? 3 : 0));   // a.zr: score pass of the shift-based A.V option
    if (p.int8) launch_decode_int8(p.d, a, GT, grid, s);
    else if (p.k == 0) launch_decode_pot4(p.nibble, p.d, mode, a, GT, grid, s);
    else if (p.k == 1) launch_decode_potm1(p.nibble, p.d, mode, a, GT, grid, s);
    else if (p.k == 2) launch_decode_potm2(p.nibble, p.d, mode, a, GT, grid, s);
    else launch_decode_potm4(p.d, mode, a, GT, grid, s);
}
}  // namespace sa

extern "C" sa_status sa_decode_attention_stages(const sa_config* cfg, const sa_cache* cache,
                                                const uint16_t* Q, float* O, void* workspace,
                                                size_t workspace_bytes, int32_t* dbg_scores, int stages,
                                                sa_stream stream) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (p.fp16) return SA_ERR_UNSUPPORTED;
    if ((stages & ~3) || stages == 0) return SA_ERR_INVALID_ARG;
    DecodeArgs a;
    int GT;
    st = make_decode_args(p, cache, Q, O, workspace, workspace_bytes, &a, &GT);
    if (st != SA_OK) return st;
    if (dbg_scores && (reinterpret_cast<uintptr_t>(dbg_scores) & 3)) return SA_ERR_ALIGNMENT;
    a.dbg_scores = dbg_scores;
    // logits in the log2 domain: A * Delta * s * 2^-F * log2(e) / sqrt(d)
    a.zscale = (float)(1.4426950408889634 / sqrt((double)p.d) / (double)(1LL << p.F));
    if (p.int8) a.zscale = (float)(1.4426950408889634 / sqrt((double)p.d) / 127.0);   // key unit = scale / 127
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (stages & 1) {
        launch_decode_main(p, a, GT, s);
        if (cudaGetLastError() != cudaSuccess) return SA_ERR_CUDA;
    }
    return (stages & 2) ? launch_merge(p, a, s) : SA_OK;
}

extern "C" sa_status sa_debug_decode_lost_copy(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q, float* O,
                                               void* workspace, size_t workspace_bytes, int b, int kv_head, int tile,
                                               sa_stream stream) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (p.fp16 || p.int8 || p.nibble || p.d != 64 || p.k != 4 || p.G != 8 || p.mulshift || p.addalu) return SA_ERR_UNSUPPORTED;
    DecodeArgs a;
    int GT;
    st = make_decode_args(p, cache, Q, O, workspace, workspace_bytes, &a, &GT);
    if (st != SA_OK) return st;
    if (b < 0 || b >= a.batch || kv_head < 0 || kv_head >= p.Hkv || tile < 0) return SA_ERR_INVALID_ARG;
    a.zscale = (float)(1.4426950408889634 / sqrt((double)p.d) / (double)(1LL << p.F));
    a.lost_b = b;
    a.lost_kvh = kv_head;
    a.lost_tile = tile;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    launch_decode_potm4_lost_copy(a, dim3((unsigned)a.n_splits, (unsigned)p.Hkv, (unsigned)a.batch), s);
    if (cudaGetLastError() != cudaSuccess) return SA_ERR_CUDA;
    return launch_merge(p, a, s);
}

extern "C" sa_status sa_decode_step(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q,
                                    const uint16_t* K_new, const uint16_t* V_new, float* O, void* workspace,
                                    size_t workspace_bytes, sa_stream stream) {
    return sa::decode_step_impl(cfg, cache, Q, K_new, V_new, O, workspace, workspace_bytes, stream, false);
}

// sa_decode_step; with q_after_wait the decode kernel reads Q only after its wait on the preceding kernel (the
// host-buffer entry, whose staging kernel writes Q and releases its dependents early).
sa_status sa::decode_step_impl(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q, const uint16_t* K_new,
                               const uint16_t* V_new, float* O, void* workspace, size_t workspace_bytes,
                               sa_stream stream, bool q_after_wait) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (!K_new || !V_new) return SA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(K_new) | reinterpret_cast<uintptr_t>(V_new)) & 15) return SA_ERR_ALIGNMENT;
    int S, GT;
    if (cache && cache->batch > 0 && cache->max_pages_per_seq > 0) split_plan(p, cache->batch, cache->max_pages_per_seq, &S, &GT);
    else GT = 0;
    if (GT != p.G) {
        // a query group wider than one block: the separate append kernel.  Everything the decode call will check
        // is checked first, so that a call that fails has neither written the token nor moved the length.
        DecodeArgs probe;
        int gt_probe;
        st = make_decode_args(p, cache, Q, O, workspace, workspace_bytes, &probe, &gt_probe);
        if (st != SA_OK) return st;
        st = sa_append_kv(cfg, cache, K_new, V_new, 1, stream);
        if (st != SA_OK) return st;
        return p.fp16 ? sa_decode_attention_fp16(cfg, cache, Q, O, workspace, workspace_bytes, stream)
                      : sa_decode_attention(cfg, cache, Q, O, workspace, workspace_bytes, nullptr, stream);
    }
    DecodeArgs a;
    st = make_decode_args(p, cache, Q, O, workspace, workspace_bytes, &a, &GT);
    if (st != SA_OK) return st;
    a.Knew = K_new;
    a.Vnew = V_new;
    a.wait_first = q_after_wait ? 1 : 0;
    a.zscale = (float)(1.4426950408889634 / sqrt((double)p.d) / (double)(1LL << p.F));
    if (p.int8) a.zscale = (float)(1.4426950408889634 / sqrt((double)p.d) / 127.0);
    if (p.fp16) a.zscale = (float)(1.4426950408889634 / sqrt((double)p.d));
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (p.fp16) launch_decode_fp16_main(p, a, GT, s);
    else launch_decode_main(p, a, GT, s);
    if (cudaGetLastError() != cudaSuccess) return SA_ERR_CUDA;
    return launch_merge(p, a, s);
}

extern "C" sa_status sa_decode_attention(const sa_config* cfg, const sa_cache* cache, const uint16_t* Q,
                                         float* O, void* workspace, size_t workspace_bytes,
                                         int32_t* dbg_scores, sa_stream stream) {
    return sa_decode_attention_stages(cfg, cache, Q, O, workspace, workspace_bytes, dbg_scores, 3, stream);
}

// ---------------------------------------------------------------------------------------------
// Decode attention for callers that cannot allocate device memory.
//
// Some hosts of this library have no way to hand it a workspace: code that runs where
// cudaMalloc is forbidden or unavailable (a plug-in called inside another runtime's execution
// callback, a latency-critical serving loop whose memory pool is frozen after start-up, a host
// process whose allocator must not be re-entered).  For them the split-K partials live in the
// fixed array below, which is part of the library image: every GPU on which the library's module
// is loaded holds these SA_STATIC_SCRATCH_BYTES until the process exits.
//
// The array's name is only a host-side stand-in for the symbol; the device address is obtained
// once per device with cudaGetSymbolAddress and cached.
// ---------------------------------------------------------------------------------------------
#include <mutex>

static __device__ __align__(256) unsigned char sa_static_scratch[SA_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxScratchDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxScratchDevices] = {};

// Device address of sa_static_scratch on the CURRENT device (looked up on first use).
sa_status static_scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxScratchDevices) return SA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress((void**)&ptr, sa_static_scratch) != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return SA_ERR_CUDA;
        }
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return SA_OK;
}
}  // namespace

extern "C" sa_status sa_decode_attention_static(const sa_config* cfg, const sa_cache* cache,
                                                const uint16_t* Q, float* O, int32_t* dbg_scores,
                                                sa_stream stream) {
    Plan p;
    sa_status st = make_plan(cfg, &p);
    if (st != SA_OK) return st;
    if (p.fp16) return SA_ERR_UNSUPPORTED;
    if (!cache || cache->batch <= 0 || cache->max_pages_per_seq <= 0) return SA_ERR_INVALID_ARG;
    int S, GT;
    split_plan(p, cache->batch, cache->max_pages_per_seq, &S, &GT);
    const size_t need = decode_workspace_bytes(p, cache->batch, S);
    if (need > (size_t)SA_STATIC_SCRATCH_BYTES) return SA_ERR_CAPACITY;   // problem too large for the fixed scratch
    void* scratch = nullptr;
    st = static_scratch_address(&scratch);
    if (st != SA_OK) return st;
    // Nothing in the scratch has to start at zero: the main kernel writes every partial that the
    // merge kernel reads, so contents left by an earlier call are simply overwritten.
    return sa_decode_attention_stages(cfg, cache, Q, O, scratch, (size_t)SA_STATIC_SCRATCH_BYTES, dbg_scores, 3,
                                      stream);
}
