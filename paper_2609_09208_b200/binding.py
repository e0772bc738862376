"""Thin ctypes binding of the C-ABI library (``include/sa.h``): argument marshalling only.

Every function takes torch CUDA tensors (device memory, owned by the caller), passes their
``data_ptr()`` and the current torch CUDA stream to the library and raises ``SaError`` on a
non-zero status.  No step of the method runs in Python, and there is no CPU fallback: if the
shared object is missing, ``lib()`` raises.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsa.so")

SA_POT4, SA_POTM1, SA_POTM2, SA_POTM4, SA_INT8, SA_KV_FP16 = 0, 1, 2, 4, 8, 16
SA_KLAYOUT_BYTE, SA_KLAYOUT_NIBBLE, SA_KLAYOUT_PLANAR = 0, 1, 2
SA_FLAG_HADAMARD = 1
SA_FLAG_SHIFT_BY_MULTIPLY = 2
SA_FLAG_ADD_ON_ALU = 4
PAGE_TOKENS = 64

EXPORTS = [
    "sa_version", "sa_status_string", "sa_get_layout", "sa_workspace_bytes", "sa_encode_keys",
    "sa_quantise_query", "sa_quantise_values", "sa_append_kv", "sa_fill_kv", "sa_decode_attention",
    "sa_decode_attention_fp16", "sa_decode_attention_stages", "sa_decode_attention_fp16_stages", "sa_debug_unpack", "sa_staging_bytes", "sa_decode_step_host",
    "sa_decode_attention_static", "sa_pipe_microbench", "sa_shiftav_workspace_bytes", "sa_decode_attention_shiftav",
    "sa_decode_step", "sa_debug_decode_lost_copy",
]


class SaConfig(C.Structure):
    _fields_ = [("head_dim", C.c_int), ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int),
                ("code", C.c_int), ("klayout", C.c_int), ("headroom_F", C.c_int),
                ("page_tokens", C.c_int), ("flags", C.c_uint)]


class SaLayout(C.Structure):
    _fields_ = [("page_bytes", C.c_size_t), ("kcode_off", C.c_size_t), ("meta_off", C.c_size_t),
                ("v_off", C.c_size_t), ("align", C.c_size_t)]


class SaCache(C.Structure):
    _fields_ = [("pages", C.c_void_p), ("page_table", C.c_void_p), ("seq_lens", C.c_void_p),
                ("batch", C.c_int), ("max_pages_per_seq", C.c_int), ("n_pages", C.c_int)]


class SaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (where, status_string(status), status))


_lib = None


def lib():
    """Load ``libsa.so``; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "CUDA library %s is missing: run `python -m paper_2609_09208_b200.build`" % LIB_PATH)
        _lib = C.CDLL(LIB_PATH)
        _lib.sa_status_string.restype = C.c_char_p
        _lib.sa_status_string.argtypes = [C.c_int]
        _lib.sa_version.restype = C.c_int
    return _lib


def status_string(status: int) -> str:
    return lib().sa_status_string(int(status)).decode()


def _check(st: int, where: str):
    if st != 0:
        raise SaError(st, where)


def make_config(head_dim: int, n_q_heads: int, n_kv_heads: int, code: int, *, nibble: bool = False,
                headroom_F: int = 0, hadamard: bool = False, shift_by_multiply: bool = False,
                add_on_alu: bool = False) -> SaConfig:
    """nibble=True selects the dense sub-byte container of the code: two 4-bit codes per byte for PoT-4,
    nibbles plus mantissa bit planes (5 / 6 bits per element) for PoT-M1 / PoT-M2.  shift_by_multiply=True
    selects the non-default decode kernels whose shifts run on the integer multiplier, add_on_alu=True the
    non-default ones without any multiply-add in the score datapath (same scores either way)."""
    klayout = SA_KLAYOUT_BYTE
    if nibble:
        klayout = SA_KLAYOUT_NIBBLE if code == SA_POT4 else SA_KLAYOUT_PLANAR
    return SaConfig(head_dim, n_q_heads, n_kv_heads, code, klayout, headroom_F, PAGE_TOKENS,
                    (SA_FLAG_HADAMARD if hadamard else 0) | (SA_FLAG_SHIFT_BY_MULTIPLY if shift_by_multiply else 0) |
                    (SA_FLAG_ADD_ON_ALU if add_on_alu else 0))


def get_layout(cfg: SaConfig) -> SaLayout:
    out = SaLayout()
    _check(lib().sa_get_layout(C.byref(cfg), C.byref(out)), "sa_get_layout")
    return out


def workspace_bytes(cfg: SaConfig, batch: int, max_pages_per_seq: int) -> int:
    out = C.c_size_t()
    _check(lib().sa_workspace_bytes(C.byref(cfg), C.c_int(batch), C.c_int(max_pages_per_seq), C.byref(out)),
           "sa_workspace_bytes")
    return out.value


def staging_bytes(cfg: SaConfig, batch: int) -> int:
    out = C.c_size_t()
    _check(lib().sa_staging_bytes(C.byref(cfg), C.c_int(batch), C.byref(out)), "sa_staging_bytes")
    return out.value


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def make_cache(pages, page_table, seq_lens, n_pages: int) -> SaCache:
    """pages: uint8 CUDA tensor; page_table int32 [B, max_pages]; seq_lens int32 [B]."""
    return SaCache(pages.data_ptr(), page_table.data_ptr(), seq_lens.data_ptr(),
                   int(page_table.shape[0]), int(page_table.shape[1]), int(n_pages))


def encode_keys(cfg, K, codes, scales):
    n = K.shape[0]
    _check(lib().sa_encode_keys(C.byref(cfg), _ptr(K), C.c_int64(n), _ptr(codes), _ptr(scales), _stream()),
           "sa_encode_keys")


def quantise_query(cfg, Q, q_hat, delta):
    _check(lib().sa_quantise_query(C.byref(cfg), _ptr(Q), C.c_int(Q.shape[0]), _ptr(q_hat), _ptr(delta),
                                   _stream()), "sa_quantise_query")


def quantise_values(cfg, V, v_hat, g):
    _check(lib().sa_quantise_values(C.byref(cfg), _ptr(V), C.c_int64(V.shape[0]), _ptr(v_hat), _ptr(g),
                                    _stream()), "sa_quantise_values")


def append_kv(cfg, cache: SaCache, K_new, V_new, bump_lens: bool = True):
    _check(lib().sa_append_kv(C.byref(cfg), C.byref(cache), _ptr(K_new), _ptr(V_new),
                              C.c_int(1 if bump_lens else 0), _stream()), "sa_append_kv")


def fill_kv(cfg, cache: SaCache, K, V, cu_lens_host):
    """cu_lens_host: numpy int64 array of batch + 1 entries (host memory)."""
    import numpy as np
    cu = np.ascontiguousarray(cu_lens_host, dtype=np.int64)
    _check(lib().sa_fill_kv(C.byref(cfg), C.byref(cache), _ptr(K), _ptr(V),
                            cu.ctypes.data_as(C.c_void_p), _stream()), "sa_fill_kv")


def decode_attention(cfg, cache: SaCache, Q, O, workspace, dbg_scores=None, stages: int = 3):
    """stages: 3 = whole call; 1 = main kernel only; 2 = split-K merge only."""
    if stages == 3:
        st = lib().sa_decode_attention(C.byref(cfg), C.byref(cache), _ptr(Q), _ptr(O), _ptr(workspace),
                                       C.c_size_t(workspace.numel() * workspace.element_size()),
                                       _ptr(dbg_scores), _stream())
    else:
        st = lib().sa_decode_attention_stages(C.byref(cfg), C.byref(cache), _ptr(Q), _ptr(O), _ptr(workspace),
                                              C.c_size_t(workspace.numel() * workspace.element_size()),
                                              _ptr(dbg_scores), C.c_int(stages), _stream())
    _check(st, "sa_decode_attention")


def decode_attention_fp16(cfg, cache: SaCache, Q, O, workspace, stages: int = 3):
    if stages == 3:
        st = lib().sa_decode_attention_fp16(C.byref(cfg), C.byref(cache), _ptr(Q), _ptr(O), _ptr(workspace),
                                            C.c_size_t(workspace.numel() * workspace.element_size()), _stream())
    else:
        st = lib().sa_decode_attention_fp16_stages(C.byref(cfg), C.byref(cache), _ptr(Q), _ptr(O), _ptr(workspace),
                                                   C.c_size_t(workspace.numel() * workspace.element_size()),
                                                   C.c_int(stages), _stream())
    _check(st, "sa_decode_attention_fp16")


def decode_step(cfg, cache: SaCache, Q, K_new, V_new, O, workspace):
    """Append the step's token and attend over the extended cache in one pass (sa_decode_step)."""
    _check(lib().sa_decode_step(C.byref(cfg), C.byref(cache), _ptr(Q), _ptr(K_new), _ptr(V_new), _ptr(O),
                                _ptr(workspace), C.c_size_t(workspace.numel() * workspace.element_size()),
                                _stream()), "sa_decode_step")


def shiftav_workspace_bytes(cfg: SaConfig, batch: int, max_pages_per_seq: int) -> int:
    out = C.c_size_t()
    _check(lib().sa_shiftav_workspace_bytes(C.byref(cfg), C.c_int(batch), C.c_int(max_pages_per_seq), C.byref(out)),
           "sa_shiftav_workspace_bytes")
    return out.value


def decode_attention_shiftav(cfg, cache: SaCache, Q, O, workspace, n_bits: int = 15, k_max: int = 15,
                             dbg_scores=None, dbg_rounded=None):
    """Log2-quantised weights and shift-based A.V (eq. (6), (7)); workspace of shiftav_workspace_bytes."""
    _check(lib().sa_decode_attention_shiftav(C.byref(cfg), C.byref(cache), _ptr(Q), _ptr(O), _ptr(workspace),
                                             C.c_size_t(workspace.numel() * workspace.element_size()),
                                             C.c_int(n_bits), C.c_int(k_max), _ptr(dbg_scores), _ptr(dbg_rounded),
                                             _stream()), "sa_decode_attention_shiftav")


PIPE_KINDS = ["shl", "lop3", "iadd3", "imad_by_one", "prmt", "shl+imad1", "lop3+imad1", "ffma", "ffma2",
              "imad", "dp4a", "popc+add", "i2f+fadd", "shl+lop3+imad1", "vshl.wrap.add", "vshl.clamp.add", "shl+add",
              "lds128_broadcast", "lds64_gather", "cvt.f32.s32", "cvt.rpi.s32.f32", "ex2", "cvt.f32.s8", "prmt+fadd",
              "mul.hi", "lds64_scattered"]
# instructions per step of a kind's chain ("a+b": a pair; the mixes alternate single instructions)
PIPE_KIND_INSTR = {"popc+add": 2, "i2f+fadd": 2, "shl+add": 2, "prmt+fadd": 2}


def pipe_microbench(kind: int, iters: int, blocks: int, sink):
    _check(lib().sa_pipe_microbench(C.c_int(kind), C.c_int(iters), C.c_int(blocks), _ptr(sink), _stream()),
           "sa_pipe_microbench")


STATIC_SCRATCH_BYTES = 4 << 20


def decode_attention_static(cfg, cache: SaCache, Q, O, dbg_scores=None):
    """sa_decode_attention without a caller workspace: the split-K partials use the library's fixed
    scratch array (for callers that cannot allocate device memory).  Raises SaError(status 4) when the
    problem needs more than STATIC_SCRATCH_BYTES.  Calls sharing a device must not overlap on the GPU."""
    _check(lib().sa_decode_attention_static(C.byref(cfg), C.byref(cache), _ptr(Q), _ptr(O), _ptr(dbg_scores),
                                            _stream()), "sa_decode_attention_static")


def debug_decode_lost_copy(cfg, cache: SaCache, Q, O, workspace, b: int, kv_head: int, tile: int):
    """Test hook: decode attention in which the copy of one 32-token tile is never issued (its rows come out NaN)."""
    _check(lib().sa_debug_decode_lost_copy(C.byref(cfg), C.byref(cache), _ptr(Q), _ptr(O), _ptr(workspace),
                                           C.c_size_t(workspace.numel() * workspace.element_size()), C.c_int(b),
                                           C.c_int(kv_head), C.c_int(tile), _stream()), "sa_debug_decode_lost_copy")


def debug_unpack(cfg, cache: SaCache, b: int, n_tokens: int, codes=None, scales=None, v_hat=None, g=None):
    _check(lib().sa_debug_unpack(C.byref(cfg), C.byref(cache), C.c_int(b), C.c_int(n_tokens), _ptr(codes),
                                 _ptr(scales), _ptr(v_hat), _ptr(g), _stream()), "sa_debug_unpack")


def decode_step_host(cfg, cache: SaCache, Q_host, K_new_host, V_new_host, O_host, staging, workspace):
    """Host (pinned) tensors in and out; device scratch `staging` and `workspace`."""
    _check(lib().sa_decode_step_host(
        C.byref(cfg), C.byref(cache), _ptr(Q_host), _ptr(K_new_host), _ptr(V_new_host), _ptr(O_host),
        _ptr(staging), C.c_size_t(staging.numel() * staging.element_size()), _ptr(workspace),
        C.c_size_t(workspace.numel() * workspace.element_size()), _stream()), "sa_decode_step_host")


class PagedCache:
    """Device buffers of one paged KV cache (allocation only; all arithmetic is in the library).

    `lens` are the per-sequence token counts to reserve room for (plus `extra_tokens` of head-room
    for appends).  Logical pages are mapped to pool slots through `permutation` (identity if None).
    """

    def __init__(self, cfg: SaConfig, lens, device, *, extra_tokens: int = 0, permutation=None):
        import numpy as np
        import torch
        self.cfg = cfg
        self.layout = get_layout(cfg)
        lens = np.asarray(lens, dtype=np.int64)
        self.batch = len(lens)
        pages_per_seq = (lens + extra_tokens + PAGE_TOKENS - 1) // PAGE_TOKENS
        pages_per_seq = np.maximum(pages_per_seq, 1)
        self.max_pages = int(pages_per_seq.max())
        self.n_pages = int(pages_per_seq.sum())
        table = np.full((self.batch, self.max_pages), -1, dtype=np.int32)
        slots = np.arange(self.n_pages, dtype=np.int32) if permutation is None else np.asarray(permutation, dtype=np.int32)
        assert len(slots) == self.n_pages
        o = 0
        for b in range(self.batch):
            table[b, : pages_per_seq[b]] = slots[o:o + pages_per_seq[b]]
            o += pages_per_seq[b]
        self.pages = torch.zeros(self.n_pages * cfg.n_kv_heads * self.layout.page_bytes, dtype=torch.uint8,
                                 device=device)
        self.page_table = torch.from_numpy(table).to(device)
        self.seq_lens = torch.zeros(self.batch, dtype=torch.int32, device=device)
        self.handle = make_cache(self.pages, self.page_table, self.seq_lens, self.n_pages)
        self.workspace = torch.empty(max(workspace_bytes(cfg, self.batch, self.max_pages), 16), dtype=torch.uint8,
                                     device=device)

    def fill(self, K, V, cu_lens_host):
        import numpy as np
        import torch
        fill_kv(self.cfg, self.handle, K, V, cu_lens_host)
        self.seq_lens.copy_(torch.from_numpy(np.diff(np.asarray(cu_lens_host)).astype(np.int32)))
