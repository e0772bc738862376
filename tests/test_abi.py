"""The C-ABI library without a GPU: it loads, exports every symbol the header declares, and its
host-side validation and layout arithmetic behave as documented (nothing here launches a kernel)."""
import ctypes as C
import os
import re

import pytest

from paper_2609_09208_b200 import binding as sa
from paper_2609_09208_b200 import build as sa_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    sa_build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "sa.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(sa_[a-z0-9_]+)\s*\(", header))
    assert declared == set(sa.EXPORTS), declared ^ set(sa.EXPORTS)
    lib = sa.lib()
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.sa_version() >= 1
    assert sa.status_string(0) == "ok" and "unsupported" in sa.status_string(2)


@pytest.mark.parametrize("d,code,nibble,want", [
    (64, sa.SA_POT4, True, 100), (64, sa.SA_POT4, False, 132), (64, sa.SA_POTM1, False, 132),
    (64, sa.SA_POTM4, False, 132), (128, sa.SA_POT4, True, 196), (128, sa.SA_POTM4, False, 260),
    (64, sa.SA_KV_FP16, False, 256), (128, sa.SA_KV_FP16, False, 512),
    (64, sa.SA_POTM1, True, 108), (64, sa.SA_POTM2, True, 116), (128, sa.SA_POTM1, True, 212), (128, sa.SA_POTM2, True, 228)])
def test_layout_bytes_per_key(d, code, nibble, want):
    lay = sa.get_layout(sa.make_config(d, 32, 4, code, nibble=nibble))
    assert lay.page_bytes == want * 64
    assert lay.page_bytes % 128 == 0 and lay.meta_off % 16 == 0 and lay.v_off % 16 == 0
    assert lay.kcode_off == 0 and lay.meta_off <= lay.v_off < lay.page_bytes


def test_layout_is_within_a_byte_of_the_papers_record_sizes():
    # the paper's records: 101 B (PoT-4), 133 B (8-bit code), 256 B (FP16) per key at d = 64
    golden = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "paper_constants.txt")):
        line = line.split("#")[0]
        if "=" in line:
            k, v = line.split("=")
            golden[k.strip()] = float(v)
    per_key = lambda code, nib: sa.get_layout(sa.make_config(64, 32, 4, code, nibble=nib)).page_bytes / 64
    assert abs(per_key(sa.SA_POT4, True) - golden["bytes_per_key_pot4"]) <= 1
    assert abs(per_key(sa.SA_POTM4, False) - golden["bytes_per_key_int8"]) <= 1
    assert per_key(sa.SA_KV_FP16, False) == golden["bytes_per_key_fp16"]
    assert abs(per_key(sa.SA_KV_FP16, False) / per_key(sa.SA_POT4, True) - golden["kv_cache_ratio"]) < 0.1


def _status(fn, *args):
    try:
        fn(*args)
    except sa.SaError as e:
        return e.status
    return 0


def test_config_validation():
    ok = sa.make_config(64, 32, 4, sa.SA_POTM4)
    assert _status(sa.get_layout, ok) == 0
    assert _status(sa.get_layout, sa.make_config(96, 32, 4, sa.SA_POTM4)) == 2          # head_dim
    assert _status(sa.get_layout, sa.make_config(64, 30, 4, sa.SA_POTM4)) == 1          # Hq % Hkv
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, 3)) == 2                     # no 3-bit mantissa
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_POTM4, nibble=True)) == 2   # 8 bits are dense already
    wrong = sa.make_config(64, 32, 4, sa.SA_POTM1)
    wrong.klayout = sa.SA_KLAYOUT_NIBBLE                                                   # nibble container: PoT-4 only
    assert _status(sa.get_layout, wrong) == 2
    wrong = sa.make_config(64, 32, 4, sa.SA_POT4)
    wrong.klayout = sa.SA_KLAYOUT_PLANAR                                                   # planar container: PoT-M1 / M2 only
    assert _status(sa.get_layout, wrong) == 2
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_KV_FP16, hadamard=True)) == 2
    bad = sa.make_config(64, 32, 4, sa.SA_POTM4)
    bad.page_tokens = 32
    assert _status(sa.get_layout, bad) == 2
    bad = sa.make_config(64, 32, 4, sa.SA_POTM4)
    bad.flags = 8
    assert _status(sa.get_layout, bad) == 1
    # the shift-by-multiply option exists for the mantissa codes only
    for code, nib in [(sa.SA_POTM1, False), (sa.SA_POTM1, True), (sa.SA_POTM2, False), (sa.SA_POTM4, False)]:
        assert _status(sa.get_layout, sa.make_config(64, 32, 4, code, nibble=nib, shift_by_multiply=True)) == 0
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_POT4, nibble=True, shift_by_multiply=True)) == 2
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_KV_FP16, shift_by_multiply=True)) == 2
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_INT8, shift_by_multiply=True)) == 2
    # head-room: F >= 6 + k (left shifts only), and the INT32 bound d*127*(2^(k+1)-1)*2^(F-k) < 2^31
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_POT4, headroom_F=5)) == 2
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_POT4, headroom_F=7)) == 0
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_POT4, headroom_F=18)) == 0   # 64*127*2^18 < 2^31
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_POT4, headroom_F=19)) == 2
    assert _status(sa.get_layout, sa.make_config(128, 32, 8, sa.SA_POTM4, headroom_F=16)) == 0  # 128*127*31*2^12 < 2^31
    assert _status(sa.get_layout, sa.make_config(128, 32, 8, sa.SA_POTM4, headroom_F=17)) == 2


def test_workspace_and_staging_sizes():
    cfg = sa.make_config(64, 32, 4, sa.SA_POTM4)
    w = sa.workspace_bytes(cfg, 1, 512)
    assert w > 0 and w % (32 * 66 * 4) == 0
    n_splits = w // (32 * 66 * 4)
    assert 1 <= n_splits <= 512
    # batches of 2 .. 128 sequences: the partials plus two words per sequence (first slot, splits) for the merge kernel
    assert (sa.workspace_bytes(cfg, 16, 256) - 16 * 8) % (16 * 32 * 66 * 4) == 0
    assert sa.workspace_bytes(cfg, 129, 256) % (129 * 32 * 66 * 4) == 0
    assert sa.workspace_bytes(cfg, 1, 1) == 32 * 66 * 4          # a single page: no split
    assert _status(sa.workspace_bytes, cfg, 0, 4) == 1
    assert sa.staging_bytes(cfg, 2) >= 2 * (32 * 64 * 2 + 2 * 4 * 64 * 2 + 32 * 64 * 4)


def test_entry_points_reject_bad_arguments_before_any_cuda_call():
    lib = sa.lib()
    cfg = sa.make_config(64, 32, 4, sa.SA_POTM4)
    null = C.c_void_p(0)
    one = C.c_void_p(256)       # a non-null, aligned, never dereferenced address
    assert lib.sa_encode_keys(C.byref(cfg), null, C.c_int64(4), one, one, null) == 1
    assert lib.sa_encode_keys(C.byref(cfg), C.c_void_p(257), C.c_int64(4), one, one, null) == 3
    assert lib.sa_encode_keys(C.byref(cfg), one, C.c_int64(0), one, one, null) == 0      # nothing to do
    assert lib.sa_quantise_query(C.byref(cfg), null, C.c_int(1), one, one, null) == 1
    assert lib.sa_quantise_values(C.byref(cfg), one, C.c_int64(-1), one, one, null) == 1
    cache = sa.SaCache(0, 256, 256, 1, 4, 4)
    assert lib.sa_decode_attention(C.byref(cfg), C.byref(cache), one, one, one, C.c_size_t(1 << 30), null, null) == 1
    cache = sa.SaCache(256, 256, 256, 1, 4, 4)
    assert lib.sa_decode_attention(C.byref(cfg), C.byref(cache), one, one, one, C.c_size_t(8), null, null) == 4
    assert lib.sa_decode_attention(C.byref(cfg), C.byref(cache), one, one, C.c_void_p(260), C.c_size_t(1 << 30), null, null) == 3
    cache = sa.SaCache(264, 256, 256, 1, 4, 4)                                            # pool base not 256-aligned
    assert lib.sa_append_kv(C.byref(cfg), C.byref(cache), one, one, C.c_int(1), null) == 3
    fp = sa.make_config(64, 32, 4, sa.SA_KV_FP16)
    cache = sa.SaCache(256, 256, 256, 1, 4, 4)
    assert lib.sa_decode_attention(C.byref(fp), C.byref(cache), one, one, one, C.c_size_t(1 << 30), null, null) == 2
    assert lib.sa_decode_attention_fp16(C.byref(cfg), C.byref(cache), one, one, one, C.c_size_t(1 << 30), null) == 2
    assert lib.sa_debug_unpack(C.byref(cfg), C.byref(cache), C.c_int(3), C.c_int(1), null, null, null, null, null) == 1
    assert lib.sa_debug_unpack(C.byref(cfg), C.byref(cache), C.c_int(0), C.c_int(4 * 64 + 1), null, null, null, null, null) == 4


def test_step_entries_check_the_decode_arguments_before_they_launch_anything():
    """sa_decode_step with a query group wider than one block appends with a separate kernel, and sa_decode_step_host
    stages its inputs first: both must have checked the decode call's arguments before that.  Without a GPU a
    launch attempt would come back as a CUDA error (5); the argument errors must win."""
    lib = sa.lib()
    null, one = C.c_void_p(0), C.c_void_p(256)
    wide = sa.make_config(64, 32, 2, sa.SA_POTM4)            # 16 query heads per KV head: the separate append
    cache = sa.SaCache(256, 256, 256, 1, 4, 4)
    need = sa.workspace_bytes(wide, 1, 4)
    step = lambda cfg, ws, nbytes, O=one: lib.sa_decode_step(C.byref(cfg), C.byref(cache), one, one, one, O, ws,
                                                             C.c_size_t(nbytes), null)
    assert step(wide, one, need - 1) == 4                    # short workspace
    assert step(wide, null, need) == 4
    assert step(wide, one, need, null) == 1                  # no output
    assert step(wide, C.c_void_p(260), need) == 3            # misaligned workspace
    ok = sa.make_config(64, 32, 4, sa.SA_POTM4)
    assert step(ok, one, sa.workspace_bytes(ok, 1, 4) - 1) == 4
    # the host-buffer entry: cache pointers, alignment and workspace are checked before the staging transfers
    stg = sa.staging_bytes(ok, 1)
    host = lambda c, ws_bytes: lib.sa_decode_step_host(C.byref(ok), C.byref(c), one, one, one, one, one, C.c_size_t(stg),
                                                        one, C.c_size_t(ws_bytes), null)
    assert host(sa.SaCache(0, 256, 256, 1, 4, 4), 1 << 30) == 1
    assert host(sa.SaCache(264, 256, 256, 1, 4, 4), 1 << 30) == 3
    assert host(cache, 8) == 4


def test_flag_combinations():
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_POTM4, add_on_alu=True)) == 0
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_POT4, nibble=True, add_on_alu=True)) == 0
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_POTM4, add_on_alu=True, shift_by_multiply=True)) == 1
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_INT8, add_on_alu=True)) == 2
    assert _status(sa.get_layout, sa.make_config(64, 32, 4, sa.SA_KV_FP16, add_on_alu=True)) == 2


def test_lost_copy_hook_validates_on_the_host():
    lib = sa.lib()
    null, one = C.c_void_p(0), C.c_void_p(256)
    cache = sa.SaCache(256, 256, 256, 2, 4, 8)
    ok = sa.make_config(64, 32, 4, sa.SA_POTM4)
    call = lambda cfg, b, h, t, nbytes=1 << 30: lib.sa_debug_decode_lost_copy(
        C.byref(cfg), C.byref(cache), one, one, one, C.c_size_t(nbytes), C.c_int(b), C.c_int(h), C.c_int(t), null)
    assert call(sa.make_config(64, 32, 4, sa.SA_POTM1), 0, 0, 0) == 2
    assert call(sa.make_config(128, 32, 4, sa.SA_POTM4), 0, 0, 0) == 2
    assert call(sa.make_config(64, 16, 4, sa.SA_POTM4), 0, 0, 0) == 2
    assert call(ok, 2, 0, 0) == 1 and call(ok, 0, 4, 0) == 1 and call(ok, 0, 0, -1) == 1
    assert call(ok, 0, 0, 0, 8) == 4


def test_static_scratch_holds_the_headline_shape_at_any_length():
    """sa_decode_attention_static documents that batch 1, 32 query heads, head_dim 64 fits its fixed scratch at any
    cache length, for every code it accepts: the split count is capped, so the workspace is bounded."""
    for code, nib in [(sa.SA_POT4, False), (sa.SA_POT4, True), (sa.SA_POTM1, False), (sa.SA_POTM1, True), (sa.SA_POTM2, False),
                      (sa.SA_POTM4, False), (sa.SA_INT8, False)]:
        cfg = sa.make_config(64, 32, 4, code, nibble=nib)
        for pages in (1, 2, 7, 64, 512, 513, 4096, 1 << 16, 1 << 20):
            assert sa.workspace_bytes(cfg, 1, pages) <= sa.STATIC_SCRATCH_BYTES, (code, nib, pages)


def test_shiftav_entry_validates_on_the_host():
    """The shift-based A.V option: workspace = partials + rounded logits + per-split statistics; the
    constants N and k_max, the code and the workspace are checked before anything is launched."""
    lib = sa.lib()
    cfg = sa.make_config(64, 32, 4, sa.SA_POTM4)
    base, full = sa.workspace_bytes(cfg, 2, 64), sa.shiftav_workspace_bytes(cfg, 2, 64)
    assert full >= base + 2 * 32 * 64 * 64 * 4               # + int32 rounded logits for every (head, key slot)
    assert full % 256 == 0
    for code in (sa.SA_INT8, sa.SA_KV_FP16):
        assert _status(sa.shiftav_workspace_bytes, sa.make_config(64, 32, 4, code), 2, 64) == 2
    null, one = C.c_void_p(0), C.c_void_p(256)
    cache = sa.SaCache(256, 256, 256, 2, 64, 128)
    big = C.c_size_t(1 << 30)
    call = lambda n, k, ws=one, nbytes=big: lib.sa_decode_attention_shiftav(
        C.byref(cfg), C.byref(cache), one, one, ws, nbytes, C.c_int(n), C.c_int(k), null, null, null)
    assert call(0, 0) == 1 and call(19, 3) == 1 and call(15, 16) == 1 and call(15, -1) == 1
    assert call(15, 15, one, C.c_size_t(full - 1)) == 4
    assert call(15, 15, C.c_void_p(256 + 16), big) == 3
