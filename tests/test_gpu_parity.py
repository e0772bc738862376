"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.  Integer results (codes, scales, quantised queries and values, INT32 scores) must be
bit-exact; the attention output must agree within 1e-3 (FP32, unit-variance values)."""
import numpy as np
import pytest

from oracle import sa_oracle as ora
from paper_2609_09208_b200 import binding as sa
from paper_2609_09208_b200 import build as sa_build
from paper_2609_09208_b200 import synth

pytestmark = pytest.mark.gpu
TOL_O = 1e-3
E = 6


@pytest.fixture(scope="module")
def dev():
    import torch
    sa_build.build()
    sa.lib()
    return torch.device("cuda:0")


def t16(x, dev):
    """float16 numpy -> CUDA tensor of its bits (int16 storage; the library only sees bytes)."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to(dev)


def cfg_of(case, *, code=None, F=0, shift_by_multiply=False, add_on_alu=False):
    code = case.code_k if code is None else code
    return sa.make_config(case.head_dim, case.n_q_heads, case.n_kv_heads, code, nibble=case.nibble,
                          headroom_F=F, hadamard=case.hadamard, shift_by_multiply=shift_by_multiply,
                          add_on_alu=add_on_alu)


def build_cache(case, dev, *, cfg=None, permute_seed=None, extra_tokens=0):
    cfg = cfg or cfg_of(case)
    n_pages = int(np.maximum((case.lens + extra_tokens + 63) // 64, 1).sum())
    perm = synth.page_permutation(n_pages, permute_seed) if permute_seed is not None else None
    cache = sa.PagedCache(cfg, case.lens, dev, extra_tokens=extra_tokens, permutation=perm)
    cache.fill(t16(case.K, dev), t16(case.V, dev), case.cu_lens)
    return cfg, cache


def run_decode(case, dev, *, F=0, want_scores=True, permute_seed=None, shift_by_multiply=False, add_on_alu=False):
    import torch
    cfg = cfg_of(case, F=F, shift_by_multiply=shift_by_multiply, add_on_alu=add_on_alu)
    cfg, cache = build_cache(case, dev, cfg=cfg, permute_seed=permute_seed)
    O = torch.full((case.batch, case.n_q_heads, case.head_dim), float("nan"), dtype=torch.float32, device=dev)
    dbg = None
    if want_scores:
        dbg = torch.full((case.batch, case.n_q_heads, cache.max_pages * 64), -7, dtype=torch.int32, device=dev)
    sa.decode_attention(cfg, cache.handle, t16(case.Q, dev), O, cache.workspace, dbg)
    torch.cuda.synchronize()
    return O.cpu().numpy(), (dbg.cpu().numpy() if want_scores else None), cache


def check_against_oracle(case, O, dbg, *, F=0, n_threads=8):
    F = F or E + case.code_k
    ref = ora.decode_attention(case.Q, case.K, case.V, case.cu_lens, case.code_k, F, hadamard=case.hadamard,
                               want_scores=dbg is not None, n_threads=n_threads)
    assert ref["overflow"] == 0
    if dbg is not None:
        for b in range(case.batch):
            T = int(case.lens[b])
            assert np.array_equal(dbg[b, :, :T].astype(np.int64), ref["A"][b][:, :T]), "integer scores differ (sequence %d)" % b
            assert np.all(dbg[b, :, T:] == -7), "scores written beyond the sequence length"
    err = np.max(np.abs(O.astype(np.float64) - ref["O"])) if O.size else 0.0
    assert np.isfinite(O).all()
    assert err <= TOL_O, "max |dO| = %g" % err
    return err


# ------------------------------------------------------------------------------- quantisers
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("k", [0, 1, 2, 4])
@pytest.mark.parametrize("hadamard", [False, True])
def test_encode_keys_bit_exact(dev, d, k, hadamard):
    import torch
    rng = np.random.default_rng(1000 + d + k)
    Hkv, n = 3, 1500                                    # 4500 vectors: many blocks and a ragged tail
    K = synth.outlier_keys_fp16(rng, n, Hkv, d)
    K[5, 1, :] = 0                                      # an all-zero vector
    K[6, 0, 3] = 0
    K.view(np.uint16)[7, 2, :8] = [1, 2, 0x8001, 0x03FF, 0x0400, 0x7BFF, 0xFBFF, 0x8000]   # subnormals, extremes, -0
    cfg = sa.make_config(d, Hkv, Hkv, k, hadamard=hadamard)
    codes = torch.zeros((n, Hkv, d), dtype=torch.uint8, device=dev)
    scales = torch.zeros((n, Hkv), dtype=torch.int16, device=dev)
    sa.encode_keys(cfg, t16(K, dev), codes, scales)
    torch.cuda.synchronize()
    Kr = ora.hadamard_fp16(K) if hadamard else K
    want_c, want_s = ora.encode_keys(Kr, k)
    assert np.array_equal(scales.cpu().numpy().view(np.uint16), want_s.view(np.uint16))
    assert np.array_equal(codes.cpu().numpy(), want_c)


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("hadamard", [False, True])
def test_quantise_query_bit_exact(dev, d, hadamard):
    import torch
    rng = np.random.default_rng(1100 + d)
    B, Hq = 37, 8
    Q = (rng.standard_normal((B, Hq, d)) * np.exp(rng.standard_normal((B, Hq, 1)))).astype(np.float16)
    Q[3, 2] = 0
    cfg = sa.make_config(d, Hq, Hq, sa.SA_POTM4, hadamard=hadamard)
    qh = torch.zeros((B, Hq, d), dtype=torch.int8, device=dev)
    dl = torch.zeros((B, Hq), dtype=torch.float32, device=dev)
    sa.quantise_query(cfg, t16(Q, dev), qh, dl)
    torch.cuda.synchronize()
    want_q, want_d = ora.quantise_query(ora.hadamard_fp16(Q) if hadamard else Q)
    assert np.array_equal(qh.cpu().numpy(), want_q)
    assert np.array_equal(dl.cpu().numpy().view(np.uint32), want_d.view(np.uint32))


@pytest.mark.parametrize("d", [64, 128])
def test_quantise_values_bit_exact(dev, d):
    import torch
    rng = np.random.default_rng(1200 + d)
    n, Hkv = 1111, 2
    V = (rng.standard_normal((n, Hkv, d)) * np.exp(rng.uniform(-9, 9, (n, Hkv, 1)))).astype(np.float16)
    V[4, 1] = 0
    V.view(np.uint16)[9, 0, :4] = [1, 0x7BFF, 0xFBFF, 0x8001]
    cfg = sa.make_config(d, Hkv, Hkv, sa.SA_POTM1)
    vh = torch.zeros((n, Hkv, d), dtype=torch.int8, device=dev)
    g = torch.zeros((n, Hkv), dtype=torch.int8, device=dev)
    sa.quantise_values(cfg, t16(V, dev), vh, g)
    torch.cuda.synchronize()
    want_v, want_g = ora.quantise_value(V)
    assert np.array_equal(g.cpu().numpy(), want_g)
    assert np.array_equal(vh.cpu().numpy(), want_v)


# ------------------------------------------------------------------------------- cache write
def _unpack(cfg, cache, b, T, case, dev):
    import torch
    Hkv, d = case.n_kv_heads, case.head_dim
    codes = torch.zeros((T, Hkv, d), dtype=torch.uint8, device=dev)
    scales = torch.zeros((T, Hkv), dtype=torch.int16, device=dev)
    vh = torch.zeros((T, Hkv, d), dtype=torch.int8, device=dev)
    g = torch.zeros((T, Hkv), dtype=torch.int8, device=dev)
    sa.debug_unpack(cfg, cache.handle, b, T, codes, scales, vh, g)
    torch.cuda.synchronize()
    return codes.cpu().numpy(), scales.cpu().numpy().view(np.uint16), vh.cpu().numpy(), g.cpu().numpy()


@pytest.mark.parametrize("d,k,nibble,hadamard", [(64, 0, True, False), (64, 0, False, True), (64, 1, False, False),
                                                 (64, 4, False, True), (128, 0, True, False), (128, 2, False, False),
                                                 (128, 4, False, True), (64, 1, True, False), (64, 2, True, True),
                                                 (128, 1, True, True), (128, 2, True, False)])
def test_fill_and_unpack_bit_exact(dev, d, k, nibble, hadamard):
    case = synth.make_case("fill", [130, 0, 64, 1, 257], 4, 2, d, k, outliers=True, nibble=nibble,
                           hadamard=hadamard, seed=1300 + d + k)
    cfg, cache = build_cache(case, dev, permute_seed=5)
    for b in range(case.batch):
        T = int(case.lens[b])
        if T == 0:
            continue
        K = case.K[case.cu_lens[b]:case.cu_lens[b + 1]]
        V = case.V[case.cu_lens[b]:case.cu_lens[b + 1]]
        want_c, want_s = ora.encode_keys(ora.hadamard_fp16(K) if hadamard else K, k)
        want_v, want_g = ora.quantise_value(V)
        codes, scales, vh, g = _unpack(cfg, cache, b, T, case, dev)
        assert np.array_equal(codes, want_c) and np.array_equal(scales, want_s.view(np.uint16))
        assert np.array_equal(vh, want_v) and np.array_equal(g, want_g)


@pytest.mark.parametrize("d,k,nibble", [(64, 4, False), (64, 0, True), (128, 1, False), (64, 1, True), (128, 2, True)])
def test_append_matches_bulk_fill(dev, d, k, nibble):
    import torch
    lens = np.array([62, 0, 127])
    n_app = 4                                          # crosses a page boundary for the first and last sequence
    full = synth.make_case("app", lens + n_app, 4, 2, d, k, nibble=nibble, seed=1400 + d + k)
    cfg = cfg_of(full)
    cache = sa.PagedCache(cfg, lens, dev, extra_tokens=n_app, permutation=synth.page_permutation(
        int(np.maximum((lens + n_app + 63) // 64, 1).sum()), 9))
    # bulk-fill the first lens[b] tokens, then append the rest one token at a time
    idx0 = np.concatenate([np.arange(full.cu_lens[b], full.cu_lens[b] + lens[b]) for b in range(3)]).astype(np.int64)
    cu0 = np.concatenate([[0], np.cumsum(lens)])
    cache.fill(t16(full.K[idx0], dev), t16(full.V[idx0], dev), cu0)
    for i in range(n_app):
        rows = np.array([full.cu_lens[b] + lens[b] + i for b in range(3)])
        sa.append_kv(cfg, cache.handle, t16(full.K[rows], dev), t16(full.V[rows], dev), True)
    torch.cuda.synchronize()
    assert cache.seq_lens.cpu().numpy().tolist() == (lens + n_app).tolist()
    for b in range(3):
        T = int(lens[b] + n_app)
        K = full.K[full.cu_lens[b]:full.cu_lens[b + 1]]
        V = full.V[full.cu_lens[b]:full.cu_lens[b + 1]]
        want_c, want_s = ora.encode_keys(K, k)
        want_v, want_g = ora.quantise_value(V)
        codes, scales, vh, g = _unpack(cfg, cache, b, T, full, dev)
        assert np.array_equal(codes, want_c) and np.array_equal(scales, want_s.view(np.uint16))
        assert np.array_equal(vh, want_v) and np.array_equal(g, want_g)
    # a full sequence is left untouched
    tight = sa.PagedCache(cfg, [64], dev)
    tight.seq_lens.fill_(64)
    sa.append_kv(cfg, tight.handle, t16(full.K[:1], dev), t16(full.V[:1], dev), True)
    torch.cuda.synchronize()
    assert int(tight.seq_lens[0]) == 64


# ------------------------------------------------------------------------------- decode attention
def test_config1_single_head_pot4(dev):
    case = synth.config1()
    O, dbg, _ = run_decode(case, dev, F=6)
    check_against_oracle(case, O, dbg, F=6)


def test_config2_llama_shape_potm1_outliers(dev):
    case = synth.config2()
    O, dbg, _ = run_decode(case, dev)
    check_against_oracle(case, O, dbg)


@pytest.mark.parametrize("k,nibble,hadamard,outliers", [
    (4, False, False, False), (4, False, True, False), (4, False, True, True),
    (0, False, False, False), (0, True, False, False), (0, True, True, True),
    (1, True, False, True), (2, True, True, False)])                 # PoT-M1 / PoT-M2 in the dense planar container
def test_config3_T32k_full_size(dev, k, nibble, hadamard, outliers):
    case = synth.config3(k, hadamard=hadamard, nibble=nibble, outliers=outliers)
    O, dbg, _ = run_decode(case, dev)
    check_against_oracle(case, O, dbg)


def test_config4_ragged_paged_batch_potm2(dev):
    case = synth.config4()
    O, dbg, _ = run_decode(case, dev, permute_seed=44)
    check_against_oracle(case, O, dbg)


@pytest.mark.parametrize("d,Hq,Hkv,k", [(64, 32, 4, 1), (64, 32, 4, 2), (128, 32, 8, 1), (128, 32, 8, 2), (64, 6, 2, 2)])
def test_planar_container_ragged_batch(dev, d, Hq, Hkv, k):
    """PoT-M1 / PoT-M2 in the dense planar container (5 / 6 bits per element): the same integer scores and
    outputs as the oracle, on a ragged paged batch with an empty sequence and shuffled pages."""
    case = synth.make_case("planar", [3000, 0, 65, 1, 777], Hq, Hkv, d, k, nibble=True, outliers=True, seed=1700 + d + k)
    O, dbg, cache = run_decode(case, dev, permute_seed=9)
    check_against_oracle(case, O, dbg)
    lay = sa.get_layout(cfg_of(case))
    assert lay.page_bytes == 64 * (d // 2 + k * d // 8 + 4 + d)


@pytest.mark.parametrize("T,B,k", [(1024, 1, 0), (1024, 8, 1), (4096, 8, 4), (16384, 1, 1), (4096, 32, 0)])
def test_config5_d128_cells_in_full(dev, T, B, k):
    case = synth.config5(T, B, k)
    O, dbg, _ = run_decode(case, dev)
    check_against_oracle(case, O, dbg)


def test_config5_largest_cells_sampled_sequences(dev):
    """T = 128k x B = 8, PoT-M4, d = 128 (the cache is built sequence by sequence from seeded
    inputs; the oracle recomputes two sampled sequences in full, scores included)."""
    import torch
    T, B, k, d, Hq, Hkv = 131072, 8, 4, 128, 32, 8
    cfg = sa.make_config(d, Hq, Hkv, k)
    cache = sa.PagedCache(cfg, [T] * B, dev)
    Q = synth.gaussian_fp16(np.random.default_rng(7), (B, Hq, d))
    kept = {}
    for b in range(B):
        one = synth.make_case("c5big", [T], Hq, Hkv, d, k, outliers=True, seed=5100 + b)
        sub = sa.SaCache(cache.pages.data_ptr(), cache.page_table[b:b + 1].contiguous().data_ptr(),
                         cache.seq_lens[b:b + 1].data_ptr(), 1, cache.max_pages, cache.n_pages)
        sa.fill_kv(cfg, sub, t16(one.K, dev), t16(one.V, dev), one.cu_lens)
        torch.cuda.synchronize()
        if b in (2, 7):
            kept[b] = one
    cache.seq_lens.fill_(T)
    O = torch.zeros((B, Hq, d), dtype=torch.float32, device=dev)
    dbg = torch.zeros((B, Hq, cache.max_pages * 64), dtype=torch.int32, device=dev)
    sa.decode_attention(cfg, cache.handle, t16(Q, dev), O, cache.workspace, dbg)
    torch.cuda.synchronize()
    O = O.cpu().numpy()
    for b, one in kept.items():
        ref = ora.decode_attention(Q[b:b + 1], one.K, one.V, one.cu_lens, k, E + k, want_scores=True, n_threads=8)
        assert np.array_equal(dbg[b].cpu().numpy().astype(np.int64), ref["A"][0])
        assert np.max(np.abs(O[b] - ref["O"][0])) <= TOL_O
    assert np.isfinite(O).all()


@pytest.mark.parametrize("lens", [[0], [1], [31], [32], [33], [63], [64], [65], [127, 0, 129, 1], [4097]])
@pytest.mark.parametrize("k,nibble", [(0, True), (4, False), (2, True)])
def test_edge_lengths(dev, lens, k, nibble):
    case = synth.make_case("edge", lens, 8, 2, 64, k, nibble=nibble, seed=1500 + sum(lens) + k)
    O, dbg, _ = run_decode(case, dev, permute_seed=3)
    check_against_oracle(case, O, dbg)
    for b, T in enumerate(lens):
        if T == 0:
            assert not O[b].any()


@pytest.mark.parametrize("Hq,Hkv", [(1, 1), (2, 1), (4, 4), (6, 2), (12, 1), (16, 2), (32, 4)])
def test_query_group_sizes(dev, Hq, Hkv):
    case = synth.make_case("gqa", [300, 77], Hq, Hkv, 64, 2, outliers=True, seed=1600 + Hq)
    O, dbg, _ = run_decode(case, dev)
    check_against_oracle(case, O, dbg)


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("nibble", [False, True])
@pytest.mark.parametrize("Hq,Hkv", [(1, 1), (2, 1), (3, 1), (8, 2), (12, 1), (16, 2)])
def test_pot4_query_group_sizes(dev, Hq, Hkv, nibble, d):
    """PoT-4 looks its shifted packed query pairs up in a table whose rows hold 1, 2 or 4 pairs (groups of 1-2, 3-4,
    5-8 query heads per block) with a different address pattern each: every row width, both containers, both head
    dimensions, an odd group (a pair with one query) and a group wider than one block."""
    case = synth.make_case("gqa4", [300, 77, 1], Hq, Hkv, d, 0, outliers=True, nibble=nibble, seed=1650 + Hq + d)
    O, dbg, _ = run_decode(case, dev, permute_seed=3)
    check_against_oracle(case, O, dbg)


@pytest.mark.parametrize("k,F", [(0, 7), (0, 18), (1, 9), (4, 12), (4, 16)])
def test_headroom_F(dev, k, F):
    # F = 7 with PoT-4 is the paper's worked bound (d * 127 * 2^7); larger F only shifts the exact integer
    d = 128 if F == 16 else 64
    case = synth.make_case("F", [200], 8, 2, d, k, seed=1700 + F)
    if (d * 127 * ((1 << (k + 1)) - 1)) << (F - k) >= 2 ** 31:
        pytest.skip("outside the INT32 bound")
    O, dbg, _ = run_decode(case, dev, F=F)
    check_against_oracle(case, O, dbg, F=F)


def test_attained_int32_bound_and_determinism(dev):
    import torch
    # keys equal to +scale everywhere (e = 0) and a constant query attain d * 127 * 2^F exactly
    d, T = 64, 100
    case = synth.make_case("bound", [T], 2, 1, d, 0, seed=1)
    case.K[:] = np.float16(1.5)
    case.Q[:] = np.float16(-2.0)
    O, dbg, _ = run_decode(case, dev, F=18)
    assert np.all(dbg[0, :, :T] == -(64 * 127 * 2 ** 18))
    check_against_oracle(case, O, dbg, F=18)
    case = synth.config3(4, T=8192)
    o1, s1, _ = run_decode(case, dev)
    o2, s2, _ = run_decode(case, dev)
    assert np.array_equal(o1.view(np.uint32), o2.view(np.uint32)) and np.array_equal(s1, s2)


def test_unmapped_pages_are_skipped_not_read(dev):
    import torch
    case = synth.make_case("unmapped", [200], 8, 2, 64, 4, seed=1800)
    cfg, cache = build_cache(case, dev)
    cache.page_table[0, 1] = -1                     # tokens 64..127 vanish
    cache.page_table[0, 2] = cache.n_pages + 5      # out of range: also skipped
    O = torch.zeros((1, 8, 64), dtype=torch.float32, device=dev)
    sa.decode_attention(cfg, cache.handle, t16(case.Q, dev), O, cache.workspace, None)
    torch.cuda.synchronize()
    keep = np.r_[0:64, 192:200]
    sub = synth.Case("sub", case.Q, case.K[keep], case.V[keep], np.array([0, len(keep)]), 8, 2, 64, 4)
    ref = ora.decode_attention(sub.Q, sub.K, sub.V, sub.cu_lens, 4, 10)
    assert np.max(np.abs(O.cpu().numpy() - ref["O"])) <= TOL_O


# ------------------------------------------------------------------------------- FP16 baseline kernel
@pytest.mark.parametrize("d,Hq,Hkv,lens", [(64, 32, 4, [4096]), (64, 8, 2, [0, 1, 33, 700]), (128, 32, 8, [2048, 100]),
                                           (64, 1, 1, [1024]), (64, 32, 4, [32768])])
def test_fp16_kernel_matches_textbook_attention(dev, d, Hq, Hkv, lens):
    import torch
    case = synth.make_case("fp16", lens, Hq, Hkv, d, 0, seed=1900 + d + len(lens))
    cfg = sa.make_config(d, Hq, Hkv, sa.SA_KV_FP16)
    _, cache = build_cache(case, dev, cfg=cfg, permute_seed=2)
    O = torch.full((case.batch, Hq, d), float("nan"), dtype=torch.float32, device=dev)
    sa.decode_attention_fp16(cfg, cache.handle, t16(case.Q, dev), O, cache.workspace)
    torch.cuda.synchronize()
    O = O.cpu().numpy()
    for b in range(case.batch):
        K = case.K[case.cu_lens[b]:case.cu_lens[b + 1]]
        V = case.V[case.cu_lens[b]:case.cu_lens[b + 1]]
        ref = ora.sdpa_fp16(case.Q[b], K, V)
        assert np.max(np.abs(O[b] - ref)) <= TOL_O


# ------------------------------------------------------------------------------- host-buffer entry
@pytest.mark.parametrize("pinned", [True, False])     # pinned: fetched / stored by kernels; pageable: copied
@pytest.mark.parametrize("code", [sa.SA_POTM4, sa.SA_KV_FP16])
def test_decode_step_from_host_buffers(dev, code, pinned):
    import torch
    lens = np.array([100, 64, 0])
    full = synth.make_case("host", lens + 1, 8, 2, 64, 4, seed=2000)
    cfg = sa.make_config(64, 8, 2, code)
    cache = sa.PagedCache(cfg, lens, dev, extra_tokens=1)
    idx0 = np.concatenate([np.arange(full.cu_lens[b], full.cu_lens[b] + lens[b]) for b in range(3)]).astype(np.int64)
    cache.fill(t16(full.K[idx0], dev), t16(full.V[idx0], dev), np.concatenate([[0], np.cumsum(lens)]))
    last = np.array([full.cu_lens[b + 1] - 1 for b in range(3)])
    pin = lambda x: (lambda t: t.pin_memory() if pinned else t)(torch.from_numpy(np.ascontiguousarray(x).view(np.int16)))
    Qh, Kh, Vh = pin(full.Q), pin(full.K[last]), pin(full.V[last])
    Oh = torch.zeros((3, 8, 64), dtype=torch.float32)
    Oh = Oh.pin_memory() if pinned else Oh
    staging = torch.empty(sa.staging_bytes(cfg, 3), dtype=torch.uint8, device=dev)
    sa.decode_step_host(cfg, cache.handle, Qh, Kh, Vh, Oh, staging, cache.workspace)
    torch.cuda.synchronize()
    assert cache.seq_lens.cpu().numpy().tolist() == (lens + 1).tolist()
    for b in range(3):
        K = full.K[full.cu_lens[b]:full.cu_lens[b + 1]]
        V = full.V[full.cu_lens[b]:full.cu_lens[b + 1]]
        if code == sa.SA_KV_FP16:
            ref = ora.sdpa_fp16(full.Q[b], K, V)
        else:
            ref = ora.decode_attention(full.Q[b:b + 1], K, V, np.array([0, len(K)]), 4, 10)["O"][0]
        assert np.max(np.abs(Oh.numpy()[b] - ref)) <= TOL_O


# ------------------------------------------------------------------------------- INT8 comparison code
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("hadamard", [False, True])
def test_int8_encode_keys_bit_exact(dev, d, hadamard):
    import torch
    rng = np.random.default_rng(2100 + d)
    Hkv, n = 2, 999
    K = synth.outlier_keys_fp16(rng, n, Hkv, d)
    K[3, 1, :] = 0
    cfg = sa.make_config(d, Hkv, Hkv, sa.SA_INT8, hadamard=hadamard)
    codes = torch.zeros((n, Hkv, d), dtype=torch.int8, device=dev)
    scales = torch.zeros((n, Hkv), dtype=torch.int16, device=dev)
    sa.encode_keys(cfg, t16(K, dev), codes, scales)
    torch.cuda.synchronize()
    want_c, want_s = ora.encode_keys_int8(ora.hadamard_fp16(K) if hadamard else K)
    assert np.array_equal(scales.cpu().numpy().view(np.uint16), want_s.view(np.uint16))
    assert np.array_equal(codes.cpu().numpy(), want_c)


@pytest.mark.parametrize("lens,Hq,Hkv,d,hadamard", [([32768], 32, 4, 64, False), ([0, 1, 33, 700, 64], 8, 2, 64, True),
                                                    ([4096, 100], 32, 8, 128, False), ([1024], 1, 1, 64, False)])
def test_int8_decode_matches_oracle(dev, lens, Hq, Hkv, d, hadamard):
    case = synth.make_case("int8", lens, Hq, Hkv, d, 8, outliers=True, hadamard=hadamard, seed=2200 + d + len(lens))
    O, dbg, cache = run_decode(case, dev, permute_seed=8)
    check_against_oracle(case, O, dbg)
    # the cache holds the oracle's codes
    for b, T in enumerate(lens):
        if T == 0:
            continue
        K = case.K[case.cu_lens[b]:case.cu_lens[b + 1]]
        want_c, want_s = ora.encode_keys_int8(ora.hadamard_fp16(K) if hadamard else K)
        codes, scales, _, _ = _unpack(cfg_of(case), cache, b, T, case, dev)
        assert np.array_equal(codes.view(np.int8), want_c) and np.array_equal(scales, want_s.view(np.uint16))


# ------------------------------------------------------------------------------- eq. (6), (7): shift-based A.V
def oracle_shiftav(case, n_bits, k_max, F=0):
    """The oracle's steps chained per sequence: (rotation,) key codes, query and value quantisers, integer
    scores, then log2-quantised weights with the shift-based A.V.  Returns O [B, Hq, d] and the rounded
    logits per sequence."""
    F = F or E + case.code_k
    O = np.zeros((case.batch, case.n_q_heads, case.head_dim))
    rounded = []
    for b in range(case.batch):
        t0, t1 = int(case.cu_lens[b]), int(case.cu_lens[b + 1])
        Q, K, V = case.Q[b], case.K[t0:t1], case.V[t0:t1]
        if case.hadamard:
            Q, K = ora.hadamard_fp16(Q), ora.hadamard_fp16(K)
        codes, scales = ora.encode_keys(K, case.code_k)
        qhat, delta = ora.quantise_query(Q)
        vhat, g = ora.quantise_value(V)
        A, ov = ora.scores(qhat, codes, case.code_k, F)
        assert ov == 0
        O[b], zr, _ = ora.attention_shiftav(A, delta, scales, vhat, g, F, n_bits, k_max)
        rounded.append(zr)
    return O, rounded


@pytest.mark.parametrize("k,nibble,d,Hq,Hkv,hadamard", [
    (0, False, 64, 32, 4, False), (0, True, 64, 32, 4, True), (1, False, 64, 32, 4, False),
    (4, False, 64, 32, 4, False), (4, False, 128, 32, 8, False), (2, False, 64, 8, 8, False),
    (1, True, 64, 32, 4, False),
])
@pytest.mark.parametrize("n_bits,k_max", [(15, 15), (18, 9)])
def test_shiftav_matches_oracle(dev, k, nibble, d, Hq, Hkv, hadamard, n_bits, k_max):
    """Rounded logits bit-exact, O within 1e-3, on a ragged batch with an empty sequence, a ragged tail,
    several tiles per warp and value rows of very different scales (so that both drop rules fire)."""
    import torch
    case = synth.make_case("shiftav", [1500, 0, 33, 2049, 64], Hq, Hkv, d, k, nibble=nibble, hadamard=hadamard,
                           outliers=True, seed=900 + k + d)
    rng = np.random.default_rng(5)
    scale = np.exp2(rng.integers(-9, 3, size=(case.V.shape[0], Hkv, 1))).astype(np.float16)
    case.V = (case.V * scale).astype(np.float16)             # value exponents g spread over 12 binades
    cfg, cache = build_cache(case, dev, permute_seed=3)
    ws = torch.empty(sa.shiftav_workspace_bytes(cfg, case.batch, cache.max_pages) + 256, dtype=torch.uint8, device=dev)
    ws = ws[(-ws.data_ptr()) % 256:]
    O = torch.full((case.batch, Hq, d), float("nan"), dtype=torch.float32, device=dev)
    zr = torch.full((case.batch, Hq, cache.max_pages * 64), -7, dtype=torch.int32, device=dev)
    sa.decode_attention_shiftav(cfg, cache.handle, t16(case.Q, dev), O, ws, n_bits, k_max, None, zr)
    torch.cuda.synchronize()
    want_O, want_zr = oracle_shiftav(case, n_bits, k_max)
    zr = zr.cpu().numpy()
    for b in range(case.batch):
        T = int(case.lens[b])
        assert np.array_equal(zr[b, :, :T], want_zr[b]), "rounded logits differ (sequence %d)" % b
        assert np.all(zr[b, :, T:] == -7)
    got = O.cpu().numpy()
    assert np.isfinite(got).all()
    assert np.max(np.abs(got - want_O)) <= TOL_O, np.max(np.abs(got - want_O))
    # same result without the test hook (rounded logits in the workspace)
    O2 = torch.full_like(O, float("nan"))
    sa.decode_attention_shiftav(cfg, cache.handle, t16(case.Q, dev), O2, ws, n_bits, k_max)
    torch.cuda.synchronize()
    assert torch.equal(O, O2)


def test_shiftav_long_sequence_and_host_checks(dev):
    import torch
    case = synth.make_case("shiftav_long", [32768], 32, 4, 64, 4, outliers=False, seed=77)
    cfg, cache = build_cache(case, dev, permute_seed=1)
    ws = torch.empty(sa.shiftav_workspace_bytes(cfg, 1, cache.max_pages) + 256, dtype=torch.uint8, device=dev)
    ws = ws[(-ws.data_ptr()) % 256:]
    O = torch.full((1, 32, 64), float("nan"), dtype=torch.float32, device=dev)
    sa.decode_attention_shiftav(cfg, cache.handle, t16(case.Q, dev), O, ws, 15, 15)
    torch.cuda.synchronize()
    want_O, _ = oracle_shiftav(case, 15, 15)
    assert np.max(np.abs(O.cpu().numpy() - want_O)) <= TOL_O
    # a workspace that is too small, or constants outside the supported range, launch nothing
    O.fill_(7.0)
    for bad in (dict(ws=ws[:1024], n=15, k=15, status=4), dict(ws=ws, n=19, k=3, status=1), dict(ws=ws, n=15, k=16, status=1)):
        with pytest.raises(sa.SaError) as err:
            sa.decode_attention_shiftav(cfg, cache.handle, t16(case.Q, dev), O, bad["ws"], bad["n"], bad["k"])
        assert err.value.status == bad["status"]
    torch.cuda.synchronize()
    assert bool((O == 7.0).all())


# ------------------------------------------------------------------------------- fused decode step
@pytest.mark.parametrize("d,Hq,Hkv,code,nibble,hadamard", [
    (64, 32, 4, sa.SA_POTM4, False, False), (64, 32, 4, sa.SA_POT4, True, True), (64, 32, 4, sa.SA_POTM1, True, False),
    (128, 32, 8, sa.SA_POTM2, False, True), (64, 8, 2, sa.SA_INT8, False, False), (64, 16, 1, sa.SA_POTM4, False, False),
    (64, 32, 4, sa.SA_KV_FP16, False, False)])
def test_decode_step_equals_append_then_decode(dev, d, Hq, Hkv, code, nibble, hadamard):
    """sa_decode_step (the decode kernel writes the step's token itself) against sa_append_kv followed by
    the decode call, over several consecutive steps: the same cache bytes, the same lengths, bit-identical
    outputs.  Lengths chosen so that the new token opens a page, opens a 32-key tile, fills a tile, lands
    in an empty sequence, and in one sequence has no mapped page (no append, length unchanged).
    16 query heads on one KV head is the case the call serves with the two separate kernels."""
    import torch
    lens = np.array([64, 31, 95, 0, 4000, 128], dtype=np.int64)
    n_steps = 3
    k = 0 if code in (sa.SA_KV_FP16, sa.SA_INT8) else code
    full = synth.make_case("step", lens + n_steps, Hq, Hkv, d, k, nibble=nibble, hadamard=hadamard, seed=3100 + d + code)
    cfg = sa.make_config(d, Hq, Hkv, code, nibble=nibble, hadamard=hadamard)
    B = len(lens)
    caches = []
    for _ in range(2):
        n_pages = int(np.maximum((lens + n_steps + 63) // 64, 1).sum())
        c = sa.PagedCache(cfg, lens, dev, extra_tokens=n_steps, permutation=synth.page_permutation(n_pages, 21))
        pre = np.concatenate([np.arange(full.cu_lens[b], full.cu_lens[b] + lens[b]) for b in range(B)])
        cu = np.concatenate([[0], np.cumsum(lens)])
        c.fill(t16(full.K[pre], dev), t16(full.V[pre], dev), cu)
        c.page_table[5, 2:] = -1                                # sequence 5 (128 tokens): no page for token 128
        caches.append(c)
    ref, fused = caches
    rng = np.random.default_rng(8)
    for step in range(n_steps):
        new = np.array([full.cu_lens[b] + lens[b] + step for b in range(B)])
        Kn, Vn = t16(full.K[new], dev), t16(full.V[new], dev)
        Q = t16(synth.gaussian_fp16(rng, (B, Hq, d)), dev)
        O1 = torch.full((B, Hq, d), float("nan"), dtype=torch.float32, device=dev)
        O2 = torch.full_like(O1, float("nan"))
        sa.append_kv(cfg, ref.handle, Kn, Vn, True)
        if code == sa.SA_KV_FP16:
            sa.decode_attention_fp16(cfg, ref.handle, Q, O1, ref.workspace)
        else:
            sa.decode_attention(cfg, ref.handle, Q, O1, ref.workspace)
        sa.decode_step(cfg, fused.handle, Q, Kn, Vn, O2, fused.workspace)
        torch.cuda.synchronize()
        want_lens = lens + step + 1
        want_lens[5] = 128
        assert fused.seq_lens.cpu().numpy().tolist() == want_lens.tolist()
        assert ref.seq_lens.cpu().numpy().tolist() == want_lens.tolist()
        assert torch.equal(O1, O2), "step %d: outputs differ" % step
    assert torch.equal(ref.pages, fused.pages)


# ------------------------------------------------------------------------------- randomised shapes
@pytest.mark.parametrize("seed", range(12))
def test_random_shapes_against_oracle(dev, seed):
    """Seeded random draws of the things a caller can vary together — head counts (groups of 1 to 16 query
    heads per KV head), head_dim, code and container, rotation, head-room, ragged lengths with empty and
    one-token sequences, shuffled pages, spare capacity — through sa_decode_step (fused append where the
    group fits one block) and checked against the oracle: integer scores of the extended cache bit-exact,
    outputs within 1e-3."""
    import torch
    rng = np.random.default_rng(7000 + seed)
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3, 8]))
    G = int(rng.choice([1, 2, 4, 8, 16]))
    k, nibble = [(0, False), (0, True), (1, False), (1, True), (2, False), (2, True), (4, False)][int(rng.integers(0, 7))]
    hadamard = bool(rng.integers(0, 2))
    F = 0 if rng.integers(0, 2) else E + k + int(rng.integers(0, 3))
    B = int(rng.integers(1, 6))
    lens = rng.integers(0, 700, size=B)
    lens[rng.integers(0, B)] = int(rng.choice([0, 1, 31, 32, 63, 64, 65, 1500]))
    full = synth.make_case("rand", lens + 1, Hkv * G, Hkv, d, k, nibble=nibble, hadamard=hadamard, outliers=bool(rng.integers(0, 2)),
                           seed=7100 + seed)
    cfg = cfg_of(full, F=F)
    n_pages = int(np.maximum((lens + 1 + 40 + 63) // 64, 1).sum())
    cache = sa.PagedCache(cfg, lens, dev, extra_tokens=41, permutation=synth.page_permutation(n_pages, seed))
    pre = np.concatenate([np.arange(full.cu_lens[b], full.cu_lens[b] + lens[b]) for b in range(B)]).astype(np.int64)
    cache.fill(t16(full.K[pre], dev), t16(full.V[pre], dev), np.concatenate([[0], np.cumsum(lens)]))
    new = np.array([full.cu_lens[b + 1] - 1 for b in range(B)])
    O = torch.full((B, Hkv * G, d), float("nan"), dtype=torch.float32, device=dev)
    sa.decode_step(cfg, cache.handle, t16(full.Q, dev), t16(full.K[new], dev), t16(full.V[new], dev), O, cache.workspace)
    torch.cuda.synchronize()
    assert cache.seq_lens.cpu().numpy().tolist() == (lens + 1).tolist()
    # scores of the extended cache through the plain decode call (test hook), outputs of both calls identical
    O2 = torch.full_like(O, float("nan"))
    dbg = torch.full((B, Hkv * G, cache.max_pages * 64), -7, dtype=torch.int32, device=dev)
    sa.decode_attention(cfg, cache.handle, t16(full.Q, dev), O2, cache.workspace, dbg)
    torch.cuda.synchronize()
    assert torch.equal(O, O2)
    check_against_oracle(full, O.cpu().numpy(), dbg.cpu().numpy(), F=F)


def test_config3_T32k_through_decode_step_in_a_cuda_graph(dev):
    """The benchmark's launch configuration at full size: PoT-M4, batch 1, 32/4 heads, d = 64, a cache of
    32 767 tokens plus the step's new one, sa_decode_step recorded in a CUDA graph and replayed — outputs
    against the oracle over all 32 768 keys, and the appended token's codes bit-exact."""
    import torch
    case = synth.config3(4)
    T = int(case.lens[0])
    cfg = cfg_of(case)
    cache = sa.PagedCache(cfg, np.array([T - 1]), dev, extra_tokens=4, permutation=synth.page_permutation((T + 3 + 63) // 64, 5))
    cache.fill(t16(case.K[:T - 1], dev), t16(case.V[:T - 1], dev), np.array([0, T - 1]))
    Q, Kn, Vn = t16(case.Q, dev), t16(case.K[T - 1:T], dev), t16(case.V[T - 1:T], dev)
    O = torch.full((1, 32, 64), float("nan"), dtype=torch.float32, device=dev)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):                      # warm-up outside the capture, on a side stream
        sa.decode_step(cfg, cache.handle, Q, Kn, Vn, O, cache.workspace)
    torch.cuda.synchronize()
    cache.seq_lens.fill_(T - 1)                          # take the warm-up's append back
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        sa.decode_step(cfg, cache.handle, Q, Kn, Vn, O, cache.workspace)
    O.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    assert int(cache.seq_lens[0]) == T
    check_against_oracle(case, O.cpu().numpy(), None)
    codes = torch.zeros((T, 4, 64), dtype=torch.uint8, device=dev)
    scales = torch.zeros((T, 4), dtype=torch.int16, device=dev)
    sa.debug_unpack(cfg, cache.handle, 0, T, codes, scales)
    torch.cuda.synchronize()
    want_c, want_s = ora.encode_keys(case.K[T - 1:T], 4)
    assert np.array_equal(codes[T - 1:].cpu().numpy(), want_c)
    assert np.array_equal(scales[T - 1:].cpu().numpy().view(np.uint16), want_s.view(np.uint16))


# ------------------------------------------------------ shifts on the integer multiplier (non-default option)
@pytest.mark.parametrize("d,Hq,Hkv", [(64, 32, 4), (128, 8, 2), (64, 6, 2)])
@pytest.mark.parametrize("k,nibble", [(1, False), (1, True), (2, False), (2, True), (4, False)])
def test_shift_by_multiply_gives_the_same_scores(dev, d, Hq, Hkv, k, nibble):
    """SA_FLAG_SHIFT_BY_MULTIPLY: INT32 scores bit-exact against the oracle (hence equal to the shift kernels'),
    outputs within the tolerance; ragged batch with an empty sequence, several tiles, head-room above the default."""
    F = 6 + k + (2 if d == 64 else 0)
    case = synth.make_case("mulshift", [700, 0, 33, 129], Hq, Hkv, d, k, outliers=True, seed=4700 + 10 * k + d, nibble=nibble)
    O, dbg, _ = run_decode(case, dev, F=F, permute_seed=7, shift_by_multiply=True)
    check_against_oracle(case, O, dbg, F=F)


def test_shift_by_multiply_step_matches_the_shift_kernel_bitwise(dev):
    """The fused step with the option on and off: the same appended token, and outputs equal bit for bit
    (the scores are the same integers and everything after them is the same code)."""
    import torch
    case = synth.config3(4, T=4096 + 1)
    T = int(case.lens[0])
    outs = []
    for flag in (False, True):
        cfg = cfg_of(case, shift_by_multiply=flag)
        cache = sa.PagedCache(cfg, np.array([T - 1]), dev, extra_tokens=1)
        cache.fill(t16(case.K[:T - 1], dev), t16(case.V[:T - 1], dev), np.array([0, T - 1]))
        O = torch.full((1, 32, 64), float("nan"), dtype=torch.float32, device=dev)
        sa.decode_step(cfg, cache.handle, t16(case.Q, dev), t16(case.K[T - 1:], dev), t16(case.V[T - 1:], dev), O, cache.workspace)
        torch.cuda.synchronize()
        assert int(cache.seq_lens[0]) == T
        outs.append((O.cpu().numpy(), cache.pages.cpu().numpy()))
    assert np.array_equal(outs[0][0].view(np.uint32), outs[1][0].view(np.uint32))
    assert np.array_equal(outs[0][1], outs[1][1])
    check_against_oracle(case, outs[1][0], None)


# ------------------------------------------- sign flips and adds on the ALU pipe only (non-default option)
@pytest.mark.parametrize("d,Hq,Hkv", [(64, 32, 4), (128, 8, 2), (64, 6, 2)])
@pytest.mark.parametrize("k,nibble", [(0, False), (0, True), (1, True), (2, False), (4, False)])
def test_add_on_alu_gives_the_same_scores(dev, d, Hq, Hkv, k, nibble):
    """SA_FLAG_ADD_ON_ALU (no multiply-add anywhere in the score datapath): INT32 scores bit-exact against the
    oracle, outputs within the tolerance; ragged batch with an empty sequence, head-room above the default."""
    F = 6 + k + (2 if d == 64 else 0)
    case = synth.make_case("addalu", [700, 0, 33, 129], Hq, Hkv, d, k, outliers=True, seed=4900 + 10 * k + d, nibble=nibble)
    O, dbg, _ = run_decode(case, dev, F=F, permute_seed=11, add_on_alu=True)
    check_against_oracle(case, O, dbg, F=F)


def test_add_on_alu_excludes_shift_by_multiply(dev):
    case = synth.make_case("addalu2", [64], 32, 4, 64, 4, seed=1)
    cfg = cfg_of(case, shift_by_multiply=True, add_on_alu=True)
    with pytest.raises(sa.SaError):
        sa.get_layout(cfg)


# ------------------------------------------------------------------ a staged copy that never arrives
@pytest.mark.parametrize("lost", [(1, 2, 3), (0, 0, 0), (2, 3, 9)])
def test_lost_copy_marks_exactly_its_rows_and_returns(dev, lost):
    """The bounded wait of the staged copies, made to run out: the copy of one tile of one (sequence, KV head) is
    never issued (test hook, 2^10 polls).  The call returns, the rows of that KV head's query heads in that
    sequence are NaN, every other row is the ordinary result, and an ordinary call afterwards is unaffected.
    The hook's kernel also takes its first guess at the length ranks wrong on purpose, so every block here repeats
    its query prologue for the sequence the ranks after the dependency wait give it."""
    import torch
    b, kvh, tile = lost
    case = synth.make_case("lost", [300, 513, 777], 32, 4, 64, 4, outliers=True, seed=5100)
    cfg, cache = build_cache(case, dev, permute_seed=3)
    Q = t16(case.Q, dev)
    O = torch.zeros((case.batch, 32, 64), dtype=torch.float32, device=dev)
    sa.debug_decode_lost_copy(cfg, cache.handle, Q, O, cache.workspace, b, kvh, tile)
    torch.cuda.synchronize()                                # the call comes back: nothing waits without a bound
    got = O.cpu().numpy()
    ref = ora.decode_attention(case.Q, case.K, case.V, case.cu_lens, 4, 10, n_threads=8)["O"]
    hit = np.zeros((case.batch, 32), dtype=bool)
    hit[b, kvh * 8:(kvh + 1) * 8] = True
    assert np.isnan(got[hit]).all(), "the rows of the lost tile must be marked"
    assert np.isfinite(got[~hit]).all()
    assert np.max(np.abs(got[~hit] - ref[~hit])) <= TOL_O
    O2 = torch.zeros_like(O)
    sa.decode_attention(cfg, cache.handle, Q, O2, cache.workspace, None)
    torch.cuda.synchronize()
    assert np.max(np.abs(O2.cpu().numpy() - ref)) <= TOL_O


def test_lost_copy_hook_refuses_other_shapes(dev):
    import torch
    case = synth.make_case("lost2", [100], 32, 4, 64, 1, seed=5101)
    cfg, cache = build_cache(case, dev)
    O = torch.zeros((1, 32, 64), dtype=torch.float32, device=dev)
    with pytest.raises(sa.SaError):
        sa.debug_decode_lost_copy(cfg, cache.handle, t16(case.Q, dev), O, cache.workspace, 0, 0, 0)


# ------------------------------------------------------------------ ragged batches: longest sequence first
@pytest.mark.parametrize("batch", [2, 17, 128, 129])
def test_length_ranked_batches_cover_every_sequence_once(dev, batch):
    """Batches up to 128 sequences are dispatched by rank of their cached length (ties by index), larger ones in
    index order: either way every sequence must come out exactly as the oracle's, whatever the mix of equal, empty
    and distinct lengths; and twice in a row bit for bit (the rank is a fixed function of the lengths)."""
    import torch
    rng = np.random.default_rng(6000 + batch)
    lens = rng.integers(0, 200, size=batch)
    lens[rng.integers(0, batch, size=max(1, batch // 4))] = 97          # ties
    lens[0] = 0
    lens[-1] = 199
    case = synth.make_case("ranked", lens, 8, 2, 64, 4, outliers=True, seed=6100 + batch)
    cfg, cache = build_cache(case, dev, permute_seed=5)
    outs = []
    for _ in range(2):
        O = torch.full((case.batch, 8, 64), float("nan"), dtype=torch.float32, device=dev)
        dbg = torch.full((case.batch, 8, cache.max_pages * 64), -7, dtype=torch.int32, device=dev)
        sa.decode_attention(cfg, cache.handle, t16(case.Q, dev), O, cache.workspace, dbg)
        torch.cuda.synchronize()
        outs.append(O.cpu().numpy())
    check_against_oracle(case, outs[0], dbg.cpu().numpy())
    assert np.array_equal(outs[0].view(np.uint32), outs[1].view(np.uint32))


@pytest.mark.parametrize("lens", [[20000] + [40] * 15, [3000, 1] + [0] * 6, [5000] + [33] * 127, [64 * k + 1 for k in range(1, 40)]])
def test_splits_dealt_by_length_for_extreme_mixes(dev, lens):
    """Batches of unequal lengths: the blocks of the grid are dealt to the sequences in proportion to their lengths
    (one sequence may take nearly all of them, more than one pass of the merge kernel; others a single block; some
    blocks none).  Integer scores and outputs as the oracle's, twice in a row bit for bit; the FP16 kernel likewise.
    (The fused step over a batch of unequal lengths: test_decode_step_equals_append_then_decode.)"""
    import torch
    lens = np.asarray(lens)
    case = synth.make_case("mix", lens, 8, 1, 64, 4, outliers=True, seed=6300 + len(lens))
    cfg, cache = build_cache(case, dev, permute_seed=11)
    outs = []
    for _ in range(2):
        O = torch.full((case.batch, 8, 64), float("nan"), dtype=torch.float32, device=dev)
        dbg = torch.full((case.batch, 8, cache.max_pages * 64), -7, dtype=torch.int32, device=dev)
        sa.decode_attention(cfg, cache.handle, t16(case.Q, dev), O, cache.workspace, dbg)
        torch.cuda.synchronize()
        outs.append(O.cpu().numpy())
    check_against_oracle(case, outs[0], dbg.cpu().numpy())
    assert np.array_equal(outs[0].view(np.uint32), outs[1].view(np.uint32))
    # the FP16 kernel deals its blocks the same way
    fcfg = sa.make_config(64, 8, 1, sa.SA_KV_FP16)
    _, fcache = build_cache(case, dev, cfg=fcfg, permute_seed=12)
    O = torch.full((case.batch, 8, 64), float("nan"), dtype=torch.float32, device=dev)
    sa.decode_attention_fp16(fcfg, fcache.handle, t16(case.Q, dev), O, fcache.workspace)
    torch.cuda.synchronize()
    O = O.cpu().numpy()
    for b in range(case.batch):
        if lens[b] == 0:
            assert np.all(O[b] == 0)
            continue
        ref = ora.sdpa_fp16(case.Q[b], case.K[case.cu_lens[b]:case.cu_lens[b + 1]], case.V[case.cu_lens[b]:case.cu_lens[b + 1]])
        assert np.max(np.abs(O[b] - ref)) <= TOL_O


@pytest.mark.parametrize("lens", [[4000, 100, 2500, 100, 37], [640] * 6, [641, 650, 672, 655], [9000] + [1] * 30, [0, 0, 500]])
def test_block_plan_left_for_the_merge_kernel(dev, lens):
    """The words the decode kernel leaves behind the partials for the merge kernel ({first slot, splits} per
    sequence) describe a sound deal of the grid's blocks: at least one split each, no more splits than blocks, the
    sequences' slots back to back in the order longest first (ties by index), equal tile counts -> the host's split
    count each in index order, and otherwise split counts that all come from one tiles-per-block."""
    import torch
    lens = np.asarray(lens)
    B, Hq, d = len(lens), 8, 64
    case = synth.make_case("plan", lens, Hq, 1, d, 4, seed=6400 + B)
    cfg, cache = build_cache(case, dev)
    O = torch.zeros((B, Hq, d), dtype=torch.float32, device=dev)
    ws = cache.workspace
    ws.view(torch.uint8).fill_(0xEE)
    sa.decode_attention(cfg, cache.handle, t16(case.Q, dev), O, ws, None)
    torch.cuda.synchronize()
    need = sa.workspace_bytes(cfg, B, cache.max_pages)
    plan_bytes = (B * 8 + 15) // 16 * 16
    S, rem = divmod(need - plan_bytes, B * Hq * (d + 2) * 4)
    assert rem == 0 and S >= 1
    plan = ws.view(torch.uint8)[need - plan_bytes:need - plan_bytes + B * 8].cpu().numpy().view(np.int32).reshape(B, 2)
    first, cnt = plan[:, 0].astype(np.int64), plan[:, 1].astype(np.int64)
    tiles = (lens + 31) // 32
    assert (cnt >= 1).all() and cnt.sum() <= S * B
    if len(set(tiles.tolist())) == 1:
        assert (cnt == S).all() and (first == np.arange(B) * S).all()
    else:
        order = sorted(range(B), key=lambda j: (-lens[j], j))
        assert [first[j] for j in order] == np.concatenate([[0], np.cumsum(cnt[order])[:-1]]).tolist()
        ok = [tpb for tpb in range(1, int(tiles.max()) + 2) if all(cnt[j] == max(1, -(-tiles[j] // tpb)) for j in range(B))]
        assert ok, "split counts %s do not come from one tiles-per-block (tiles %s)" % (cnt, tiles)
        # ... and the smallest tiles-per-block that fits the grid row was taken, or one close to it
        fits = [tpb for tpb in range(1, int(tiles.max()) + 2) if sum(max(1, -(-t // tpb)) for t in tiles) <= S * B]
        assert min(ok) <= fits[0] * 1.25 + 1
    ref = ora.decode_attention(case.Q, case.K, case.V, case.cu_lens, 4, 10, n_threads=4)["O"]
    assert np.max(np.abs(O.cpu().numpy() - ref)) <= TOL_O


@pytest.mark.parametrize("fp16", [False, True])
def test_rank_follows_lengths_rewritten_by_the_preceding_kernel(dev, fp16):
    """The decode kernels rank the sequences twice: ahead of their dependency wait (a guess, so that the query prologue
    can run early) and after it (the rank that counts; a differing guess repeats the prologue).  Here the kernel in
    front of every call rewrites the lengths so that the order of the sequences flips, back to back with no
    synchronisation in between: each call must come out as the oracle's for the lengths then in force, whichever
    lengths its guess saw."""
    import dataclasses
    import torch
    full = synth.make_case("flip", [700, 400, 450, 700], 32, 4, 64, 4, outliers=not fp16, seed=6200)
    cfg = sa.make_config(64, 32, 4, sa.SA_KV_FP16) if fp16 else None
    cfg, cache = build_cache(full, dev, cfg=cfg, permute_seed=9)
    Q = t16(full.Q, dev)
    orders = [[700, 400, 150, 90], [60, 200, 450, 700], [33, 400, 31, 64], [700, 1, 450, 2]]
    lens_dev = [torch.tensor(o, dtype=torch.int32, device=dev) for o in orders]
    outs = [torch.full((4, 32, 64), float("nan"), dtype=torch.float32, device=dev) for _ in range(12)]
    for i, O in enumerate(outs):                               # nothing synchronises inside this loop
        cache.seq_lens.copy_(lens_dev[i % len(orders)])
        if fp16:
            sa.decode_attention_fp16(cfg, cache.handle, Q, O, cache.workspace)
        else:
            sa.decode_attention(cfg, cache.handle, Q, O, cache.workspace, None)
    torch.cuda.synchronize()
    for j, lens in enumerate(orders):
        rows = np.concatenate([np.arange(full.cu_lens[b], full.cu_lens[b] + lens[b]) for b in range(4)])
        cut = dataclasses.replace(full, K=full.K[rows], V=full.V[rows], cu_lens=np.concatenate([[0], np.cumsum(lens)]))
        if fp16:
            ref = np.stack([ora.sdpa_fp16(cut.Q[b], cut.K[cut.cu_lens[b]:cut.cu_lens[b + 1]], cut.V[cut.cu_lens[b]:cut.cu_lens[b + 1]])
                            for b in range(4)])
        else:
            ref = ora.decode_attention(cut.Q, cut.K, cut.V, cut.cu_lens, 4, 10, n_threads=8)["O"]
        for i in range(j, len(outs), len(orders)):
            assert np.max(np.abs(outs[i].cpu().numpy() - ref)) <= TOL_O, "call %d" % i


# ------------------------------------------------------------------ split-K merge: every block shape and pass count
@pytest.mark.parametrize("code,Hq,Hkv,T", [(4, 8, 1, 20000), (1, 8, 1, 20000), (0, 32, 4, 3000)])
def test_split_merge_with_many_splits(dev, code, Hq, Hkv, T):
    """A single KV head spreads one sequence over up to 295 splits: the merge then runs with its 256-thread blocks
    and (above 192 splits) takes the partials in two passes; 32/4 heads at a short length stay below 96 splits
    (128-thread blocks).  Outputs against the oracle, and identical twice in a row."""
    import torch
    case = synth.make_case("merge", [T], Hq, Hkv, 64, code, outliers=True, seed=7000 + code)
    cfg, cache = build_cache(case, dev, permute_seed=9)
    n_splits = sa.workspace_bytes(cfg, 1, cache.max_pages) // (Hq * 66 * 4)
    assert (n_splits > 192) == (code == 1) and (n_splits <= 96) == (code == 0)
    outs = []
    for _ in range(2):
        O = torch.full((1, Hq, 64), float("nan"), dtype=torch.float32, device=dev)
        sa.decode_attention(cfg, cache.handle, t16(case.Q, dev), O, cache.workspace, None)
        torch.cuda.synchronize()
        outs.append(O.cpu().numpy())
    check_against_oracle(case, outs[0], None)
    assert np.array_equal(outs[0].view(np.uint32), outs[1].view(np.uint32))
