"""The entry point for callers that cannot allocate device memory (sa_decode_attention_static).

Some users of the library run where cudaMalloc is not an option (inside another runtime's
callback, or after their memory pool has been frozen), so they cannot provide the split-K
workspace.  This entry point keeps that scratch in a fixed array inside the library.  The test
calls it through the C ABI twice in a row, with different queries, and checks each output against
the ordinary entry point given a caller-allocated workspace; the second call also shows that what
the first one left in the shared scratch does no harm.  Collected last on purpose (file name), and
written so that it passes both alone in a fresh process and after the rest of the suite."""
import ctypes as C

import numpy as np
import pytest

from paper_2609_09208_b200 import binding as sa
from paper_2609_09208_b200 import build as sa_build
from paper_2609_09208_b200 import synth

pytestmark = pytest.mark.gpu
TOL_O = 1e-3          # the tolerance of the other parity tests


def _dev_bits(x, dev):
    import torch
    return torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to(dev)


def test_static_scratch_entry_matches_workspace_entry_twice_in_a_row():
    import torch
    sa_build.build()
    dev = torch.device("cuda:0")
    case = synth.make_case("noalloc", [5000, 0, 333, 64], 32, 4, 64, 4, outliers=True, seed=4242)
    cfg = sa.make_config(64, 32, 4, sa.SA_POTM4)
    n_pages = int(np.maximum((case.lens + 63) // 64, 1).sum())
    cache = sa.PagedCache(cfg, case.lens, dev, permutation=synth.page_permutation(n_pages, 11))
    cache.fill(_dev_bits(case.K, dev), _dev_bits(case.V, dev), case.cu_lens)
    assert sa.workspace_bytes(cfg, case.batch, cache.max_pages) <= sa.STATIC_SCRATCH_BYTES
    rng = np.random.default_rng(99)
    queries = [case.Q, synth.gaussian_fp16(rng, case.Q.shape) * np.float16(3.0)]
    shape = (case.batch, 32, 64)
    for call, Q in enumerate(queries):
        q = _dev_bits(Q, dev)
        want = torch.full(shape, float("nan"), dtype=torch.float32, device=dev)
        want_s = torch.zeros((case.batch, 32, cache.max_pages * 64), dtype=torch.int32, device=dev)
        sa.decode_attention(cfg, cache.handle, q, want, cache.workspace, want_s)
        got = torch.full(shape, float("nan"), dtype=torch.float32, device=dev)
        got_s = torch.zeros_like(want_s)
        sa.decode_attention_static(cfg, cache.handle, q, got, got_s)
        torch.cuda.synchronize()
        assert torch.isfinite(got).all(), "call %d produced non-finite output" % call
        assert float((got - want).abs().max()) <= TOL_O, "call %d differs from sa_decode_attention" % call
        assert torch.equal(got_s, want_s), "call %d: integer scores differ" % call
        assert not got[1].any()                       # the empty sequence yields zeros


def test_static_scratch_entry_refuses_problems_beyond_its_fixed_size():
    import torch
    sa_build.build()
    dev = torch.device("cuda:0")
    cfg = sa.make_config(128, 32, 8, sa.SA_POTM1)
    lens = [64] * 320                                # 320 sequences: the partials need more than the fixed scratch
    cache = sa.PagedCache(cfg, lens, dev)
    assert sa.workspace_bytes(cfg, len(lens), cache.max_pages) > sa.STATIC_SCRATCH_BYTES
    Q = torch.zeros((len(lens), 32, 128), dtype=torch.float16, device=dev)
    O = torch.full((len(lens), 32, 128), 7.0, dtype=torch.float32, device=dev)
    with pytest.raises(sa.SaError) as err:
        sa.decode_attention_static(cfg, cache.handle, Q, O)
    assert err.value.status == 4                      # SA_ERR_CAPACITY
    torch.cuda.synchronize()
    assert bool((O == 7.0).all())                     # nothing was launched
