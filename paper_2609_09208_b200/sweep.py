"""Throughput sweep over the workload configurations other than the benchmark's headline:
`python -m paper_2609_09208_b200.sweep [out.json] [--quick]`.

For every cell it builds seeded synthetic caches on the device (enough distinct copies that one pass
reads more than the 126 MB L2), times whole `sa_decode_attention` calls (main kernel + split-K merge) with
CUDA events, and prints keys/s and algorithmic GB/s.  Cells:
  - Llama-1.1B shape (32 query / 4 KV heads, d = 64): T = 4096 PoT-M1 with per-channel outlier keys;
    T = 32768 for every code, with and without the Hadamard flag, batch 1 / 8 / 32, and the FP16 kernel;
  - ragged paged batch 16, lengths uniform in [2048, 16384], PoT-M2;
  - long-context grid (32 query / 8 KV heads, d = 128): T in {1k, 4k, 16k, 64k, 128k} x batch in {1, 8, 32},
    PoT-4 / PoT-M1 / PoT-M4;
  - the shift-based A.V option (eq. (6), (7)) on the T = 32768 shape for PoT-4 nibble and PoT-M4.
"""
from __future__ import annotations

import json
import sys

import numpy as np


def bytes_per_key(d, code, nibble):
    if code == 16:
        return 4 * d
    return (d // 2 + code * d // 8 if nibble else d) + 4 + d         # dense containers: nibbles + k mantissa bit planes


class Cell:
    def __init__(self, dev, lens, Hq, Hkv, d, code, nibble=False, hadamard=False, outliers=True, seed=1, min_bytes=400e6,
                 shiftav=False, shift_by_multiply=False):
        import torch
        from . import binding as sa
        from . import synth
        self.sa, self.torch = sa, torch
        self.cfg = sa.make_config(d, Hq, Hkv, code, nibble=nibble, hadamard=hadamard and code != 16,
                                  shift_by_multiply=shift_by_multiply)      # non-default: shifts on the integer multiplier
        self.fp16 = code == 16
        self.shiftav = shiftav                                # eq. (6), (7) option: N = k_max = 15
        lens = np.asarray(lens, dtype=np.int64)
        self.keys = int(lens.sum()) * Hkv
        self.bytes = self.keys * bytes_per_key(d, code, nibble)
        n_copies = max(1, min(24, int(np.ceil(min_bytes / max(self.bytes, 1)))))
        self.caches, self.Q, self.O = [], [], []
        gen = torch.Generator(device=dev)
        for c in range(n_copies):
            gen.manual_seed(seed * 100 + c)
            n_pages = int(np.maximum((lens + 63) // 64, 1).sum())
            cache = sa.PagedCache(self.cfg, lens, dev, permutation=synth.page_permutation(n_pages, seed + c))
            for b, T in enumerate(lens):          # sequence by sequence keeps the fp16 source tensors small
                T = int(T)
                if T == 0:
                    continue
                K = torch.randn((T, Hkv, d), generator=gen, device=dev, dtype=torch.float32)
                if outliers:
                    K = K * torch.exp(torch.randn((1, Hkv, d), generator=gen, device=dev, dtype=torch.float32))
                V = torch.randn((T, Hkv, d), generator=gen, device=dev, dtype=torch.float32).half()
                sub = sa.SaCache(cache.pages.data_ptr(), cache.page_table[b:b + 1].data_ptr(),
                                 cache.seq_lens[b:b + 1].data_ptr(), 1, cache.max_pages, cache.n_pages)
                sa.fill_kv(self.cfg, sub, K.half(), V, np.array([0, T], dtype=np.int64))
                torch.cuda.synchronize()
                del K, V
            cache.seq_lens.copy_(torch.from_numpy(lens.astype(np.int32)))
            self.caches.append(cache)
            self.Q.append(torch.randn((len(lens), Hq, d), generator=gen, device=dev, dtype=torch.float32).half())
            self.O.append(torch.zeros((len(lens), Hq, d), dtype=torch.float32, device=dev))
        if shiftav:
            raw = torch.empty(sa.shiftav_workspace_bytes(self.cfg, len(lens), self.caches[0].max_pages) + 256,
                              dtype=torch.uint8, device=dev)
            self.shift_ws = raw[(-raw.data_ptr()) % 256:]

    def run_once(self):
        sa = self.sa
        for c, q, o in zip(self.caches, self.Q, self.O):
            if self.fp16:
                sa.decode_attention_fp16(self.cfg, c.handle, q, o, c.workspace)
            elif self.shiftav:
                sa.decode_attention_shiftav(self.cfg, c.handle, q, o, self.shift_ws, 15, 15)
            else:
                sa.decode_attention(self.cfg, c.handle, q, o, c.workspace)

    def time_us(self, reps=10):
        torch = self.torch
        for _ in range(3):
            self.run_once()
        torch.cuda.synchronize()
        # one pass over the caches recorded in a CUDA graph: launched one by one from Python, short calls
        # would be bound by the host's launch rate instead of the GPU
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.run_once()
        graph.replay()
        torch.cuda.synchronize()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for _ in range(reps):
            graph.replay()
        e.record()
        torch.cuda.synchronize()
        return s.elapsed_time(e) * 1e3 / (reps * len(self.caches))


def main():
    import torch
    from . import build as sa_build
    sa_build.build()
    dev = torch.device("cuda:0")
    quick = "--quick" in sys.argv
    out_path = next((a for a in sys.argv[1:] if not a.startswith("--")), None)
    rows = []

    def cell(name, lens, Hq, Hkv, d, code, **kw):
        c = Cell(dev, lens, Hq, Hkv, d, code, **kw)
        us = c.time_us()
        row = {"cell": name, "keys": c.keys, "us_per_call": us, "keys_per_s": c.keys / (us * 1e-6),
               "algorithmic_gbs": c.bytes / (us * 1e-6) / 1e9, "copies": len(c.caches)}
        rows.append(row)
        print("%-46s %10d keys %9.1f us %10.3e keys/s %8.1f GB/s" % (name, c.keys, us, row["keys_per_s"], row["algorithmic_gbs"]), flush=True)
        del c
        torch.cuda.empty_cache()

    names = {0: "pot4", 1: "potm1", 2: "potm2", 4: "potm4", 8: "int8mac", 16: "fp16"}
    cell("cfg1 single head T=1024 pot4", [1024], 1, 1, 64, 0, outliers=False)
    cell("cfg2 llama-1.1B T=4096 potm1 outliers", [4096], 32, 4, 64, 1)
    for B in ([1] if quick else [1, 8, 32]):
        for code, nib, had in [(0, True, False), (0, True, True), (0, False, False), (1, False, False), (1, True, False),
                               (2, False, False), (2, True, False),
                               (4, False, False), (4, False, True), (8, False, False), (16, False, False)]:
            cell("cfg3 T=32768 B=%d %s%s%s" % (B, names[code], ("_nibble" if code == 0 else "_planar") if nib else "", "+hadamard" if had else ""),
                 [32768] * B, 32, 4, 64, code, nibble=nib, hadamard=had, outliers=False)
        for code, nib in ([] if quick else [(0, True), (4, False)]):
            cell("cfg3 T=32768 B=%d %s%s shift-based A.V (N = k_max = 15)" % (B, names[code], "_nibble" if nib else ""),
                 [32768] * B, 32, 4, 64, code, nibble=nib, outliers=False, shiftav=True)
        for code, nib in ([] if quick else [(1, False), (4, False)]):
            cell("cfg3 T=32768 B=%d %s%s shifts on the integer multiplier" % (B, names[code], "_nibble" if nib else ""),
                 [32768] * B, 32, 4, 64, code, nibble=nib, outliers=False, shift_by_multiply=True)
    lens4 = np.random.Generator(np.random.PCG64(4001)).integers(2048, 16385, size=16)
    cell("cfg4 ragged B=16 [2048,16384] potm2", lens4, 32, 4, 64, 2)
    cell("cfg4 ragged B=16 [2048,16384] fp16", lens4, 32, 4, 64, 16)
    Ts = [1024, 16384] if quick else [1024, 4096, 16384, 65536, 131072]
    Bs = [1, 8] if quick else [1, 8, 32]
    for T in Ts:
        for B in Bs:
            for code, nib in [(0, True), (1, False), (4, False)]:
                cell("cfg5 d=128 T=%d B=%d %s%s" % (T, B, names[code], "_nibble" if nib else ""), [T] * B, 32, 8, 128, code,
                     nibble=nib, min_bytes=300e6)
    if out_path:
        json.dump(rows, open(out_path, "w"), indent=1)


if __name__ == "__main__":
    main()
