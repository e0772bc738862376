#!/usr/bin/env python
"""Benchmark of the decode-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--variant ...]
    python bench.py --sweep OUT.json [--quick]     # every workload configuration, with the oracle timed beside it
    python bench.py --pipes OUT.json               # instruction-throughput table of this GPU

Workload (N = 1 and every N: one replica per GPU, weak scaling): the Llama-1.1B-shaped decode
step at T = 32768 with the PoT-M4 8-bit key code — batch 1, 32 query heads sharing 4 KV heads,
head_dim 64, 22 decoder layers each with its own paged KV cache (64-token pages, shuffled page
table).  One step = for every layer: append the new token's K, V to the cache (key encode, value
quantise, cache write) and run decode attention (query quantise, integer shift-accumulate scores,
integer-maximum online softmax, A.V, split-K merge).  The 22 caches total ~380 MB, three times the
126 MB L2, so no layer's cache survives in L2 until the next step.

Timed with CUDA events on the launching stream, barrier + synchronize on both sides, maximum over
ranks; rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_09208_b200 import dist_util  # noqa: E402
from paper_2609_09208_b200 import synth  # noqa: E402

METRIC = "decode_attention_keys_per_s"
UNIT = "keys/s"
NOMINAL_HBM_GBS = 8000.0          # the peak the target is quoted against
FALLBACK_HBM_GBS = 6650.0


# ----------------------------------------------------------------------------------------------
# workload description
# ----------------------------------------------------------------------------------------------
VARIANTS = {
    # name: (code_k, nibble, hadamard, fp16)
    "potm4": (4, False, False, False),
    "potm4_had": (4, False, True, False),
    "potm2": (2, False, False, False),
    "potm1": (1, False, False, False),
    "pot4": (0, False, False, False),
    "pot4_nibble": (0, True, False, False),
    "pot4_nibble_had": (0, True, True, False),
    "potm1_planar": (1, True, False, False),  # dense 5-bit container: sign/exponent nibbles + one mantissa bit plane
    "potm2_planar": (2, True, False, False),  # dense 6-bit container
    "fp16": (0, False, False, True),
    "int8mac": (8, False, False, False),      # uniform INT8 keys, dp4a scores: the paper's multiply-native comparison
}
# the same codes with the shifts executed by the integer multiplier (SA_FLAG_SHIFT_BY_MULTIPLY; not the default)
MULSHIFT = {"potm4_mulshift": "potm4", "potm1_mulshift": "potm1", "potm2_mulshift": "potm2"}
# ... and with every sign flip and add on the ALU pipe, no multiply-add at all (SA_FLAG_ADD_ON_ALU; not the default)
ADDALU = {"potm4_alu": "potm4", "pot4_nibble_alu": "pot4_nibble", "potm1_alu": "potm1"}
for _name, _base in list(MULSHIFT.items()) + list(ADDALU.items()):
    VARIANTS[_name] = VARIANTS[_base]


def bytes_per_key(d, code_k, nibble, fp16):
    if fp16:
        return 4 * d
    return (d // 2 + code_k * d // 8 if nibble else d) + 4 + d      # dense containers: nibbles + k mantissa bit planes


def new_tokens(seed, l, batch, Hkv, d):
    """The step's new K, V rows of layer l (binary16), seeded."""
    rng = np.random.Generator(np.random.PCG64(seed * 1000 + 500 + l))
    return synth.gaussian_fp16(rng, (batch, Hkv, d)), synth.gaussian_fp16(rng, (batch, Hkv, d))


def layer_case(variant, seed, l, T, batch):
    """Layer l of the workload as host arrays: the ONE recipe both the GPU arm and the oracle legs draw from."""
    code_k = VARIANTS[variant][0]
    return synth.make_case("layer%d" % l, [T] * batch, 32, 4, 64, code_k, seed=seed * 1000 + l)


class Workload:
    """Layer caches resident in HBM plus the per-layer query / new-token tensors.

    source = "synth": every layer is generated on the host by layer_case() — the same binary16 bits the CPU
    oracle legs use — and uploaded; "device": drawn on the GPU (context rows at large batch, which no oracle
    leg reads)."""

    def __init__(self, dev, variant, layers, T, batch, room_tokens, seed=3000, d=64, Hq=32, Hkv=4, source="synth"):
        import torch
        from paper_2609_09208_b200 import binding as sa
        self.sa = sa
        self.dev = dev
        code_k, nibble, hadamard, fp16 = VARIANTS[variant]
        self.variant, self.layers, self.T, self.batch = variant, layers, T, batch
        self.d, self.Hq, self.Hkv = d, Hq, Hkv
        self.fp16, self.code_k, self.hadamard, self.seed = fp16, code_k, hadamard, seed
        self.bpk = bytes_per_key(d, code_k, nibble, fp16)
        self.cfg = sa.make_config(d, Hq, Hkv, sa.SA_KV_FP16 if fp16 else code_k, nibble=nibble, hadamard=hadamard,
                                  shift_by_multiply=variant in MULSHIFT, add_on_alu=variant in ADDALU)
        self.caches, self.Q, self.Kn, self.Vn, self.O = [], [], [], [], []
        cu = np.arange(batch + 1, dtype=np.int64) * T
        pages_per_seq = (T + room_tokens + 63) // 64
        to_dev = lambda x: torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).to(dev).view(torch.float16)
        for l in range(layers):
            perm = synth.page_permutation(pages_per_seq * batch, seed + l)
            cache = sa.PagedCache(self.cfg, [T] * batch, dev, extra_tokens=room_tokens, permutation=perm)
            if source == "synth":
                case = layer_case(variant, seed, l, T, batch)
                cache.fill(to_dev(case.K), to_dev(case.V), cu)
                self.Q.append(to_dev(case.Q))
                kn, vn = new_tokens(seed, l, batch, Hkv, d)
                self.Kn.append(to_dev(kn))
                self.Vn.append(to_dev(vn))
                del case
            else:
                gen = torch.Generator(device=dev)
                gen.manual_seed(seed * 1000 + l)
                K = torch.randn((batch * T, Hkv, d), generator=gen, device=dev, dtype=torch.float32).half()
                V = torch.randn((batch * T, Hkv, d), generator=gen, device=dev, dtype=torch.float32).half()
                cache.fill(K, V, cu)
                self.Q.append(torch.randn((batch, Hq, d), generator=gen, device=dev, dtype=torch.float32).half())
                self.Kn.append(torch.randn((batch, Hkv, d), generator=gen, device=dev, dtype=torch.float32).half())
                self.Vn.append(torch.randn((batch, Hkv, d), generator=gen, device=dev, dtype=torch.float32).half())
                del K, V
            self.caches.append(cache)
            self.O.append(torch.zeros((batch, Hq, d), dtype=torch.float32, device=dev))
        torch.cuda.synchronize()
        self.keys_per_step = layers * batch * T * Hkv
        self.launches_per_step = layers * 2          # main kernel (appends the new token), merge

    def decode(self, l, stages=3):
        sa = self.sa
        c = self.caches[l]
        if self.fp16:
            sa.decode_attention_fp16(self.cfg, c.handle, self.Q[l], self.O[l], c.workspace, stages=stages)
        else:
            sa.decode_attention(self.cfg, c.handle, self.Q[l], self.O[l], c.workspace, None, stages=stages)

    def step(self):
        # one decode step per layer through the library's step entry: the decode kernel writes the new token
        # itself (2 kernels per layer: decode and split-K merge)
        for l in range(self.layers):
            c = self.caches[l]
            self.sa.decode_step(self.cfg, c.handle, self.Q[l], self.Kn[l], self.Vn[l], self.O[l], c.workspace)

    def algorithmic_bytes_per_main_launch(self):
        """Cache bytes one main-kernel launch must read, plus its query read and partials write."""
        sa = self.sa
        keys = self.batch * self.T * self.Hkv
        ws = sa.workspace_bytes(self.cfg, self.batch, self.caches[0].max_pages)
        return keys * self.bpk + self.batch * self.Hq * self.d * 2 + ws


# ----------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read-only) every few ms."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, dev):
        super().__init__(daemon=True)
        self.samples = []          # (t, sm_mhz, reasons_mask)
        self.stop_flag = False
        self.ok = False
        self.sm_max = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(dev).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(dev.index or 0)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # pragma: no cover
            self.err = repr(e)

    def _reasons(self):
        nv = self.nv
        for name in ("nvmlDeviceGetCurrentClocksEventReasons", "nvmlDeviceGetCurrentClocksThrottleReasons"):
            fn = getattr(nv, name, None)
            if fn is not None:
                try:
                    return int(fn(self.h))
                except Exception:
                    continue
        return 0

    def run(self):
        if not self.ok:
            return
        while not self.stop_flag:
            try:
                mhz = int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                self.samples.append((time.perf_counter(), mhz, self._reasons()))
            except Exception:
                pass
            time.sleep(0.003)

    def summary(self, t0, t1):
        if not self.ok:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML unavailable"}
        win = [s for s in self.samples if t0 <= s[0] <= t1]
        mask = 0
        for s in win:
            mask |= s[2]
        reasons = [n for b, n in self.REASONS.items() if mask & b]
        return {"sm_mhz": float(np.median([s[1] for s in win])) if win else None, "sm_max_mhz": self.sm_max,
                "reasons": reasons, "samples": len(win)}


# ----------------------------------------------------------------------------------------------
# CPU oracle legs
# ----------------------------------------------------------------------------------------------
class OracleSample:
    """The decode-time stages of the CPU oracle (query quantise, integer scores, two-pass softmax
    and A.V) on layers of a workload, cache pre-encoded (not timed), optionally spread over
    the independent (sequence, KV head) units with one host thread each."""

    def __init__(self, variant, T, batch, n_layers, seed=3000, cases=None, hadamard=None):
        from oracle import sa_oracle as ora
        self.ora = ora
        code_k, nibble, had, fp16 = VARIANTS[variant]
        hadamard = had if hadamard is None else hadamard
        self.k, self.F, self.fp16 = code_k, 6 + code_k, fp16
        self.layers = []
        if cases is None:
            cases = [layer_case(variant, seed, l, T, batch) for l in range(n_layers)]   # the bits the GPU arm uploads
        for case in cases:
            Q, K = case.Q, case.K
            if hadamard:
                Q, K = ora.hadamard_fp16(Q), ora.hadamard_fp16(K)
            G = case.n_q_heads // case.n_kv_heads
            per_head = []
            for b in range(case.batch):
                rows = slice(case.cu_lens[b], case.cu_lens[b + 1])
                if case.cu_lens[b + 1] == case.cu_lens[b]:
                    continue
                for kv in range(case.n_kv_heads):
                    Kh = np.ascontiguousarray(K[rows, kv:kv + 1])
                    Vh = np.ascontiguousarray(case.V[rows, kv:kv + 1])
                    Qh = np.ascontiguousarray(Q[b, kv * G:(kv + 1) * G])
                    if fp16:
                        per_head.append((Qh, Kh, Vh))
                    else:
                        codes, scales = ora.encode_keys_int8(Kh) if code_k == 8 else ora.encode_keys(Kh, code_k)
                        vhat, g = ora.quantise_value(Vh)
                        per_head.append((Qh, codes, scales, vhat, g))
            self.layers.append(per_head)
        self.keys_per_layer = cases[0].n_keys

    def _unit(self, u):
        ora = self.ora
        if self.fp16:
            return ora.sdpa_fp16(*u)
        Qh, codes, scales, vhat, g = u
        qhat, delta = ora.quantise_query(Qh)
        if self.k == 8:                                      # uniform INT8 comparison code
            return ora.attention_twopass_int8(ora.scores_int8(qhat, codes), delta, scales, vhat, g)
        A, _ = ora.scores(qhat, codes, self.k, self.F)
        return ora.attention_twopass(A, delta, scales, vhat, g, self.F)

    def run_layer(self, l, threads):
        units = self.layers[l % len(self.layers)]
        if threads <= 1:
            for u in units:
                self._unit(u)
            return
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(self._unit, units))

    def time_layers(self, n, threads):
        t0 = time.perf_counter()
        for i in range(n):
            self.run_layer(i, threads)
        dt = time.perf_counter() - t0
        return n * self.keys_per_layer / dt, dt


def cpu_baseline(variant, T, batch):
    from oracle import sa_oracle as ora
    hw = ora.hardware_threads() or os.cpu_count() or 1
    sample = OracleSample(variant, T, batch, n_layers=2)
    threads = max(1, min(hw, 4 * batch))
    sample.run_layer(0, 1)                                   # warm the page cache
    v1, t1 = sample.time_layers(48, 1)                       # about 8 s on one core
    vm, tm = sample.time_layers(120, threads)                # about 6 s on four
    stages = None
    code_k, nibble, hadamard, fp16 = VARIANTS[variant]
    if not fp16:
        # one layer through the oracle's whole chain on one core, with its per-stage clocks (the cache build —
        # key encode and value quantise — is not part of a decode step; it is shown for proportion)
        case = synth.make_case("cpu_stages", [T] * batch, 32, 4, 64, code_k if code_k != 8 else 0, seed=4242)
        res = ora.decode_attention(case.Q, case.K, case.V, case.cu_lens, code_k, 6 + (code_k if code_k != 8 else 0),
                                   hadamard=hadamard, n_threads=1)
        st = [float(x) for x in res["stage_seconds"]]
        stages = {"rotate_and_quantise_query": st[0], "encode_keys_and_quantise_values": st[1], "integer_scores": st[2],
                  "softmax_and_av": st[3], "what": "one layer (%d keys), one core, seconds" % (batch * T * 4)}
    return {"value": vm, "unit": UNIT, "cores": threads, "kind": "oracle", "stage_seconds": stages,
            "sample": "decode-time oracle stages (query quantise, integer scores, two-pass softmax + A.V; cache "
                      "pre-encoded) on 120 layer passes of the workload (2 distinct layers, %d keys each), one host "
                      "thread per KV head; %.1f s" % (sample.keys_per_layer, tm),
            "value_1core": v1, "seconds_1core": t1, "host_threads_available": hw}


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the same config / metric."""
    rank, world, _ = dist_util.env_rank_world()
    if rank != 0:
        return
    from oracle import sa_oracle as ora
    hw = ora.hardware_threads() or os.cpu_count() or 1
    sample = OracleSample(args.variant, args.seq_len, args.batch, n_layers=2)
    threads = max(1, min(hw, 4 * args.batch))
    for i in range(args.warmup):
        sample.run_layer(i, threads)
    t0 = time.perf_counter()
    for i in range(args.steps):
        sample.run_layer(i, threads)
    dt = time.perf_counter() - t0
    value = args.steps * sample.keys_per_layer / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(args, note="each step = one layer pass (a bounded sample of the 22-layer step) "
                                             "by the CPU oracle's decode-time stages"),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": "one layer (%d keys) per step, cache pre-encoded, one host thread per KV head"
                                   % sample.keys_per_layer},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(args, note=None):
    cfg = {"workload": "config 3: Llama-1.1B-shaped decode step, batch %d, 32 q heads / 4 KV heads, d=64, T=%d, "
                       "%s key code, %d layer caches, paged (64-token pages, shuffled)" %
                       (args.batch, args.seq_len, args.variant, args.layers),
           "variant": args.variant, "batch": args.batch, "seq_len": args.seq_len, "layers": args.layers,
           "n_q_heads": 32, "n_kv_heads": 4, "head_dim": 64,
           "l2_policy": "inputs larger than L2: %d layer caches are walked per step" % args.layers,
           "parallelism": "replica per GPU (independent sequences/heads, no data-path collective)"}
    if note:
        cfg["note"] = note
    return cfg


# ----------------------------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------------------------
def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def recorded_traffic(variant):
    """DRAM bytes per main-kernel launch from the committed ncu capture (profiles/dram_traffic.txt)."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    try:
        for line in open(path):
            parts = line.split("#")[0].split()
            if len(parts) == 2 and parts[0] == variant:
                return int(parts[1])
    except Exception:
        pass
    return None


def recorded_pipes(variant):
    """Issue-slot and pipe utilisation of the main kernel from the committed ncu capture
    (profiles/pipe_utilisation.txt: a `source` line with the hash of the kernel sources the captures were taken at, then variant,
    batch and per cent of peak while the SM is active).  Recorded figures, not measured by the run that prints them."""
    path = os.path.join(ROOT, "profiles", "pipe_utilisation.txt")
    rows, commit = [], None
    try:
        for line in open(path):
            parts = line.split("#")[0].split()
            if len(parts) == 2 and parts[0] == "source":
                commit = parts[1]
            if len(parts) == 7 and parts[0] == variant:
                rows.append({"batch": int(parts[1]), "issue_slots_pct": float(parts[2]), "alu_pipe_pct": float(parts[3]),
                             "fma_pipe_pct": float(parts[4]), "lsu_pipe_pct": float(parts[5]),
                             "shared_wavefronts_pct": float(parts[6])})
    except Exception:
        pass
    return {"rows": rows, "kernel_source_hash": commit, "describes_this_revision": commit == source_hash(),
            "source": "ncu captures under profiles/, not this run"} if rows else None


def recorded(fn, warm=2):
    """Run fn a few times, then record it once in a CUDA graph and return the replay callable: small kernels
    launched one by one from Python are bound by the host's launch rate (about 12 us per launch), not by the GPU."""
    import torch
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    torch.cuda.synchronize()
    return g.replay


def parity_check(wl, dev):
    """Layer 0 of the workload through sa_decode_attention (with the raw INT32 scores) against the CPU oracle on the
    SAME binary16 bits, before anything is timed.  Returns the record for the JSON line; raises on a mismatch."""
    import torch
    from oracle import sa_oracle as ora
    sa = wl.sa
    case = layer_case(wl.variant, wl.seed, 0, wl.T, wl.batch)
    c = wl.caches[0]
    O = torch.full((wl.batch, wl.Hq, wl.d), float("nan"), dtype=torch.float32, device=dev)
    rec = {"layer": 0, "keys": wl.batch * wl.T * wl.Hkv, "tolerance_O": 1e-3}
    if wl.fp16:
        sa.decode_attention_fp16(wl.cfg, c.handle, wl.Q[0], O, c.workspace)
        torch.cuda.synchronize()
        ref = np.stack([ora.sdpa_fp16(case.Q[b], case.K[case.cu_lens[b]:case.cu_lens[b + 1]],
                                      case.V[case.cu_lens[b]:case.cu_lens[b + 1]]) for b in range(wl.batch)])
        rec["score_mismatches"] = None
    else:
        dbg = torch.full((wl.batch, wl.Hq, c.max_pages * 64), -7, dtype=torch.int32, device=dev)
        sa.decode_attention(wl.cfg, c.handle, wl.Q[0], O, c.workspace, dbg)
        torch.cuda.synchronize()
        hw = ora.hardware_threads() or os.cpu_count() or 1
        res = ora.decode_attention(case.Q, case.K, case.V, case.cu_lens, wl.code_k, 6 + (wl.code_k if wl.code_k != 8 else 0),
                                   hadamard=wl.hadamard, want_scores=True, n_threads=max(1, min(hw, 8)))
        ref = res["O"]
        got = dbg[:, :, :wl.T].cpu().numpy().astype(np.int64)
        rec["score_mismatches"] = int(np.count_nonzero(got != res["A"][:, :, :wl.T]))
        rec["scores_compared"] = int(got.size)
        del dbg
    rec["max_dO"] = float(np.max(np.abs(O.cpu().numpy().astype(np.float64) - ref)))
    rec["what"] = "sa_decode_attention on layer 0 vs the CPU oracle on the same binary16 inputs, before timing"
    if rec["score_mismatches"] or not (rec["max_dO"] <= 1e-3):
        raise SystemExit("parity check failed, nothing was timed: %s" % json.dumps(rec))
    return rec


def time_replays(replay, n, dev):
    """n replays, each between its own pair of CUDA events on the current stream (barrier + synchronize on both
    sides of the whole region).  Returns (total ms from the first event to the last, list of per-replay ms, t0, t1)."""
    import torch
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
    dist_util.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    ev[0].record()
    for i in range(n):
        replay()
        ev[i + 1].record()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    dist_util.barrier()
    return ev[0].elapsed_time(ev[n]), [ev[i].elapsed_time(ev[i + 1]) for i in range(n)], t0, t1


def source_hash():
    """Short hash of the kernel sources and the C header: names the revision of the kernels a number belongs to
    (the ncu captures under profiles/ record the same hash)."""
    import glob
    import hashlib
    h = hashlib.sha1()
    files = sorted(glob.glob(os.path.join(ROOT, "paper_2609_09208_b200", "csrc", "*.cu*"))) + [os.path.join(ROOT, "include", "sa.h")]
    for f in files:
        h.update(os.path.basename(f).encode())
        h.update(open(f, "rb").read())
    return h.hexdigest()[:12]


def run_ours(args):
    import torch
    rank, world, local_rank = dist_util.env_rank_world()
    if world != args.gpus:
        if args.gpus != 1:
            raise SystemExit("launch with torchrun for --gpus > 1 (WORLD_SIZE=%d, --gpus=%d)" % (world, args.gpus))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist_util.init_from_env("nccl")
    from paper_2609_09208_b200 import build as sa_build
    if rank == 0 and not args.no_build:
        sa_build.build()
    dist_util.barrier()
    from paper_2609_09208_b200 import binding as sa
    sa.lib()

    K, W = args.steps, max(args.warmup, 3)
    n_cont = 200                                            # at most this many extra replays for clock sampling
    room = W + 2 * K + n_cont + 128                         # every append needs a mapped slot
    wl = Workload(dev, args.variant, args.layers, args.seq_len, args.batch, room,
                  source="device" if args.device_inputs else "synth")

    # ---- parity first: one layer against the CPU oracle on the same bits (aborts on a mismatch) ----
    parity = None
    if rank == 0 and not args.device_inputs and not args.no_parity:
        parity = parity_check(wl, dev)
    dist_util.barrier()

    # ---- capture one step (append + decode for every layer) in a CUDA graph ----
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        wl.step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        wl.step()
    torch.cuda.synchronize()

    sampler = ClockSampler(dev)
    sampler.start()
    for _ in range(W):
        graph.replay()
    ms, per_step, t0, t1 = time_replays(graph.replay, K, dev)
    # the timed region can be shorter than a few NVML samples: keep the same load running a little
    # longer (untimed) so that the clock record describes this load
    tc0 = time.perf_counter()
    done = 0
    while time.perf_counter() - tc0 < 0.25 and done < n_cont:
        for _ in range(8):
            graph.replay()
        done += 8
        torch.cuda.synchronize()
    tc1 = time.perf_counter()
    clocks = sampler.summary(t0, tc1)
    clocks["window"] = "timed region plus %.2f s of the same replay" % (tc1 - tc0)
    ms = dist_util.max_over_ranks(ms, dev)
    keys_all = dist_util.sum_over_ranks(wl.keys_per_step, dev)
    ms_per_step = ms / K
    value = keys_all / (ms_per_step * 1e-3)

    # ---- the dominant kernel alone: main decode kernel over the 22 caches back to back ----
    def main_kernels():
        for l in range(wl.layers):
            wl.decode(l, stages=1)
    replay_main = recorded(main_kernels)
    for _ in range(2):
        replay_main()
    ms_main, per_main, _, _ = time_replays(replay_main, K, dev)
    main_us = ms_main / (K * wl.layers) * 1e3
    alg_bytes = wl.algorithmic_bytes_per_main_launch()
    achieved = alg_bytes / (main_us * 1e-6) / 1e9
    peak, peak_kind = measured_hbm_peak()
    # the capture is of one batch-1, T = 32768 launch; traffic grows with the keys a launch reads
    traffic = recorded_traffic(BASE_OF.get(args.variant, args.variant))
    if traffic is not None:
        traffic = int(traffic * (wl.batch * wl.T) / 32768.0)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "peak_kind": "of %s copy bandwidth" % peak_kind,
                "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "kernel": "decode main kernel (scores + softmax + A.V)", "kernel_us": main_us,
                "kernel_us_median": float(np.median(per_main)) / wl.layers * 1e3,
                "kernel_us_best": float(np.min(per_main)) / wl.layers * 1e3,
                "algorithmic_bytes_per_launch": alg_bytes,
                "how": "CUDA events around %d back-to-back launches over %d distinct layer caches, replayed from a CUDA graph "
                       "(one event pair per replay: mean, median and best are of %d replays)" % (K * wl.layers, wl.layers, K)}

    # ---- end to end through the host-buffer entry: pinned H2D of Q / new K,V and D2H of O per layer ----
    # one pinned input buffer per layer, Q | K_new | V_new after one another (the entry then needs one copy)
    def host_buffers(offset_halves):
        Qh, Knh, Vnh = [], [], []
        for l in range(wl.layers):
            nq, nkv = wl.Q[l].numel(), wl.Kn[l].numel()
            buf = torch.empty(nq + 2 * nkv + offset_halves, dtype=torch.float16).pin_memory()[offset_halves:]
            buf[:nq].copy_(wl.Q[l].reshape(-1))
            buf[nq:nq + nkv].copy_(wl.Kn[l].reshape(-1))
            buf[nq + nkv:].copy_(wl.Vn[l].reshape(-1))
            Qh.append(buf[:nq])
            Knh.append(buf[nq:nq + nkv])
            Vnh.append(buf[nq + nkv:])
        Oh = [torch.zeros((wl.batch, wl.Hq, wl.d), dtype=torch.float32).pin_memory() for _ in range(wl.layers)]
        return Qh, Knh, Vnh, Oh
    staging = torch.empty(sa.staging_bytes(wl.cfg, wl.batch), dtype=torch.uint8, device=dev)

    def e2e_time(offset_halves):
        Qh, Knh, Vnh, Oh = host_buffers(offset_halves)

        def calls():
            for l in range(wl.layers):
                c = wl.caches[l]
                sa.decode_step_host(wl.cfg, c.handle, Qh[l], Knh[l], Vnh[l], Oh[l], staging, c.workspace)
        for _ in range(3):
            calls()
        torch.cuda.synchronize()
        # The calls allocate nothing and never synchronise, so a user can record them once (copies from and to
        # the pinned buffers included) and replay the recording every step, as the device-resident step does.
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            calls()

        def step():
            g.replay()
            torch.cuda.synchronize()                         # the step's output is on the host
        for _ in range(3):
            step()
        ms_e, per_e, _, _ = time_replays(step, K, dev)
        return dist_util.max_over_ranks(ms_e, dev), per_e
    ms_e2e, per_e2e = e2e_time(0)
    # the same with host buffers that are pinned but not 16-byte aligned: the entry then cannot let its kernels
    # address them and falls back to copy-engine transfers (what pageable or unmapped memory would get)
    ms_copy, _ = e2e_time(4)
    e2e = {"value": keys_all / (ms_e2e / K * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": wl.layers * wl.batch * (wl.Hq + 2 * wl.Hkv) * wl.d * 2,
           "d2h_bytes_per_step": wl.layers * wl.batch * wl.Hq * wl.d * 4, "ms_per_step": ms_e2e / K,
           "ms_per_step_median": float(np.median(per_e2e)), "ms_per_step_best": float(np.min(per_e2e)),
           "ms_per_step_copy_engine_branch": ms_copy / K,
           "api": "sa_decode_step_host per layer.  This figure needs device-mapped, 16-byte aligned pinned host buffers: "
                  "the library's kernels then fetch the inputs from, and store O to, host memory themselves (no copy "
                  "engine).  With any other host memory the entry issues cudaMemcpyAsync transfers instead "
                  "(ms_per_step_copy_engine_branch).  Recorded once in a CUDA graph and replayed; stream synchronised once per step"}
    sampler.stop_flag = True

    # ---- cold single call: one layer's step with L2 flushed (a 256 MB buffer written) before every call ----
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cold = []
    for r in range(5):
        flush.fill_(r)
        c = wl.caches[r % wl.layers]
        ev0.record()
        sa.decode_step(wl.cfg, c.handle, wl.Q[0], wl.Kn[0], wl.Vn[0], wl.O[0], c.workspace)
        ev1.record()
        torch.cuda.synchronize()
        cold.append(ev0.elapsed_time(ev1) * 1e3)
    del flush
    group = wl.Hq // wl.Hkv

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K, "warmup": W,
        "ms_per_step": ms_per_step, "ms_per_step_median": float(np.median(per_step)), "ms_per_step_best": float(np.min(per_step)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if wl.fp16 else "int32", "data": "synthetic", "config": workload_config(args),
        "clocks": clocks, "parity": parity, "e2e": e2e, "gpu_launches": wl.launches_per_step * K,
        "hbm_gbs_step": value / args.gpus * wl.bpk / 1e9, "roofline": roofline,
        "scores_per_s": value * group,                      # (query, key) scores: keys/s x query heads per KV head
        "cold_call_us": {"median": sorted(cold)[len(cold) // 2], "best": min(cold),
                         "what": "one sa_decode_step call (one layer), L2 flushed before each of 5 calls"},
        "pipe_utilisation": recorded_pipes(BASE_OF.get(args.variant, args.variant) if args.variant in MULSHIFT else args.variant),
        "kernel_source_hash": source_hash(),
    }
    pipes = line["pipe_utilisation"]
    if pipes and pipes.get("rows"):
        # The resource that actually binds the shift kernels is the integer ALU pipe (shift, logic, permute):
        # 64 lanes per SM and clock.  Fraction from the recorded capture of the nearest batch size.
        row = min(pipes["rows"], key=lambda r: abs(r["batch"] - wl.batch))
        n_sms = torch.cuda.get_device_properties(dev).multi_processor_count
        alu_peak = n_sms * 64 * (clocks.get("sm_mhz") or 1965.0) * 1e6    # no clock sample in a very short run: the maximum
        line["roofline_alu"] = {"bound": "alu", "peak": alu_peak, "unit": "thread-instr/s", "frac": row["alu_pipe_pct"] / 100.0,
                                "achieved": alu_peak * row["alu_pipe_pct"] / 100.0, "issue_slots_frac": row["issue_slots_pct"] / 100.0,
                                "source": "ncu sm__inst_executed_pipe_alu of the capture at batch %d, kernel sources %s (profiles/); "
                                          "not measured by this run" % (row["batch"], pipes.get("kernel_source_hash"))}
    code_k = VARIANTS[args.variant][0]
    if code_k in (1, 2, 4) and not wl.fp16:
        # The floor of the table datapath of the mantissa codes, measured live: every (key, element, query pair) update
        # gathers one 8-byte table entry from shared memory, and an SM's shared-memory pipe moves 128 bytes per clock
        # (profiles/instruction_throughput_b200.md: a 64-bit gather is two wavefronts wherever its lanes point).
        pairs = (group + 1) // 2
        table_bytes = wl.batch * wl.T * wl.Hkv * wl.d * pairs * 8.0      # per launch: one layer's cached keys
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        smem_peak = sms * 128.0 * (clocks.get("sm_mhz") or 1965.0) * 1e6
        line["roofline_shared"] = {"bound": "shared-memory pipe", "unit": "B/s", "peak": smem_peak,
                                   "achieved": table_bytes / (main_us * 1e-6), "frac": table_bytes / (main_us * 1e-6) / smem_peak,
                                   "what": "table entries gathered per launch (keys x head_dim x query pairs x 8 B) / main kernel "
                                           "time, against SMs x 128 B/clk x sampled SM clock; the kernel's other shared-memory "
                                           "traffic (key codes, values, weights) is not counted"}
    if rank == 0 and args.gpus == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(args.variant, args.seq_len, args.batch)
    if rank == 0 and args.gpus == 1 and not args.no_context:
        del wl, graph, staging
        torch.cuda.empty_cache()
        line["context"] = context_rows(args, dev)
    if rank == 0:
        print(json.dumps(line))
    dist_util.barrier()


# the recorded captures are of the default kernels; a labelled variant reads its base code's DRAM traffic
BASE_OF = dict(list(MULSHIFT.items()) + list(ADDALU.items()))


def context_rows(args, dev):
    """The main kernel alone for the other variants and batch sizes at the same T (cells of the paper's Table III
    grid and the labelled datapath variants), inputs drawn on the device.  Not part of the headline."""
    import torch
    variants = ["fp16", "int8mac", "pot4_nibble", "potm4"]
    cells = [(v, b) for b in (1, 8, 32) for v in variants]
    cells += [("potm4_alu", 1), ("potm4_mulshift", 1), ("potm4_alu", 32), ("potm4_mulshift", 32),
              ("pot4_nibble_alu", 32), ("potm1", 1), ("potm1", 32)]
    rows, us_of = [], {}
    for variant, batch in cells:
        code_k, nibble, _, fp16 = VARIANTS[variant]
        layer_bytes = batch * args.seq_len * 4 * bytes_per_key(64, code_k, nibble, fp16)
        layers = max(2, min(args.layers, int(400e6 // layer_bytes) + 1))
        wl = Workload(dev, variant, layers, args.seq_len, batch, 64, source="device")

        def main_kernels():
            for l in range(wl.layers):
                wl.decode(l, stages=1)
        replay_main = recorded(main_kernels)
        for _ in range(2):
            replay_main()
        ms, per, _, _ = time_replays(replay_main, 10, dev)
        us = ms / (10 * wl.layers) * 1e3
        keys = wl.batch * wl.T * wl.Hkv
        us_of[(variant, batch)] = us
        rows.append({"variant": variant, "batch": batch, "layers": layers, "main_kernel_us": us,
                     "main_kernel_us_best": float(np.min(per)) / wl.layers * 1e3, "keys_per_s": keys / (us * 1e-6),
                     "hbm_gbs": wl.algorithmic_bytes_per_main_launch() / (us * 1e-6) / 1e9})
        del wl, replay_main
        torch.cuda.empty_cache()
    derived = []
    r_int8 = bytes_per_key(64, 8, False, False)
    for b in (1, 8, 32):
        d = {"batch": b}
        for v in ("potm4", "pot4_nibble"):
            code_k, nibble, _, _ = VARIANTS[v]
            # speed relative to the in-library FP16 kernel on the same shapes (> 1: faster than FP16)
            d["%s_vs_fp16" % v] = us_of[("fp16", b)] / us_of[(v, b)]
            # eq. (10): the time a shift-native datapath as fast as the MAC kernel per byte would take
            t_proj = us_of[("int8mac", b)] * bytes_per_key(64, code_k, nibble, False) / r_int8
            d["%s_t_proj_us" % v] = t_proj
            d["%s_measured_over_projected" % v] = us_of[(v, b)] / t_proj
        derived.append(d)
    return {"rows": rows, "derived": derived,
            "what": "main decode kernel only, T = %d, 32/4 heads, d = 64, device-drawn N(0,1) inputs; *_vs_fp16 = t_fp16 / t_code; "
                    "t_proj = t_int8mac * bytes_per_key(code) / bytes_per_key(int8) (eq. (10))" % args.seq_len}


# ----------------------------------------------------------------------------------------------
# sweep over all workload configurations (with the oracle timed beside every cell) and the pipe table
# ----------------------------------------------------------------------------------------------
SWEEP_CODES = {0: "pot4", 1: "potm1", 2: "potm2", 4: "potm4", 8: "int8mac", 16: "fp16"}


class SweepCell:
    """Seeded synthetic caches of one cell on the device, enough distinct copies that one pass reads more than L2."""

    def __init__(self, dev, lens, Hq, Hkv, d, code, nibble=False, hadamard=False, outliers=True, seed=1, min_bytes=400e6,
                 shiftav=False, shift_by_multiply=False, add_on_alu=False):
        import torch
        from paper_2609_09208_b200 import binding as sa
        self.sa, self.torch = sa, torch
        self.cfg = sa.make_config(d, Hq, Hkv, code, nibble=nibble, hadamard=hadamard and code != 16,
                                  shift_by_multiply=shift_by_multiply, add_on_alu=add_on_alu)
        self.fp16 = code == 16
        self.shiftav = shiftav                                # eq. (6), (7) option: N = k_max = 15
        lens = np.asarray(lens, dtype=np.int64)
        self.keys = int(lens.sum()) * Hkv
        self.bytes = self.keys * bytes_per_key(d, code if code != 16 else 0, nibble, code == 16)
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


_ORACLE_CACHE = {}


def oracle_rate(lens, Hq, Hkv, d, code, hadamard, outliers, token_cap=1 << 17):
    """keys/s of the CPU oracle's decode-time stages on this shape, on one host thread and on all (sequence, KV head)
    units in parallel.  Shapes above token_cap tokens are timed on their first sequences up to the cap (at least
    one, cut to the cap if longer) and labelled extrapolated: the oracle's cost is linear in the keys."""
    if code == 16:
        variant = "fp16"
    else:
        variant = SWEEP_CODES[code]
    lens = [int(x) for x in lens if x > 0]
    sample, tot = [], 0
    for T in lens:
        if tot >= token_cap:
            break
        T = min(T, token_cap - tot) if tot + T > token_cap else T
        sample.append(T)
        tot += T
    key = (tuple(sample), Hq, Hkv, d, variant, hadamard, outliers)
    if key not in _ORACLE_CACHE:
        from oracle import sa_oracle as ora
        case = synth.make_case("oracle", sample, Hq, Hkv, d, VARIANTS[variant][0], outliers=outliers, seed=77)
        smp = OracleSample(variant, 0, 0, 1, cases=[case], hadamard=hadamard and code != 16)
        hw = ora.hardware_threads() or os.cpu_count() or 1
        threads = max(1, min(hw, len(smp.layers[0])))
        smp.run_layer(0, 1)
        reps = max(1, int(2e5 // max(case.n_keys, 1)))
        v1, _ = smp.time_layers(reps, 1)
        vm, _ = smp.time_layers(reps, threads)
        _ORACLE_CACHE[key] = {"oracle_keys_per_s_1thread": v1, "oracle_keys_per_s_threads": vm, "oracle_threads": threads,
                              "oracle_sample_tokens": tot}
    return dict(_ORACLE_CACHE[key], oracle_extrapolated=tot < sum(lens))


def run_sweep(args):
    """Every workload configuration other than the headline: whole sa_decode_attention calls (main kernel + split-K
    merge) timed with CUDA events on seeded device-drawn inputs, and the CPU oracle timed beside every cell on
    host arrays of the same shape and distribution."""
    import torch
    from paper_2609_09208_b200 import build as sa_build
    if not args.no_build:
        sa_build.build()
    dev = torch.device("cuda:0")
    quick = args.quick
    rows = []

    def cell(name, lens, Hq, Hkv, d, code, *, oracle=True, **kw):
        c = SweepCell(dev, lens, Hq, Hkv, d, code, **kw)
        us = c.time_us()
        row = {"cell": name, "keys": c.keys, "us_per_call": us, "keys_per_s": c.keys / (us * 1e-6),
               "algorithmic_gbs": c.bytes / (us * 1e-6) / 1e9, "copies": len(c.caches)}
        del c
        torch.cuda.empty_cache()
        if oracle and not args.no_cpu_baseline:
            row.update(oracle_rate(lens, Hq, Hkv, d, code, kw.get("hadamard", False), kw.get("outliers", True)))
        rows.append(row)
        print("%-58s %10d keys %9.1f us %10.3e keys/s %8.1f GB/s   oracle %s" % (
            name, row["keys"], us, row["keys_per_s"], row["algorithmic_gbs"],
            ("%.2e / %.2e keys/s (1 / %d threads)%s" % (row["oracle_keys_per_s_1thread"], row["oracle_keys_per_s_threads"],
                                                       row["oracle_threads"], " extrapolated" if row["oracle_extrapolated"] else ""))
            if "oracle_threads" in row else "-"), flush=True)

    names = SWEEP_CODES
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
                 [32768] * B, 32, 4, 64, code, nibble=nib, outliers=False, shiftav=True, oracle=False)
        for code, nib in ([] if quick else [(1, False), (4, False)]):
            cell("cfg3 T=32768 B=%d %s%s shifts on the integer multiplier" % (B, names[code], "_nibble" if nib else ""),
                 [32768] * B, 32, 4, 64, code, nibble=nib, outliers=False, shift_by_multiply=True, oracle=False)
        for code, nib in ([] if quick else [(0, True), (4, False)]):
            cell("cfg3 T=32768 B=%d %s%s adds on the ALU pipe" % (B, names[code], "_nibble" if nib else ""),
                 [32768] * B, 32, 4, 64, code, nibble=nib, outliers=False, add_on_alu=True, oracle=False)
    lens4 = np.random.Generator(np.random.PCG64(4001)).integers(2048, 16385, size=16)
    cell("cfg4 ragged B=16 [2048,16384] potm2", lens4, 32, 4, 64, 2)
    cell("cfg4 uniform B=16 T=%d potm2 (same mean length)" % int(lens4.mean()), [int(lens4.mean())] * 16, 32, 4, 64, 2, oracle=False)
    cell("cfg4 ragged B=16 [2048,16384] fp16", lens4, 32, 4, 64, 16)
    for draw in ([] if quick else [2, 3]):          # other draws of the same distribution (other capacities, other split counts)
        lens_d = np.random.Generator(np.random.PCG64(4000 + draw)).integers(2048, 16385, size=16)
        cell("cfg4 ragged B=16 [2048,16384] potm2, draw %d" % draw, lens_d, 32, 4, 64, 2, oracle=False)
        cell("cfg4 uniform B=16 T=%d potm2 (mean of draw %d)" % (int(lens_d.mean()), draw), [int(lens_d.mean())] * 16, 32, 4, 64, 2,
             oracle=False)
    Ts = [1024, 16384] if quick else [1024, 4096, 16384, 65536, 131072]
    Bs = [1, 8] if quick else [1, 8, 32]
    for T in Ts:
        for B in Bs:
            for code, nib in [(0, True), (1, False), (4, False)]:
                cell("cfg5 d=128 T=%d B=%d %s%s" % (T, B, names[code], "_nibble" if nib else ""), [T] * B, 32, 8, 128, code,
                     nibble=nib, min_bytes=300e6)
    json.dump(rows, open(args.sweep, "w"), indent=1)


def run_pipes(args):
    """Instruction-throughput table of this GPU: CUDA events around the library's micro-benchmark kernels, SM clock read
    through NVML during the run; thread-instructions per clock per SM for each instruction kind."""
    import torch
    from paper_2609_09208_b200 import binding as sa
    from paper_2609_09208_b200 import build as sa_build
    if not args.no_build:
        sa_build.build()
    dev = torch.device("cuda:0")
    props = torch.cuda.get_device_properties(dev)
    sms = props.multi_processor_count
    try:
        import pynvml
        pynvml.nvmlInit()
        h = pynvml.nvmlDeviceGetHandleByIndex(0)
        clock = lambda: pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)
    except Exception:
        clock = lambda: props.clock_rate / 1000.0
    sink = torch.zeros(4, dtype=torch.int32, device=dev)
    blocks, iters = sms * 8, 2000
    rows = {}
    for kind, name in enumerate(sa.PIPE_KINDS):
        sa.pipe_microbench(kind, 50, blocks, sink)
        torch.cuda.synchronize()
        best, mhz = None, None
        for _ in range(3):
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record()
            sa.pipe_microbench(kind, iters, blocks, sink)
            mhz_now = clock()
            e.record()
            torch.cuda.synchronize()
            ms = s.elapsed_time(e)
            if best is None or ms < best:
                best, mhz = ms, mhz_now
        per_thread = iters * 64 * sa.PIPE_KIND_INSTR.get(name, 1)
        total = per_thread * 256 * blocks
        rate = total / (best * 1e-3) / (mhz * 1e6) / sms
        rows[name] = {"ms": best, "sm_mhz": mhz, "thread_instr_per_clk_per_sm": rate}
        print("%-16s %8.3f ms  %5d MHz  %7.1f thread-instr/clk/SM" % (name, best, mhz, rate))
    json.dump(rows, open(args.pipes, "w"), indent=1)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", default="potm4", choices=sorted(VARIANTS))
    ap.add_argument("--seq-len", type=int, default=32768)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--layers", type=int, default=synth.LLAMA_1B_LAYERS)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-context", action="store_true", help="skip the other variants and batch sizes (main kernel only rows)")
    ap.add_argument("--no-parity", action="store_true", help="skip the oracle check of layer 0 before timing")
    ap.add_argument("--no-build", action="store_true", help="use libsa.so as it is (e.g. an ablation build)")
    ap.add_argument("--device-inputs", action="store_true",
                    help="draw the inputs on the GPU instead of uploading the oracle legs' host arrays (large batches; no parity leg)")
    ap.add_argument("--sweep", metavar="OUT.json", help="run the sweep over all workload configurations instead")
    ap.add_argument("--pipes", metavar="OUT.json", help="run the instruction-throughput micro-benchmarks instead")
    ap.add_argument("--quick", action="store_true", help="with --sweep: a reduced grid")
    ap.add_argument("--source-hash", action="store_true", help="print the hash of the kernel sources and exit")
    args = ap.parse_args()
    if args.source_hash:
        print(source_hash())
        return
    if args.sweep:
        return run_sweep(args)
    if args.pipes:
        return run_pipes(args)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
