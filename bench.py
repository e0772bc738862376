#!/usr/bin/env python
"""Benchmark of the decode-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--variant ...]

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
for _name, _base in MULSHIFT.items():
    VARIANTS[_name] = VARIANTS[_base]


def bytes_per_key(d, code_k, nibble, fp16):
    if fp16:
        return 4 * d
    return (d // 2 + code_k * d // 8 if nibble else d) + 4 + d      # dense containers: nibbles + k mantissa bit planes


class Workload:
    """22 layer caches resident in HBM plus the per-layer query / new-token tensors."""

    def __init__(self, dev, variant, layers, T, batch, room_tokens, seed=3000, d=64, Hq=32, Hkv=4):
        import torch
        from paper_2609_09208_b200 import binding as sa
        self.sa = sa
        self.dev = dev
        code_k, nibble, hadamard, fp16 = VARIANTS[variant]
        self.variant, self.layers, self.T, self.batch = variant, layers, T, batch
        self.d, self.Hq, self.Hkv = d, Hq, Hkv
        self.fp16 = fp16
        self.bpk = bytes_per_key(d, code_k, nibble, fp16)
        self.cfg = sa.make_config(d, Hq, Hkv, sa.SA_KV_FP16 if fp16 else code_k, nibble=nibble, hadamard=hadamard,
                                  shift_by_multiply=variant in MULSHIFT)
        self.caches, self.Q, self.Kn, self.Vn, self.O = [], [], [], [], []
        cu = np.arange(batch + 1, dtype=np.int64) * T
        pages_per_seq = (T + room_tokens + 63) // 64
        for l in range(layers):
            gen = torch.Generator(device=dev)
            gen.manual_seed(seed * 1000 + l)
            K = torch.randn((batch * T, Hkv, d), generator=gen, device=dev, dtype=torch.float32).half()
            V = torch.randn((batch * T, Hkv, d), generator=gen, device=dev, dtype=torch.float32).half()
            perm = synth.page_permutation(pages_per_seq * batch, seed + l)
            cache = sa.PagedCache(self.cfg, [T] * batch, dev, extra_tokens=room_tokens, permutation=perm)
            cache.fill(K, V, cu)
            self.caches.append(cache)
            self.Q.append(torch.randn((batch, Hq, d), generator=gen, device=dev, dtype=torch.float32).half())
            self.Kn.append(torch.randn((batch, Hkv, d), generator=gen, device=dev, dtype=torch.float32).half())
            self.Vn.append(torch.randn((batch, Hkv, d), generator=gen, device=dev, dtype=torch.float32).half())
            self.O.append(torch.zeros((batch, Hq, d), dtype=torch.float32, device=dev))
            del K, V
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
    and A.V) on one layer of the workload, cache pre-encoded (not timed), optionally spread over
    the independent KV heads with one host thread each."""

    def __init__(self, variant, T, batch, n_layers, seed=3000):
        from oracle import sa_oracle as ora
        self.ora = ora
        code_k, nibble, hadamard, fp16 = VARIANTS[variant]
        self.k, self.F, self.fp16 = code_k, 6 + code_k, fp16
        self.layers = []
        for l in range(n_layers):
            case = synth.make_case("cpu", [T] * batch, 32, 4, 64, code_k, seed=seed * 1000 + l)
            Q, K = case.Q, case.K
            if hadamard:
                Q, K = ora.hadamard_fp16(Q), ora.hadamard_fp16(K)
            per_head = []
            for b in range(batch):
                rows = slice(case.cu_lens[b], case.cu_lens[b + 1])
                for kv in range(4):
                    Kh = np.ascontiguousarray(K[rows, kv:kv + 1])
                    Vh = np.ascontiguousarray(case.V[rows, kv:kv + 1])
                    Qh = np.ascontiguousarray(Q[b, kv * 8:(kv + 1) * 8])
                    if fp16:
                        per_head.append((Qh, Kh, Vh))
                    else:
                        codes, scales = ora.encode_keys(Kh, code_k)
                        vhat, g = ora.quantise_value(Vh)
                        per_head.append((Qh, codes, scales, vhat, g))
            self.layers.append(per_head)
        self.keys_per_layer = batch * T * 4

    def _unit(self, u):
        ora = self.ora
        if self.fp16:
            return ora.sdpa_fp16(*u)
        Qh, codes, scales, vhat, g = u
        qhat, delta = ora.quantise_query(Qh)
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
    (profiles/pipe_utilisation.txt: variant, batch, then per cent of peak while the SM is active)."""
    path = os.path.join(ROOT, "profiles", "pipe_utilisation.txt")
    rows = []
    try:
        for line in open(path):
            parts = line.split("#")[0].split()
            if len(parts) == 7 and parts[0] == variant:
                rows.append({"batch": int(parts[1]), "issue_slots_pct": float(parts[2]), "alu_pipe_pct": float(parts[3]),
                             "fma_pipe_pct": float(parts[4]), "lsu_pipe_pct": float(parts[5]),
                             "shared_wavefronts_pct": float(parts[6])})
    except Exception:
        pass
    return rows or None


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


def time_steps(fn, n, dev):
    """n calls of fn between two CUDA events on the current stream; returns milliseconds."""
    import torch
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dist_util.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    start.record()
    for _ in range(n):
        fn()
    end.record()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    dist_util.barrier()
    return start.elapsed_time(end), t0, t1


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
    if rank == 0:
        sa_build.build()
    dist_util.barrier()
    from paper_2609_09208_b200 import binding as sa
    sa.lib()

    K, W = args.steps, max(args.warmup, 3)
    n_cont = 200                                            # at most this many extra replays for clock sampling
    room = W + 2 * K + n_cont + 128                         # every append needs a mapped slot
    wl = Workload(dev, args.variant, args.layers, args.seq_len, args.batch, room)

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
    ms, t0, t1 = time_steps(graph.replay, K, dev)
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
    ms_main, _, _ = time_steps(replay_main, K, dev)
    main_us = ms_main / (K * wl.layers) * 1e3
    alg_bytes = wl.algorithmic_bytes_per_main_launch()
    achieved = alg_bytes / (main_us * 1e-6) / 1e9
    peak, peak_kind = measured_hbm_peak()
    # the capture is of one batch-1, T = 32768 launch; traffic grows with the keys a launch reads
    traffic = recorded_traffic(args.variant)
    if traffic is not None:
        traffic = int(traffic * (wl.batch * wl.T) / 32768.0)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "peak_kind": "of %s copy bandwidth" % peak_kind,
                "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "kernel": "decode main kernel (scores + softmax + A.V)", "kernel_us": main_us,
                "algorithmic_bytes_per_launch": alg_bytes,
                "how": "CUDA events around %d back-to-back launches over %d distinct layer caches, replayed from a CUDA graph" % (K * wl.layers, wl.layers)}

    # ---- end to end through the host-buffer entry: pinned H2D of Q / new K,V and D2H of O per layer ----
    # one pinned input buffer per layer, Q | K_new | V_new after one another (the entry then needs one copy)
    Qh, Knh, Vnh = [], [], []
    for l in range(wl.layers):
        nq, nkv = wl.Q[l].numel(), wl.Kn[l].numel()
        buf = torch.empty(nq + 2 * nkv, dtype=torch.float16).pin_memory()
        buf[:nq].copy_(wl.Q[l].reshape(-1))
        buf[nq:nq + nkv].copy_(wl.Kn[l].reshape(-1))
        buf[nq + nkv:].copy_(wl.Vn[l].reshape(-1))
        Qh.append(buf[:nq])
        Knh.append(buf[nq:nq + nkv])
        Vnh.append(buf[nq + nkv:])
    Oh = [torch.zeros((wl.batch, wl.Hq, wl.d), dtype=torch.float32).pin_memory() for _ in range(wl.layers)]
    staging = torch.empty(sa.staging_bytes(wl.cfg, wl.batch), dtype=torch.uint8, device=dev)

    def e2e_calls():
        for l in range(wl.layers):
            c = wl.caches[l]
            sa.decode_step_host(wl.cfg, c.handle, Qh[l], Knh[l], Vnh[l], Oh[l], staging, c.workspace)
    for _ in range(3):
        e2e_calls()
    torch.cuda.synchronize()
    # The calls allocate nothing and never synchronise, so a user can record them once (copies from and to
    # the pinned buffers included) and replay the recording every step, as the device-resident step does.
    e2e_graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(e2e_graph):
        e2e_calls()

    def e2e_step():
        e2e_graph.replay()
        torch.cuda.synchronize()                             # the step's output is on the host
    for _ in range(3):
        e2e_step()
    ms_e2e, _, _ = time_steps(e2e_step, K, dev)
    ms_e2e = dist_util.max_over_ranks(ms_e2e, dev)
    e2e = {"value": keys_all / (ms_e2e / K * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": wl.layers * wl.batch * (wl.Hq + 2 * wl.Hkv) * wl.d * 2,
           "d2h_bytes_per_step": wl.layers * wl.batch * wl.Hq * wl.d * 4, "ms_per_step": ms_e2e / K,
           "api": "sa_decode_step_host per layer: inputs fetched from, and O stored to, device-addressable pinned "
                  "host buffers by the library's kernels (no copy engine); recorded once in a CUDA graph and "
                  "replayed; stream synchronised once per step"}
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
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if wl.fp16 else "int32", "data": "synthetic", "config": workload_config(args),
        "clocks": clocks, "e2e": e2e, "gpu_launches": wl.launches_per_step * K,
        "hbm_gbs_step": value / args.gpus * wl.bpk / 1e9, "roofline": roofline,
        "scores_per_s": value * group,                      # (query, key) scores: keys/s x query heads per KV head
        "cold_call_us": {"median": sorted(cold)[len(cold) // 2], "best": min(cold),
                         "what": "one sa_decode_step call (one layer), L2 flushed before each of 5 calls"},
        "pipe_utilisation": recorded_pipes(args.variant),   # from the ncu captures under profiles/ (not measured live)
    }
    pipes = line["pipe_utilisation"]
    if pipes:
        # The resource that actually binds the shift kernels is the integer ALU pipe (shift, logic, permute):
        # 64 lanes per SM and clock.  Fraction from the recorded capture of the nearest batch size.
        row = min(pipes, key=lambda r: abs(r["batch"] - wl.batch))
        alu_peak = 148 * 64 * (clocks.get("sm_mhz") or 1965.0) * 1e6      # no clock sample in a very short run: the maximum
        line["roofline_alu"] = {"bound": "alu", "peak": alu_peak, "unit": "thread-instr/s", "frac": row["alu_pipe_pct"] / 100.0,
                                "achieved": alu_peak * row["alu_pipe_pct"] / 100.0, "issue_slots_frac": row["issue_slots_pct"] / 100.0,
                                "source": "ncu sm__inst_executed_pipe_alu of the capture at batch %d (profiles/)" % row["batch"]}
    if rank == 0 and args.gpus == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(args.variant, args.seq_len, args.batch)
    if rank == 0 and args.context:
        line["context"] = context_rows(args, dev)
    if rank == 0:
        print(json.dumps(line))
    dist_util.barrier()


def context_rows(args, dev):
    """Other variants / batch sizes at the same T, main kernel only (not part of the headline)."""
    import torch
    rows = []
    for variant, batch in [("fp16", 1), ("pot4_nibble", 1), ("pot4", 1), ("potm1", 1), ("potm4", 8), ("pot4_nibble", 8),
                           ("fp16", 8), ("potm4", 32), ("pot4_nibble", 32), ("fp16", 32)]:
        layers = max(2, min(args.layers, int(400e6 // (batch * args.seq_len * 4 * bytes_per_key(64, *VARIANTS[variant][:2], VARIANTS[variant][3]))) + 1))
        wl = Workload(dev, variant, layers, args.seq_len, batch, 64)

        def main_kernels():
            for l in range(wl.layers):
                wl.decode(l, stages=1)
        replay_main = recorded(main_kernels)
        for _ in range(2):
            replay_main()
        ms, _, _ = time_steps(replay_main, 10, dev)
        us = ms / (10 * wl.layers) * 1e3
        keys = wl.batch * wl.T * wl.Hkv
        rows.append({"variant": variant, "batch": batch, "layers": layers, "main_kernel_us": us,
                     "keys_per_s": keys / (us * 1e-6), "hbm_gbs": wl.algorithmic_bytes_per_main_launch() / (us * 1e-6) / 1e9})
        del wl
        torch.cuda.empty_cache()
    return rows


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
    ap.add_argument("--context", action="store_true", help="also time other variants and batch sizes (main kernel only)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
