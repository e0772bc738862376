"""Instruction-throughput table for this GPU: `python -m paper_2609_09208_b200.pipebench`.

Times the library's micro-benchmark kernels with CUDA events and prints thread-instructions per
clock per SM for each instruction kind (SM clock read through NVML during the run)."""
from __future__ import annotations

import json
import sys


def main():
    import torch
    from . import binding as sa
    from . import build as sa_build
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
    if len(sys.argv) > 1:
        json.dump(rows, open(sys.argv[1], "w"), indent=1)


if __name__ == "__main__":
    main()
