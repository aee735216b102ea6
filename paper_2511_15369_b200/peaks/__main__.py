"""Builds and runs the micro-benchmarks that give the ceilings `bench.py` reports against (dense INT8 tensor rate of
a bare `tcgen05.mma.kind::i8` issue loop, alone and as a CTA pair, integer instruction issue rates, TMEM load rate
alone and beside running MMAs, the rate at which copies from L2 refill shared memory beside running MMAs, cost of a
satisfied mbarrier wait) and samples the SM clock and the power meanwhile.

    python -m paper_2511_15369_b200.peaks [--sustained]

Needs a B200; prints the probes' text output followed by one JSON line with the clock samples."""
from __future__ import annotations

import json
import os
import statistics
import subprocess
import sys
import threading
import time

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
OUT = os.path.join(HERE, "_build")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def build():
    os.makedirs(OUT, exist_ok=True)
    exes = []
    for name in ("probe", "probe_wait", "probe_feed"):
        exe = os.path.join(OUT, name)
        subprocess.check_call([NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
                               "-I", os.path.join(ROOT, "include"), "-I", os.path.join(os.path.dirname(HERE), "csrc"),
                               os.path.join(HERE, name + ".cu"), "-o", exe])
        exes.append(exe)
    return exes


def main():
    exes = build()
    samples, stop = [], threading.Event()

    def sample():
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(0)
            while not stop.is_set():
                samples.append((time.perf_counter(), int(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)),
                                pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0,
                                int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(h))))
                time.sleep(0.02)
        except Exception:
            pass

    th = threading.Thread(target=sample, daemon=True)
    th.start()
    t0 = time.perf_counter()
    args = ["sustained"] if "--sustained" in sys.argv else []
    rc = 0
    for exe in exes:
        res = subprocess.run([exe] + (args if exe.endswith("probe") else []), capture_output=True, text=True)
        sys.stdout.write(res.stdout)
        rc |= res.returncode
    t1 = time.perf_counter()
    stop.set()
    th.join()
    busy = [s for s in samples if t0 <= s[0] <= t1 and s[2] > 250.0]      # samples taken under load
    mask = 0
    for s in busy:
        mask |= s[3]
    print(json.dumps({"samples_under_load": len(busy),
                      "sm_mhz_median": statistics.median(s[1] for s in busy) if busy else None,
                      "sm_mhz_min": min((s[1] for s in busy), default=None),
                      "power_w_max": max((s[2] for s in busy), default=None),
                      "reasons_mask": hex(mask)}))
    sys.exit(rc)


if __name__ == "__main__":
    main()
