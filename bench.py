#!/usr/bin/env python
"""Benchmark of the TuNA hot path on one B200 (or N independent replicas).

A step is one pass of the whole path over one batch: the device-side re-plan
for the batch's counts (count-metadata exchange + segmented prefix sums), then
the exchange itself (one fused pack-move-unpack launch per digit phase and the
rotation launch).  The headline workload is the mixture-of-experts token
dispatch shape (P = 64 ranks, 8192 tokens per rank routed top-2, 8 KiB rows,
8 GiB of payload) at the radix named by --radix; the other schedules (radix
sweep, hierarchical, the single-pass direct exchange) are timed the same way
and reported under "sweep".

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "alltoallv_payload_throughput"
UNIT = "GB/s"

# DRAM traffic of the dominant kernel from ncu captures of it
# (dram__bytes_read.sum + dram__bytes_write.sum per launch) divided by the payload
# bytes that launch moved, keyed by the SHA-256 of the kernel source the capture
# was taken with, then by "workload/schedule".  Traffic grows in proportion to the
# bytes moved, so the full-size figure is this ratio times the launch's bytes.  A
# changed source makes the figures stale: the traffic is then reported as null.
NCU_TRAFFIC_PER_PAYLOAD_BYTE: dict[str, dict[str, float]] = {
    "3caae7ab91d126f8fdb8d1198d3337598395d5529248d37da030b3ef7b8b2b48": {
        "c4/flat radix 64": 1.997,                                  # reduced to 2 GiB for the capture
        "c5/flat radix 2048": 2.166, "c5/flat radix 2": 2.256,      # at full size (0.75 GB)
        "c3/hierarchical l=16 g=16 radix 16/16": 1.539,             # at full size, both launches
    },
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4", choices=["c1", "c2", "c3", "c4", "c4_skew", "c5", "normal", "powerlaw", "fft_n1", "fft_n2"])
    ap.add_argument("--radix", type=int, default=0, help="headline radix (0: the workload's largest)")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-small-blocks", action="store_true",
                    help="skip the secondary entries that time the small-block build (c5, c3)")
    ap.add_argument("--sweep-steps", type=int, default=10)
    ap.add_argument("--replicas", action="store_true",
                    help="N > 1: N independent exchanges, one per GPU, instead of one exchange "
                         "whose ranks are spread over the N GPUs")
    ap.add_argument("--same-device", action="store_true",
                    help="N > 1: every process uses GPU 0 and the gloo backend (a check of the "
                         "sharded orchestration on a one-GPU machine, not a measurement)")
    ap.add_argument("--tokens", type=int, default=0,
                    help="c4 only: tokens per rank (default 8192); smaller values give the "
                         "reduced case used for profiler captures")
    return ap.parse_args()


def make_workload(name, tokens=0):
    from paper_2411_02581_b200 import workloads as W
    if name.startswith("c4"):
        return W.make_c4(skew=name.endswith("skew"), **({"tokens": tokens} if tokens else {}))
    return W.FULL[name]()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and slowdown reasons through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x2: "applications_clocks_setting"}

    def __init__(self, device_index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            uuid = getattr(torch.cuda.get_device_properties(device_index), "uuid", None)
            h = None
            if uuid is not None:
                try:
                    h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
                except Exception:
                    h = None
            if h is None:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES")
                idx = device_index
                if vis:
                    try:
                        idx = int(vis.split(",")[device_index])
                    except Exception:
                        pass
                h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self._h = h
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._h = None

    def _loop(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                    nv.nvmlDeviceGetCurrentClocksThrottleReasons
                bits = get(self._h)
                for b, name in self.REASONS.items():
                    if bits & b:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.01)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml unavailable"]}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(ms, dist=None, device="cpu"):
    """Slowest rank's time: the job is over when the last replica is."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms)
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(payload_bytes_per_rank, world, ms_per_step):
    """Whole-job GB/s: what all replicas moved in a step over the slowest replica's time."""
    return world * payload_bytes_per_rank / (ms_per_step * 1e-3) / 1e9


def kernel_source_sha():
    h = hashlib.sha256()
    with open(os.path.join(ROOT, "paper_2411_02581_b200", "csrc", "tuna_move.cu"), "rb") as f:
        h.update(f.read())
    return h.hexdigest()


# ----------------------------------------------------------------------------- reference arm

def oracle_sample_workload(name, budget_s):
    """A scaled-down instance of the workload that the oracle moves in about budget_s."""
    from paper_2411_02581_b200 import workloads as W
    if name.startswith("c4"):
        rate = 0.8e9  # bytes/s the plain oracle sustains on large blocks, order of magnitude
        tokens = 64
        while tokens < 2048 and (2 * tokens) * 64 * 2 * 8192 <= budget_s * rate:
            tokens *= 2
        wl = W.make_c4(tokens=tokens, skew=name.endswith("skew"))
        return wl, f"{name} shape with {tokens} of 8192 tokens per rank ({wl.payload_bytes_total / 2**30:.2f} GiB)"
    wl = make_workload(name)
    return wl, f"{name} at full size ({wl.payload_bytes_total / 2**20:.1f} MiB)"


def default_radix(wl, radix):
    if radix:
        return radix
    return max(wl.radices) if wl.radices else 0


def configure_host_allocator():
    """Pins down glibc's allocator for the oracle's timing (harness only; the oracle's
    arithmetic is untouched).  The oracle mallocs and frees every message of every
    round.  Left alone, glibc serves requests above a threshold by mmap (fresh,
    page-faulting memory every time) and moves that threshold whenever a large chunk
    is freed, so the same run measured 2.2 GB/s in a fresh process and 5.3 GB/s in one
    that had freed large arrays before.  With the threshold at its maximum and the heap
    never trimmed, messages up to 32 MiB reuse warm heap memory in every process."""
    import ctypes
    try:
        libc = ctypes.CDLL("libc.so.6")
        M_TRIM_THRESHOLD, M_MMAP_THRESHOLD = -1, -3
        ok1 = libc.mallopt(M_MMAP_THRESHOLD, 32 << 20)
        ok2 = libc.mallopt(M_TRIM_THRESHOLD, 1 << 30)
        return bool(ok1 and ok2)
    except Exception:
        return False


def cpu_model():
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    import platform
    return platform.processor() or platform.machine()


def usable_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def host_memory_available():
    import psutil
    avail = psutil.virtual_memory().available
    for limit, used in (("/sys/fs/cgroup/memory.max", "/sys/fs/cgroup/memory.current"),
                        ("/sys/fs/cgroup/memory/memory.limit_in_bytes",
                         "/sys/fs/cgroup/memory/memory.usage_in_bytes")):
        try:
            lim = open(limit).read().strip()
            if lim != "max":
                avail = min(avail, int(lim) - int(open(used).read().strip()))
        except (OSError, ValueError):
            pass
    return avail


def run_oracle_once(wl, radix, send, recv, threads=1):
    """One run of the oracle's schedule (the workload's headline one); seconds."""
    import oracle
    t0 = time.perf_counter()
    if wl.hier and not wl.radices:
        l, g = wl.hier
        rl, rg = wl.hier_radices[-1]
        oracle.tuna_hier(wl, l, g, rl, rg, send, recv)
    elif threads > 1:
        oracle.tuna_flat_mt(wl, radix, send, recv, threads)   # timing variant, checked against the oracle by a test
    else:
        oracle.tuna_flat(wl, radix, send, recv)
    return time.perf_counter() - t0


def run_bruteforce_once(wl, send, recv):
    import oracle
    t0 = time.perf_counter()
    oracle.bruteforce(wl, send, recv)
    return time.perf_counter() - t0


def cpu_baseline_block(wl_name, radix_arg, full_send=None, full_wl=None, runs=7):
    """The oracle, as it stands, on the host cores: the definition of the exchange (the
    CPU's own direct exchange), the headline schedule on one thread and, for flat
    schedules, the same steps with the ranks shared out over all cores; on a bounded
    sample of the workload, and once at full size when the host has the memory."""
    import numpy as np
    pinned = configure_host_allocator()
    cores = usable_cores()
    wls, sample = oracle_sample_workload(wl_name, 8.0)
    hs = wls.make_send().numpy()
    hr = np.empty(max(wls.recv_bytes, 1), dtype=np.uint8)[:wls.recv_bytes]
    r = default_radix(wls, radix_arg)
    pay = wls.payload_bytes_total
    flat = not (wls.hier and not wls.radices)
    first = run_oracle_once(wls, r, hs, hr)                       # first touch of every buffer
    run_oracle_once(wls, r, hs, hr)                               # (one more: the allocator's pools settle)
    one = [run_oracle_once(wls, r, hs, hr) for _ in range(runs)]
    brute = [run_bruteforce_once(wls, hs, hr) for _ in range(runs)]
    block = {"value": pay / statistics.median(one) / 1e9, "unit": UNIT, "cores": 1, "threads": 1,
             "kind": "oracle", "sample": sample + f", median of {runs} runs after two warm-up runs",
             "first_run_GBps": pay / first / 1e9,
             "min_max_GBps": [pay / max(one) / 1e9, pay / min(one) / 1e9],
             "bruteforce_GBps": pay / statistics.median(brute) / 1e9,
             "cpu_model": cpu_model(), "host_cores_available": cores,
             "allocator_pinned": pinned}
    if flat and cores > 1:
        run_oracle_once(wls, r, hs, hr, threads=cores)
        many = [run_oracle_once(wls, r, hs, hr, threads=cores) for _ in range(runs)]
        block["all_cores"] = {"value": pay / statistics.median(many) / 1e9, "unit": UNIT, "threads": min(cores, wls.P),
                              "kind": "threaded timing variant of the oracle's flat schedule "
                                      "(ranks of a round shared out over plain threads)"}
    else:
        block["all_cores"] = None
    del hs, hr
    # once at full size (the oracle's buffers need twice the payload in host memory)
    if full_wl is not None and full_wl.payload_bytes_total > pay:
        need = 2 * full_wl.payload_bytes_total + (4 << 30)
        if host_memory_available() < need:
            block["full_size"] = {"skipped": f"needs {need >> 30} GiB of host memory"}
        else:
            fs = full_send.cpu().numpy() if full_send is not None else full_wl.make_send().numpy()
            fr = np.empty(full_wl.recv_bytes, dtype=np.uint8)
            fpay = full_wl.payload_bytes_total
            rf = default_radix(full_wl, radix_arg)
            tb = run_bruteforce_once(full_wl, fs, fr)
            t1 = run_oracle_once(full_wl, rf, fs, fr)
            full = {"payload_bytes": fpay, "runs": 1, "bruteforce_GBps": fpay / tb / 1e9,
                    "oracle_GBps": fpay / t1 / 1e9, "threads": 1}
            if flat and cores > 1:
                tm = run_oracle_once(full_wl, rf, fs, fr, threads=cores)
                full["oracle_all_cores_GBps"] = fpay / tm / 1e9
            block["full_size"] = full
            del fs, fr
    return block


def reference_arm(args):
    """Times the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import numpy as np
    configure_host_allocator()
    wl, sample = oracle_sample_workload(args.workload, 8.0)
    radix = default_radix(wl, args.radix)
    send = wl.make_send().numpy()
    recv = np.empty(max(wl.recv_bytes, 1), dtype=np.uint8)[:wl.recv_bytes]
    for _ in range(max(1, args.warmup)):
        run_oracle_once(wl, radix, send, recv)
    t = [run_oracle_once(wl, radix, send, recv) for _ in range(args.steps)]
    total = sum(t)
    value = wl.payload_bytes_total * args.steps / total / 1e9
    sched = (f"hierarchical {wl.hier[0]}x{wl.hier[1]} radix {wl.hier_radices[-1][0]}/{wl.hier_radices[-1][1]}"
             if wl.hier and not wl.radices else f"flat radix {radix}")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
        "data": "synthetic",
        "config": {"workload": f"{wl.name} P={wl.P} {sched}", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "threads": 1, "kind": "oracle",
                         "sample": sample, "cpu_model": cpu_model(),
                         "host_cores_available": usable_cores(),
                         "median_GBps": wl.payload_bytes_total / statistics.median(t) / 1e9},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- our arm

def time_schedule(plan, wl, send, recv, steps, warmup, d_counts, direct=False, replan=True):
    """Median-free timing of `steps` back-to-back steps with CUDA events; returns ms per step."""
    import torch
    run = plan.direct_alltoallv if direct else plan.alltoallv

    def step():
        if replan:  # the batch's counts are in device memory, like its payload
            plan.update_counts_device(d_counts)
        run(send, recv)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        step()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / steps


def token_dispatch_entry(wl, args, send, recv, payload):
    """The token dispatch in one pass (gather from token order, exchange, scatter into
    expert order) against the same thing as three passes; `send` and `recv` serve as
    the intermediate buffers of the three-pass route."""
    import numpy as np
    import torch
    from paper_2411_02581_b200 import binding as B, workloads as W
    P, rb = wl.P, wl.elem_size
    tokens = int(wl.sendcounts[0].sum()) // 2
    first, second = W.moe_top2_routing(wl.seed, P, tokens, skew=args.workload == "c4_skew")
    g_np, s_np = W.moe_row_maps(first, second)
    gather, scatter = torch.from_numpy(g_np).cuda(), torch.from_numpy(s_np).cuda()
    rows_in = torch.empty((P * tokens, rb), dtype=torch.uint8, device="cuda")
    rows_in.view(torch.int64).random_()
    rows_out = torch.empty((2 * P * tokens, rb), dtype=torch.uint8, device="cuda")
    plan = B.plan_for(wl, P, explicit_layout=False)

    def timed(fn, steps, warmup=3):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / steps

    d_counts = torch.from_numpy(np.ascontiguousarray(wl.sendcounts, dtype=np.int64)).cuda()

    def fused_step():
        plan.update_counts_device(d_counts)
        plan.set_row_maps(gather, scatter, rows_in.shape[0], rows_out.shape[0])
        plan.rows_alltoallv(rows_in, rows_out)

    ms = timed(fused_step, args.sweep_steps)
    ms_x = timed(lambda: plan.rows_alltoallv(rows_in, rows_out), args.sweep_steps, 1)
    send2, recv2 = send.view(-1, rb), recv.view(-1, rb)

    def three_passes():
        torch.index_select(rows_in, 0, gather, out=send2)
        plan.direct_alltoallv(send, recv)
        rows_out.index_copy_(0, scatter, recv2)

    fused = rows_out.clone()
    ms_3 = timed(three_passes, args.sweep_steps, 1)
    same = bool(torch.equal(fused, rows_out))
    plan.destroy()
    return {"schedule": "token dispatch in one pass: gather + exchange + scatter (rows)",
            "ms_per_step": ms, "payload_GBps": payload / ms / 1e6, "exchange_only_ms": ms_x,
            "rounds": 1, "launches": 1, "moved_over_payload": 1.0,
            "effective_hbm_GBps": 2 * payload / ms_x / 1e6, "frac": 2 * payload / ms_x / 1e6 / measured_peaks()[0],
            "workspace_bytes": 0,
            "three_passes_exchange_only_ms": ms_3, "matches_three_passes": same}


def verify_samples(wl, recv, n=4096):
    """Sampled parity at full size: a received byte must equal the generator's byte
    at the position the exchange's definition says it came from."""
    import numpy as np
    import torch
    from paper_2411_02581_b200 import workloads as W
    if wl.payload_kind != "bytes" or wl.payload_bytes_total == 0:
        return None
    rng = np.random.default_rng(12345)
    C = wl.sendcounts
    nz = np.argwhere(C > 0)
    pick = nz[rng.integers(0, len(nz), size=n)]
    s, d = pick[:, 0], pick[:, 1]
    k = (rng.random(n) * (C[s, d] * wl.elem_size)).astype(np.int64)
    src = (wl.sendbase[s] + wl.sdispls[s, d]) * wl.elem_size + k
    dst = (wl.recvbase[d] + wl.rdispls[d, s]) * wl.elem_size + k
    want = W.payload_byte_at(wl.seed, torch.from_numpy(src))
    got = recv[torch.from_numpy(dst).to(recv.device)].cpu()
    return bool(torch.equal(want, got))


def small_block_entries(dev, peak, peak_kind, steps=20, warmup=3):
    """Exchange-only timing of the schedules whose launches run the small-block build:
    c5 (P = 2048, 179-byte unaligned blocks) in one hop and at radix 2, c3 (16 x 16
    ranks, Zipf-sized blocks) at radix 16/16.  Per entry a roofline of its own: 2 x bytes
    moved by the timed launches over their CUDA-event time (events inside the library,
    around every launch)."""
    import torch
    from paper_2411_02581_b200 import binding as B, workloads as W
    out = []
    sha = kernel_source_sha()
    for name, make, kw, label in (
            ("c5", W.make_c5, dict(radix=2048), "flat radix 2048"),
            ("c5", W.make_c5, dict(radix=2), "flat radix 2"),
            ("c3", W.make_c3, dict(radix=16, l=16, g=16, radix_global=16), "hierarchical l=16 g=16 radix 16/16")):
        wl = make()
        send = wl.make_send(dev)
        recv = wl.make_recv(dev)
        plan = B.plan_for(wl, explicit_layout=False, flags=B.FLAG_NO_DIRECT, **kw)
        plan.alloc_workspace(device=dev)
        for _ in range(warmup):
            plan.alltoallv(send, recv)
        torch.cuda.synchronize()
        ok = verify_samples(wl, recv)
        plan.enable_timing(True)
        plan.get_timing(reset=True)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            plan.alltoallv(send, recv)
        b.record()
        torch.cuda.synchronize()
        t = plan.get_timing(reset=True)
        plan.enable_timing(False)
        ms = t["round_local"]["ms"] + t["round_global"]["ms"]
        ln = t["round_local"]["launches"] + t["round_global"]["launches"]
        by = t["round_local"]["bytes"] + t["round_global"]["bytes"]
        ach = 2.0 * by / (ms * 1e-3) / 1e9 if ms > 0 else 0.0
        n_small, n_all = plan.last_small_launches(), plan.last_launches()
        per_byte = NCU_TRAFFIC_PER_PAYLOAD_BYTE.get(sha, {}).get(f"{name}/{label}")
        out.append({"workload": f"{name} P={wl.P} {label}", "payload_bytes": wl.payload_bytes_total,
                    "exchange_ms": a.elapsed_time(b) / steps, "steps": steps, "parity_samples_ok": ok,
                    "roofline": {"bound": "hbm",
                                 "kernel": "tuna_round_small_kernel" if n_small == n_all else
                                           "tuna_round_kernel" if n_small == 0 else "both builds",
                                 "achieved": ach, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                                 "frac": ach / peak, "frac_of_nominal_8000": ach / 8000.0,
                                 "traffic": per_byte * by / ln if per_byte and ln else None,
                                 "algorithmic_bytes_per_launch": 2.0 * by / ln if ln else 0,
                                 "avg_launch_ms": ms / ln if ln else None, "launches": ln}})
        plan.set_workspace(None)
        plan.destroy()
        del send, recv
        torch.cuda.empty_cache()
    return out


def sharded_arm(args):
    """N > 1: ONE exchange whose P ranks are spread over the N GPUs, P / N per GPU (the
    hierarchical schedule with one group per GPU: local phases in each GPU's memory, the
    inter-group phase as stores into the other GPUs' receive buffers).  The total payload
    is the workload's whatever N is: strong scaling.  A step is, on every GPU, the re-plan
    for the batch's counts (all-gather of the count matrix, count-metadata exchange and
    prefix sums of this GPU's plan) and its share of the exchange between two barriers."""
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2411_02581_b200 import binding as B
    from paper_2411_02581_b200 import build as build_mod
    from paper_2411_02581_b200 import sharded as S

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = 0 if args.same_device else int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if args.same_device:
        dist.init_process_group("gloo")
    else:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build_mod.build()
    dist.barrier()
    B.lib()
    wl = make_workload(args.workload, args.tokens)
    if wl.P % world:
        raise SystemExit(f"{wl.name}: P = {wl.P} ranks do not divide over {world} GPUs")
    l, E = wl.P // world, wl.elem_size
    mine = S.ranks_of_gpu(wl.P, world, rank)
    my_rows = np.ascontiguousarray(wl.sendcounts[mine.start:mine.stop])
    radix = args.radix if args.radix else 0
    ex = S.ShardedExchange(wl.P, E, my_rows, radix=radix, dist=dist)
    # this GPU's part of the workload's send buffer: the regions of its own ranks
    lo = int(wl.sendbase[mine.start]) * E
    full = wl.make_send(dev) if wl.send_bytes <= (24 << 30) else None
    if full is not None:
        send = full[lo:lo + ex.send_bytes].clone()
        del full
    else:
        send = torch.empty(ex.send_bytes, dtype=torch.uint8, device=dev)
        send.view(torch.int64)[:ex.send_bytes // 8].random_()
    torch.cuda.empty_cache()

    d_rows = torch.from_numpy(my_rows).to(dev)   # the batch's counts are in device memory, like its payload

    def step():
        ex.update_counts_device(d_rows)
        ex.exchange(send)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    # sampled parity: bytes this GPU received against the generator at their source position
    rng = np.random.default_rng(777 + rank)
    C = wl.sendcounts
    nz = np.argwhere(C[:, mine.start:mine.stop] > 0)
    ok = None
    if len(nz):
        pick = nz[rng.integers(0, len(nz), 4096)]
        s, d = pick[:, 0], pick[:, 1] + mine.start
        k = (rng.random(len(s)) * (C[s, d] * E)).astype(np.int64)
        src = (wl.sendbase[s] + wl.sdispls[s, d]) * E + k
        dst = (wl.recvbase[d] - wl.recvbase[mine.start] + wl.rdispls[d, s]) * E + k
        from paper_2411_02581_b200 import workloads as W
        want = W.payload_byte_at(wl.seed, torch.from_numpy(src))
        ok = bool(torch.equal(want, ex.recv[torch.from_numpy(dst).to(dev)].cpu())) if wl.send_bytes <= (24 << 30) else None
    ex.plan.enable_timing(True)
    ex.plan.get_timing(reset=True)
    launches0 = ex.plan.launch_count()
    dist.barrier()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        ev0.record()
        for _ in range(args.steps):
            step()
        ev1.record()
        torch.cuda.synchronize()
    dist.barrier()
    ms_per_step = max_over_ranks(ev0.elapsed_time(ev1), dist, dev if not args.same_device else "cpu") / args.steps
    timing = ex.plan.get_timing(reset=True)
    launches = ex.plan.launch_count() - launches0
    payload = wl.payload_bytes_total
    g_ms, g_by = timing["round_global"]["ms"], timing["round_global"]["bytes"]
    l_ms, l_by = timing["round_local"]["ms"], timing["round_local"]["bytes"]
    peak, peak_kind = measured_peaks()
    # the push crosses NVLink: bytes this GPU stores into other GPUs over its device time,
    # against the measured 770 GB/s per direction of a peer copy on this kind of machine
    link_peak = 770.0
    ach_link = g_by / (g_ms * 1e-3) / 1e9 if g_ms > 0 else 0.0
    ach_local = 2.0 * l_by / (l_ms * 1e-3) / 1e9 if l_ms > 0 else 0.0
    flags = torch.tensor([1.0 if ok in (True, None) else 0.0], dtype=torch.float64,
                         device="cpu" if args.same_device else dev)
    dist.all_reduce(flags, op=dist.ReduceOp.MIN)
    if rank == 0:
        line = {
            "metric": METRIC, "value": payload / (ms_per_step * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": f"{wl.name} P={wl.P}, {l} ranks per GPU: local radix {radix or max(2, l)}, "
                                   f"inter-GPU phase pushed into the peers' receive buffers, payload {payload} bytes "
                                   f"in total, elem {E} B, re-plan every step from counts in device memory (all-gathered there)",
                       "l2": "inputs larger than L2" if payload / world > 256e6 else "inputs fit in L2",
                       "sharding": "one group of the hierarchical schedule per GPU",
                       "emulated_on_one_gpu": bool(args.same_device)},
            "gpu_launches": int(launches) * world, "parity_samples_ok": bool(flags.item() == 1.0),
            "clocks": clocks.summary(),
            "roofline": {"bound": "nvlink", "kernel": "tuna_round_kernel (inter-GPU push of rank 0)",
                         "achieved": ach_link, "peak": link_peak, "peak_kind": "of the measured peer-copy rate",
                         "unit": "GB/s", "frac": ach_link / link_peak, "traffic": None,
                         "local_phases_GBps": ach_local, "local_frac_of_hbm": ach_local / peak,
                         "hbm_peak_kind": f"of {peak_kind}"},
            "e2e": None, "cpu_baseline": None,
        }
        print(json.dumps(line), flush=True)
    dist.barrier()
    ex.destroy()
    dist.destroy_process_group()


def ours_arm(args):
    import numpy as np
    import torch
    from paper_2411_02581_b200 import binding as B
    from paper_2411_02581_b200 import build as build_mod

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build_mod.build()
    if dist:
        dist.barrier()
    B.lib()

    wl = make_workload(args.workload, args.tokens)
    radix = default_radix(wl, args.radix)
    hier_headline = not wl.radices and wl.hier
    dev = torch.device("cuda", local)
    send = wl.make_send(dev)
    recv = wl.make_recv(dev)
    payload = wl.payload_bytes_total

    def make_plan(r, l=None, g=1, rg=2, flags=0, block_count=0, direct=False):
        # plans that only run their own schedule are told so: multi-phase plans then keep
        # no direct list, which shortens every re-plan
        if not direct:
            flags |= B.FLAG_NO_DIRECT
        return B.plan_for(wl, r, l=l, g=g, radix_global=rg, flags=flags, explicit_layout=False,
                          block_count=block_count)

    if hier_headline:
        l, g = wl.hier
        rl, rg = wl.hier_radices[-1]
        plan = make_plan(rl, l=l, g=g, rg=rg)
        sched = f"hierarchical l={l} g={g} radix {rl}/{rg}"
    else:
        plan = make_plan(radix)
        sched = f"flat radix {radix}"
    plan.alloc_workspace(host_staging=not args.no_e2e, device=dev)
    # The workloads are packed back to back.  In the device-timed step the batch's
    # count matrix is resident in HBM like its payload (routing decided on the GPU);
    # the end-to-end leg below starts from host arrays instead ("no displacement
    # arrays": only the counts cross to the device, the rest is computed there).
    layout = (wl.sendcounts, None, None, None, None)
    d_counts = torch.from_numpy(np.ascontiguousarray(wl.sendcounts, dtype=np.int64)).to(dev)

    def step():
        plan.update_counts_device(d_counts)
        plan.alltoallv(send, recv)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    ok = verify_samples(wl, recv)
    plan.enable_timing(True)
    plan.get_timing(reset=True)
    launches0 = plan.launch_count()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]  # end of every step
    with ClockSampler(local) as clocks:
        ev0.record()
        for i in range(args.steps):
            step()
            marks[i].record()
        ev1.record()
        torch.cuda.synchronize()
    if dist:
        dist.barrier()
    elapsed_ms = ev0.elapsed_time(ev1)
    per_step = [a.elapsed_time(b) for a, b in zip([ev0] + marks[:-1], marks)]
    step_ms = {"median": statistics.median(per_step), "min": min(per_step), "max": max(per_step),
               "stddev": statistics.pstdev(per_step)} if per_step else None
    launches = plan.launch_count() - launches0
    timing = plan.get_timing(reset=True)
    plan.enable_timing(False)
    elapsed_ms = max_over_ranks(elapsed_ms, dist, dev)
    ms_per_step = elapsed_ms / args.steps
    value = job_throughput(payload, world, ms_per_step)

    # roofline of the dominant kernel: the fused pack-move-unpack kernel, one launch
    # per digit phase
    peak, peak_kind = measured_peaks()
    n_small, n_all = plan.last_small_launches(), plan.last_launches()
    kname = ("tuna_round_small_kernel" if n_small == n_all else "tuna_round_kernel" if n_small == 0
             else f"tuna_round_kernel ({n_all - n_small} launches) + tuna_round_small_kernel ({n_small})")
    rk_ms = timing["round_local"]["ms"] + timing["round_global"]["ms"]
    rk_launches = timing["round_local"]["launches"] + timing["round_global"]["launches"]
    rk_bytes = timing["round_local"]["bytes"] + timing["round_global"]["bytes"]
    achieved = 2.0 * rk_bytes / (rk_ms * 1e-3) / 1e9 if rk_ms > 0 else 0.0
    per_byte = NCU_TRAFFIC_PER_PAYLOAD_BYTE.get(kernel_source_sha(), {}).get(f"{wl.name}/{sched}")
    roofline = {
        "bound": "hbm", "kernel": kname, "achieved": achieved, "peak": peak,
        "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
        "frac_of_nominal_8000": achieved / 8000.0,
        "traffic": (per_byte * rk_bytes / rk_launches) if per_byte and rk_launches else None,
        "algorithmic_bytes_per_launch": 2.0 * rk_bytes / rk_launches if rk_launches else 0,
        "avg_launch_ms": rk_ms / rk_launches if rk_launches else None,
        "launches": rk_launches,
        "ms_per_step": {k: v["ms"] / args.steps for k, v in timing.items()},
    }

    # end to end through the host-buffer entry point (pinned host memory)
    e2e = None
    if not args.no_e2e:
        hs = torch.empty(max(wl.send_bytes, 1), dtype=torch.uint8, pin_memory=True)[:wl.send_bytes]
        hr = torch.empty(max(wl.recv_bytes, 1), dtype=torch.uint8, pin_memory=True)[:wl.recv_bytes]
        hs.copy_(send)
        e_steps = max(2, min(args.steps, 5))

        def estep():
            plan.update_counts(*layout)
            plan.alltoallv_host(hs, hr, B.SCHEDULE_TUNA)
            torch.cuda.synchronize()

        estep()
        if dist:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(e_steps):
            estep()
        e_ms = (time.perf_counter() - t0) * 1e3 / e_steps
        e_ms = max_over_ranks(e_ms, dist, dev)
        # the same with the buffers staged through device copies, for comparison
        def sstep():
            plan.update_counts(*layout)
            plan.alltoallv_host(hs, hr, B.SCHEDULE_TUNA | B.HOST_STAGED)
            torch.cuda.synchronize()

        sstep()
        t0 = time.perf_counter()
        for _ in range(2):
            sstep()
        staged_ms = (time.perf_counter() - t0) * 1e3 / 2
        e2e = {"value": job_throughput(payload, world, e_ms), "unit": UNIT,
               "path": "in place on the pinned host buffers for blocks of 2 KiB and more on average, "
                       "staged through device copies below that",
               "staged_copies_ms_per_step": staged_ms,
               "h2d_bytes_per_step": wl.send_bytes + 8 * (wl.P * wl.P + 2 * wl.P),
               "d2h_bytes_per_step": wl.recv_bytes, "ms_per_step": e_ms, "steps": e_steps}
        del hs, hr

    # the re-plan alone (count-metadata exchange + prefix sums), wall clock: from the
    # device-resident counts and from a host array
    replan = None
    if not args.no_sweep:
        def wall(fn, n):
            fn()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(n):
                fn()
            torch.cuda.synchronize()
            return (time.perf_counter() - t0) * 1e3 / n

        replan = {"from_device_counts_ms": wall(lambda: plan.update_counts_device(d_counts), 5),
                  "from_host_counts_ms": wall(lambda: plan.update_counts(*layout), 5)}

    # the other schedules of the workload, timed the same way (exchange + re-plan)
    sweep = []
    if not args.no_sweep and rank == 0:
        def entry(name, p, direct=False):
            p.alloc_workspace(device=dev)
            ms = time_schedule(p, wl, send, recv, args.sweep_steps, 3, d_counts, direct=direct)
            ms_x = time_schedule(p, wl, send, recv, args.sweep_steps, 1, d_counts, direct=direct, replan=False)
            # bytes every launch of the exchange moves: each hop of each block, the self
            # blocks (rotation launch) and, in classic mode, every block once more
            if direct:
                moved = payload
            else:
                moved = sum(r["bytes"] for r in p.rounds()) + p.phase_info(-1)["bytes"]
            sweep.append({"schedule": name, "ms_per_step": ms, "payload_GBps": payload / ms / 1e6,
                          "exchange_only_ms": ms_x, "rounds": 1 if direct else p.num_rounds(),
                          "launches": p.last_launches(),
                          "moved_over_payload": moved / max(payload, 1),
                          "effective_hbm_GBps": 2 * moved / ms_x / 1e6,
                          "frac": 2 * moved / ms_x / 1e6 / peak,
                          "small_build_launches": p.last_small_launches(),
                          "workspace_bytes": 0 if direct else p.workspace_bytes()})
            p.set_workspace(None)
            p.destroy()
            torch.cuda.empty_cache()

        plan.set_workspace(None)
        torch.cuda.empty_cache()
        entry("direct", make_plan(wl.P, direct=True), direct=True)
        for r in wl.radices:
            entry(f"flat r={r}", make_plan(r))
        if wl.radices:
            entry(f"flat r={wl.radices[0]} classic-rotate", make_plan(wl.radices[0], flags=B.FLAG_CLASSIC_ROTATE))
            entry(f"flat r={wl.radices[-1]} bulk-copy route", make_plan(wl.radices[-1], flags=B.FLAG_BULK_COPY))
        if wl.hier:
            l, g = wl.hier
            for rl, rg in wl.hier_radices:
                entry(f"hier {l}x{g} r={rl}/{rg}", make_plan(rl, l=l, g=g, rg=rg))
            # staggered inter-group exchange: one block per step, block_count steps per launch
            rl = max(a for a, _ in wl.hier_radices)
            for bc in (1, l, wl.P):
                entry(f"hier {l}x{g} r={rl} staggered block_count={bc}",
                      make_plan(rl, l=l, g=g, block_count=bc))

        # Two plans taking turns: while one plan's exchange runs on the first stream,
        # the other plan re-plans the next batch on a second stream, so the count-metadata
        # exchange and the prefix sums of batch k + 1 overlap the data movement of batch k.
        if not hier_headline:
            pair = [make_plan(radix), make_plan(radix)]
            for p in pair:
                p.alloc_workspace(device=dev)
            s_x, s_p = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev, priority=-1)  # the small plan kernels go first

            done = [torch.cuda.Event(), torch.cuda.Event()]  # end of each plan's last exchange

            def turns(n):
                for i in range(n):
                    p = pair[i % 2]
                    done[i % 2].synchronize()                     # its tables are in use until then
                    p.update_counts_device(d_counts, stream=s_p)  # returns when this plan's tables are ready
                    p.alltoallv(send, recv, stream=s_x)           # enqueued behind the previous exchange
                    done[i % 2].record(s_x)

            torch.cuda.synchronize()
            turns(4)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            turns(args.sweep_steps * 2)
            torch.cuda.synchronize()
            ms = (time.perf_counter() - t0) * 1e3 / (args.sweep_steps * 2)
            sweep.append({"schedule": f"flat r={radix}, two plans taking turns (re-plan of the next batch "
                                      "beside the exchange; wall clock)",
                          "ms_per_step": ms, "payload_GBps": payload / ms / 1e6,
                          "frac": None,
                          "launches": pair[0].last_launches()})
            for p in pair:
                p.set_workspace(None)
                p.destroy()
            torch.cuda.empty_cache()

        if args.workload in ("c4", "c4_skew"):
            sweep.append(token_dispatch_entry(wl, args, send, recv, payload))

    # the small-block build of the mover under the same clock: the all-unaligned single
    # hop and the radix-2 schedule on c5-sized blocks, and the short launches of c3
    small = None
    if rank == 0 and not args.no_small_blocks and args.workload == "c4":
        small = small_block_entries(dev, peak, peak_kind)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle  # noqa: F401  (the CPU-baseline leg is the one place bench.py runs the oracle)
        full = None if args.tokens else wl
        cpu = cpu_baseline_block(args.workload, args.radix, full_send=send if full is not None else None,
                                 full_wl=full)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": f"{wl.name} P={wl.P} {sched}, payload {payload} bytes, "
                                   f"elem {wl.elem_size} B, re-plan every step from counts in device memory",
                       "l2": "inputs larger than L2" if payload > 256e6 else
                             "inputs fit in L2 (latency-bound case)",
                       "replicas": "one independent exchange per GPU" if world > 1 else "single GPU"},
            "gpu_launches": int(launches), "parity_samples_ok": ok,
            "clocks": clocks.summary(), "e2e": e2e, "roofline": roofline,
            "cpu_baseline": cpu, "small_blocks": small, "step_ms": step_ms, "replan_ms": replan, "sweep": sweep,
        }
        print(json.dumps(line), flush=True)
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        reference_arm(args)
    elif int(os.environ.get("WORLD_SIZE", "1")) > 1 and not args.replicas:
        sharded_arm(args)
    else:
        ours_arm(args)


if __name__ == "__main__":
    main()
