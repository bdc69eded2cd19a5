#!/usr/bin/env python
"""Benchmark of libpdattn: one step = one paged-decode-attention call (split-KV kernel + combine
kernel) over one rollout batch, through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--cfg 2]

Workload: the benchmark's second configuration, the 7B-shaped rollout step (256 sequences, 28 q heads / 4 KV
heads, head_dim 128, page size 16, context = 512-token prompt + lognormal response), synthetic and
seeded.  With N > 1 (torchrun, one rank per GPU) every rank runs its own batch of that shape
(sequences are independent: no collective on the data path) and the value is the sum over ranks
divided by the slowest rank's time: weak scaling.

Prints ONE JSON line.  `value` is seq-steps/s with everything resident in HBM; `e2e` is the same
metric through pdattn_decode_host with the step's q / block_table / context_lens in pinned host
memory and `out` read back every step; `roofline` is the split-KV kernel's algorithmic KV bytes
over its own CUDA-event duration against the measured HBM copy bandwidth; `cpu_baseline` is the
fp64 oracle timed on this machine's host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

METRIC = "paged decode attn: seq-steps/s (achieved HBM TB/s in roofline) at N GPUs"
UNIT = "seq-steps/s"
CFG_DESC = {
    1: "configs[0] tiny: 4 seqs, 4/1 heads, d64",
    2: "configs[1] 7B-shaped rollout step: 256 seqs, 28 q / 4 kv heads, d128, page 16, "
       "ctx = 512 + lognormal(median 2048, sigma 0.8) capped 8192, seed 1",
    3: "configs[2] GRPO group sharing: 64x8 seqs, 40/8 heads, d128, shared 1024-token prompt pages",
    4: "configs[3] 32B-shaped long context: 128 seqs, 64/8 heads, d128",
    5: "configs[4] long-tail straggler phase: 8 seqs, 28/4 heads, d128, ctx U[32768,65536]",
}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cfg", type=int, default=2, help="benchmark configuration, 1-based (default 2: the one the metric is quoted on)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fp8", action="store_true",
                    help="time pdattn_decode_fp8 over an e4m3 copy of the same pools (half the KV bytes per step) "
                         "instead of the bf16 step; head_dim 128 configurations only")
    ap.add_argument("--short-batches", nargs="?", const="all", default=None, metavar="NAME",
                    help="also time batches of 4096 short contexts under every merge mode and with the short-piece "
                         "kernel off, and a large GRPO batch early in its rollout under both prefix kernels "
                         "(secondary results, N = 1); with NAME (4096x64, 4096x128, 4096xU[50,400], 4096x512, grpo) "
                         "only that batch, e.g. for a profiler capture of one small case")
    ap.add_argument("--grouped", action="store_true",
                    help="config 3 only: time pdattn_decode_grouped (shared prompt pages read once per group)")
    ap.add_argument("--no-all-configs", action="store_true",
                    help="skip secondary.configs (the other four workloads; taken by the default run at N = 1)")
    ap.add_argument("--num-seqs", type=int, default=None,
                    help="shrink the batch (profiling captures only; not the metric's workload)")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, STREAM-style copy)"
    except Exception:
        return 6650.0, "fallback (earlier measurement on this pool)"


def profiled_traffic(cfg):
    """DRAM bytes per decode_kernel launch from the committed ncu summary, with where it comes from.  The summary
    records the fingerprint of the kernel sources it was captured on; when the sources have changed since, the
    figure is withheld (None) rather than passed off as a measurement of the current kernel."""
    from paper_2607_09207_b200 import build as pd_build
    p = os.path.join(ROOT, "profiles", f"decode_kernel_cfg{cfg}_ncu.md")
    try:
        text = open(p).read()
        m = re.search(r"traffic_bytes_per_launch:\s*([0-9.eE+]+)", text)
        f = re.search(r"kernel_source_sha256:\s*([0-9a-f]{64})", text)
        if not m:
            return None, f"no traffic figure in profiles/{os.path.basename(p)}"
        now = pd_build.source_fingerprint()
        if not f or f.group(1) != now:
            return None, (f"withheld: profiles/{os.path.basename(p)} was captured on kernel sources "
                          f"{f.group(1)[:12] if f else 'unknown'}, this build is {now[:12]}")
        return float(m.group(1)), (f"ncu dram__bytes_read.sum + dram__bytes_write.sum, profiles/{os.path.basename(p)}, "
                                   f"kernel sources {now[:12]} (same as this build)")
    except Exception as e:
        return None, f"unavailable: {e}"


class ClockSampler:
    """Polls NVML for SM clock and throttle reasons while the timed regions run."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._stop.clear()
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        if self._thr is not None:
            self._stop.set()
            self._thr.join()
            self._thr = None

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_pass(wc, n_seqs):
    """Time the oracle, as it stands, on the first n_seqs sequences of the host copy of the workload."""
    from oracle import pdattn_oracle as orc
    cores = orc.host_cores()
    sl = slice(0, n_seqs)
    t0 = time.perf_counter()
    orc.decode(wc.q[sl], wc.k_cache, wc.v_cache, wc.block_table[sl], wc.context_lens[sl], wc.scale,
               num_threads=cores)
    return time.perf_counter() - t0, cores


def run_reference(args):
    """The reference arm is the fp64 CPU oracle (there is no reference implementation of this path):
    each step is one oracle pass over a bounded sample of the workload, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2607_09207_b200 import workloads as W
    w = W.make_config(args.cfg, device="cpu", poison=True)
    S = w.num_seqs
    t_probe, cores = oracle_pass(w, min(S, 8))
    per_seq = t_probe / min(S, 8)
    budget = 150.0 / max(1, args.steps + args.warmup)          # whole run within a few minutes
    n = int(max(1, min(S, min(budget, 3.0) / max(per_seq, 1e-9))))
    for _ in range(args.warmup):
        oracle_pass(w, n)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_pass(w, n)
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    sample = f"first {n} of {S} sequences of the workload per step, {args.steps} steps"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": CFG_DESC[args.cfg], "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def batch_stats(step, stream, n_batches=10, calls=20, warm=5):
    """Procedure of the metric: `warm` untimed calls, then n_batches batches of `calls` back-to-back calls with
    one CUDA-event pair per batch (time / calls includes launch gaps and the hand-off between the step's kernels
    as an engine would see them); median and best batch."""
    i = 0
    for _ in range(warm):
        step(i)
        i += 1
    torch.cuda.synchronize()
    ms = []
    for _ in range(n_batches):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(calls):
            step(i)
            i += 1
        b.record(stream)
        torch.cuda.synchronize()
        ms.append(a.elapsed_time(b) / calls)
    return {"batches": n_batches, "calls_per_batch": calls, "median_ms": float(np.median(ms)), "best_ms": float(min(ms))}


def kernel_events_ms(pdattn, step, stream, n=40):
    """Mean duration of the split-KV kernel alone: CUDA events the library records around it on its stream."""
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    for a, b in evs:                      # force creation of the underlying CUDA events
        a.record(stream)
        b.record(stream)
    torch.cuda.synchronize()
    L = pdattn.lib()
    for i, (a, b) in enumerate(evs):
        L.pdattn_profile_events(a.cuda_event, b.cuda_event)
        step(i)
    L.pdattn_profile_events(None, None)
    torch.cuda.synchronize()
    return float(np.mean([a.elapsed_time(b) for a, b in evs]))


def oracle_full(wc, threads):
    """One oracle pass over every sequence of the host copy of a workload with `threads` threads: seconds."""
    from oracle import pdattn_oracle as orc
    t0 = time.perf_counter()
    orc.decode(wc.q, wc.k_cache, wc.v_cache, wc.block_table, wc.context_lens, wc.scale, num_threads=threads)
    return time.perf_counter() - t0


def other_configs(pdattn, W, dev, stream, local, peak, with_oracle):
    """The metric's other workloads (configurations 1, 3, 3 through the grouped entry point, 4 and 5), each at full
    size: step time as median and best of 10 batches of 20 calls, the split-KV kernel's own time, unique KV bytes,
    TB/s and fraction of the measured copy bandwidth, the SM clock and throttle reasons seen during that region,
    and the oracle timed once on the host cores.  Configuration 1 (96 KB, cache resident) reports latency only."""
    from oracle import pdattn_oracle as orc
    res = {}
    for cfg in (1, 3, 4, 5):
        w = W.make_config(cfg, device=dev)
        S = w.num_seqs
        uniq = w.unique_kv_bytes()
        copies = [w]
        if cfg != 1 and uniq < (24 << 30):
            copies.append(_physical_copy(w, seed=177 + cfg))
        outs = [torch.empty_like(c.q) for c in copies]
        ws = pdattn.alloc_grouped_workspace(S, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size, device=dev)
        variants = [("", False)] + ([("_grouped", True)] if cfg == 3 else [])
        for suffix, grouped in variants:
            if grouped:
                pth = np.full(S // 8, 1024 // 64, dtype=np.int32)
                ptd = torch.from_numpy(pth).to(dev)

            def step(i):
                c, o = copies[i % len(copies)], outs[i % len(copies)]
                if grouped:
                    pdattn.decode_grouped(c.q, c.k_cache, c.v_cache, c.block_table, c.context_lens, c.scale, o, ws,
                                          c.context_lens_host, 8, ptd, pth, stream=stream)
                else:
                    pdattn.decode_ex(c.q, c.k_cache, c.v_cache, c.block_table, c.context_lens, c.scale, o, ws,
                                     context_lens_host=c.context_lens_host, stream=stream)

            sampler = ClockSampler(local)
            sampler.start()
            bt = batch_stats(step, stream)
            k_ms = None if grouped else kernel_events_ms(pdattn, step, stream)
            sampler.stop()
            assert pdattn.check(ws) == pdattn.OK
            row = {"workload": CFG_DESC[cfg] + (" [grouped entry point: shared prompt tiles read once per group]"
                                                if grouped else ""),
                   "num_seqs": S, "step_ms": bt, "clocks": sampler.summary()}
            if cfg == 1:
                row["latency_us"] = {"median": bt["median_ms"] * 1e3, "best": bt["best_ms"] * 1e3}
                row["note"] = "96 KB of KV, cache resident: latency only"
            else:
                ms = bt["median_ms"]
                row.update({"seq_steps_per_s": S / (ms * 1e-3), "unique_kv_bytes": uniq,
                            "logical_kv_bytes": w.logical_kv_bytes(),
                            "hbm_tbs_step": uniq / (ms * 1e-3) / 1e12, "frac_of_measured_peak_step": uniq / (ms * 1e-3) / 1e9 / peak,
                            "pct_of_8tbs_nominal_step": uniq / (ms * 1e-3) / 8e12 * 100.0,
                            "l2": f"steps rotate over {len(copies)} physically distinct copies of pools/tables"})
                if k_ms is not None:
                    row.update({"kernel_ms": k_ms, "kernel_tbs": uniq / (k_ms * 1e-3) / 1e12,
                                "kernel_frac_of_measured_peak": uniq / (k_ms * 1e-3) / 1e9 / peak})
            res[f"cfg{cfg}{suffix}"] = row
        if with_oracle:
            del copies[1:], outs[1:]
            wc = w.to("cpu")
            cores = orc.host_cores()
            t_all = oracle_full(wc, cores)
            res[f"cfg{cfg}"]["oracle"] = {"seq_steps_per_s": S / t_all, "seconds_per_pass": t_all, "cores": cores,
                                          "sample": f"one pass over all {S} sequences"}
            if cfg == 1:
                t_one = oracle_full(wc, 1)
                res["cfg1"]["oracle_single_thread"] = {"seq_steps_per_s": S / t_one, "seconds_per_pass": t_one, "cores": 1,
                                                       "sample": f"one pass over all {S} sequences"}
            del wc
        del w, copies, outs, ws
        torch.cuda.empty_cache()
    return res


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
        return

    from paper_2607_09207_b200 import pdattn
    from paper_2607_09207_b200 import workloads as W
    pdattn.lib()   # fail loudly if the CUDA library is missing

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    local = local % torch.cuda.device_count()     # ranks may share a GPU in a functional test of this script
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        backend = os.environ.get("PDATTN_BENCH_BACKEND", "nccl")   # "gloo" when ranks share one GPU
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=dev)
        else:
            dist.init_process_group(backend)

    K, Wm = args.steps, max(3, args.warmup)
    # ---- inputs: this rank's batch, in two physically distinct copies (pools, tables, q) so that
    # consecutive steps never find the previous step's pages in L2
    base = W.make_config(args.cfg, device=dev, num_seqs=args.num_seqs)
    if world > 1:
        # every rank gets its own lengths and values: same shape, different seed stream
        lens = W.config_lengths(args.cfg)
        rng = np.random.default_rng(1000 + rank)
        base = W.make_config(args.cfg, device=dev) if rank == 0 else _reseeded(W, args.cfg, rank, dev, lens, rng)
    copies = [base]
    if base.unique_kv_bytes() < (40 << 30):
        copies.append(_physical_copy(base, seed=77 + rank))
    S = base.num_seqs
    uniq = base.unique_kv_bytes()
    logical = base.logical_kv_bytes()
    ws = pdattn.alloc_grouped_workspace(S, base.num_q_heads, base.num_kv_heads, base.head_dim, base.block_size,
                                        device=dev)
    grouped = args.grouped and args.cfg == 3
    if grouped:
        pth = np.full(S // 8, 1024 // 64, dtype=np.int32)       # 64 shared prompt pages = 16 tiles per group
        ptd = torch.from_numpy(pth).to(dev)
    outs = [torch.empty_like(c.q) for c in copies]
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(local)
    fp8 = None
    if args.fp8:
        ks8 = torch.full((base.num_kv_heads,), 1.25, dtype=torch.float32, device=dev)
        vs8 = torch.full((base.num_kv_heads,), 0.75, dtype=torch.float32, device=dev)
        fp8 = [W.fp8_caches(c, ks8, vs8) for c in copies]
        uniq //= 2
        logical //= 2

    def step(i):
        c = copies[i % len(copies)]
        if fp8 is not None:
            k8, v8 = fp8[i % len(copies)]
            pdattn.decode_fp8(c.q, k8, v8, ks8, vs8, c.block_table, c.context_lens, c.scale, outs[i % len(copies)], ws,
                              context_lens_host=c.context_lens_host, stream=stream)
            return
        if grouped:
            pdattn.decode_grouped(c.q, c.k_cache, c.v_cache, c.block_table, c.context_lens, c.scale,
                                  outs[i % len(copies)], ws, c.context_lens_host, 8, ptd, pth, stream=stream)
            return
        pdattn.decode_ex(c.q, c.k_cache, c.v_cache, c.block_table, c.context_lens, c.scale, outs[i % len(copies)],
                         ws, context_lens_host=c.context_lens_host, stream=stream)

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- region A: headline
    for i in range(Wm):
        step(i)
    launches_per_step = pdattn.last_launch_count()
    assert pdattn.check(ws) == pdattn.OK
    sync_all()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(K):
        step(i)
    e1.record(stream)
    sync_all()
    ms_total = e0.elapsed_time(e1)
    if dist is not None:
        t = torch.tensor([ms_total], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_step = ms_total / K
    value = world * S / (ms_step * 1e-3)
    # the same step as 10 batches of 20 calls, one event pair per batch: median and best batch (this rank)
    batch_timing = batch_stats(step, stream)

    # ---- region B: the split-KV kernel's own duration, CUDA events recorded around it by the library
    k_iso_ms = kernel_events_ms(pdattn, step, stream, n=min(K, 200))
    k1_ms, kernel_name = k_iso_ms, "decode_kernel"
    kernel_note = ("CUDA events recorded by the library right around the kernel (that launch is then not a programmatic "
                   "dependent of its predecessor)")
    if launches_per_step == 1:
        # The step is this one kernel (it merges its cut units itself): over the timed region its K launches took
        # K * ms_per_step, set-up overlapped with the previous launch's drain as in any steady decode loop.  The
        # isolated figure is kept beside it.
        k1_ms = ms_step
        kernel_note = ("one launch per step: the kernel's average duration over the timed region is the step's "
                       "(event pair around all K launches); kernel_ms_isolated times single launches between events")
    if grouped:      # the prefix kernel does part of the reading: account the whole step
        k1_ms, kernel_name = ms_step, "prefix_kernel + decode_kernel + combine_kernel (whole step)"
    peak, peak_src = measured_peak()
    achieved = uniq / (k1_ms * 1e-3) / 1e9
    traffic, traffic_src = (None, "not captured for the fp8 step") if fp8 is not None else profiled_traffic(args.cfg)

    # ---- region C: end to end from pinned host buffers through pdattn_decode_host
    c0 = copies[0]
    qh, bth, lh = c0.q.cpu().pin_memory(), c0.block_table.cpu().pin_memory(), c0.context_lens.cpu().pin_memory()
    oh = torch.empty_like(qh).pin_memory()
    staging = torch.empty(pdattn.host_staging_size(S, c0.num_q_heads, c0.head_dim, c0.max_blocks_per_seq),
                          dtype=torch.uint8, device=dev)
    ke = min(K, 500)

    oh_bits = oh.view(torch.int16).numpy()        # the host buffer itself, for the per-step read

    host_step = pdattn.HostStep(qh, bth, lh, oh, c0.k_cache, c0.v_cache, c0.scale, staging, ws, stream=stream)

    def e2e_step():
        host_step()                       # pdattn_decode_host on the same pinned buffers every step
        stream.synchronize()              # the caller reads `out` on the host every step
        return int(oh_bits[0, 0, 0])

    for _ in range(5):
        e2e_step()
    sync_all()
    t0 = time.perf_counter()
    for _ in range(ke):
        e2e_step()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if dist is not None:
        t = torch.tensor([e2e_s], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    sampler.stop()
    e2e_value = world * S * ke / e2e_s
    # bytes that cross the bus per step: q rows, the lengths, and the used part of every block_table row (fetched in
    # 16-byte units by the library's gather kernel when the table is pinned and mapped, as here)
    used_pages = (c0.context_lens_host.astype(np.int64) + c0.block_size - 1) // c0.block_size
    h2d = qh.numel() * 2 + int((((used_pages * 4) + 15) // 16 * 16).sum()) + lh.numel() * 4
    d2h = oh.numel() * 2
    assert pdattn.check(ws) == pdattn.OK

    # ---- secondary runs (N = 1 only): bandwidth ceilings from the library's probes, the device-side
    # planner (no host copy of the lengths) and the token-major cache layout through strides
    extras = None
    if world == 1 and fp8 is not None:
        extras = {"note": "fp8 run: e2e and the secondary results are not taken (they describe the bf16 step)"}
    elif world == 1:
        def timed(fn, n=20, reps=5):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            best = []
            for _ in range(reps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for _ in range(n):
                    fn()
                b.record(stream)
                torch.cuda.synchronize()
                best.append(a.elapsed_time(b) / n)
            return float(np.median(best))

        c = copies[0]
        sink = torch.zeros(4, dtype=torch.int32, device=dev)
        pool_bytes = 2 * c.k_cache.numel() * 2
        t_stream = timed(lambda: (pdattn.stream_read_probe(c.k_cache, sink), pdattn.stream_read_probe(c.v_cache, sink)))
        t_gather = timed(lambda: pdattn.decode_ex(c.q, c.k_cache, c.v_cache, c.block_table, c.context_lens, c.scale,
                                                  outs[0], ws, context_lens_host=c.context_lens_host, probe=True))
        t_devplan = timed(lambda: pdattn.decode_ex(c.q, c.k_cache, c.v_cache, c.block_table, c.context_lens, c.scale,
                                                   outs[0], ws, context_lens_host=None))
        extras = {"stream_read_gbs": pool_bytes / (t_stream * 1e-3) / 1e9,
                  "page_gather_gbs": uniq / (t_gather * 1e-3) / 1e9,
                  "device_plan_ms_per_step": t_devplan}
        if uniq < (20 << 30):
            k_nhd = c.k_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
            v_nhd = c.v_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
            extras["token_major_layout_ms_per_step"] = timed(
                lambda: pdattn.decode_ex(c.q, k_nhd, v_nhd, c.block_table, c.context_lens, c.scale, outs[0], ws,
                                         context_lens_host=c.context_lens_host))
            del k_nhd, v_nhd
        assert pdattn.check(ws) == pdattn.OK
        if args.cfg == 2 and args.num_seqs is None:
            extras["decode_loop"] = decode_loop(pdattn, W, dev, stream)
            # two query tokens per sequence (a verification step of the engine): 14 rows share each KV head's tiles
            q2 = W.normal_bf16(S * 2 * c.num_q_heads * c.head_dim, 77, 7, device=dev).view(S, 2, c.num_q_heads, c.head_dim)
            o2 = torch.empty_like(q2)
            mws = pdattn.alloc_multi_workspace(S, c.num_q_heads, c.num_kv_heads, c.head_dim, c.block_size, 2, device=dev)
            t_multi = timed(lambda: pdattn.decode_multi(q2, c.k_cache, c.v_cache, c.block_table, c.context_lens, c.scale,
                                                        o2, mws, context_lens_host=c.context_lens_host))
            assert pdattn.check(mws) == pdattn.OK
            extras["two_query_tokens_ms_per_step"] = t_multi
            del q2, o2, mws
            # the same batch over an fp8 (e4m3, per-head scales) cache: half the bytes per history token
            ks8 = torch.full((c.num_kv_heads,), 1.25, dtype=torch.float32, device=dev)
            vs8 = torch.full((c.num_kv_heads,), 0.75, dtype=torch.float32, device=dev)
            k8, v8 = W.fp8_caches(c, ks8, vs8)
            t_fp8 = timed(lambda: pdattn.decode_fp8(c.q, k8, v8, ks8, vs8, c.block_table, c.context_lens, c.scale,
                                                    outs[0], ws, context_lens_host=c.context_lens_host))
            assert pdattn.check(ws) == pdattn.OK
            extras["fp8_kv_cache"] = {"ms_per_step": t_fp8, "seq_steps_per_s": S / (t_fp8 * 1e-3),
                                      "kv_bytes_per_step": uniq // 2, "kv_gbs": uniq / 2 / (t_fp8 * 1e-3) / 1e9}
            del k8, v8
        if args.cfg == 3 and args.num_seqs is None:
            # GRPO groups of 8 share their 1024-token prompt pages: read them once per group
            gws = pdattn.alloc_grouped_workspace(S, c.num_q_heads, c.num_kv_heads, c.head_dim, device=dev)
            pth = np.full(S // 8, 1024 // 64, dtype=np.int32)
            ptd = torch.from_numpy(pth).to(dev)
            t_grouped = timed(lambda: pdattn.decode_grouped(c.q, c.k_cache, c.v_cache, c.block_table, c.context_lens,
                                                            c.scale, outs[0], gws, c.context_lens_host, 8, ptd, pth),
                              n=10)
            assert pdattn.check(gws) == pdattn.OK
            extras["grouped_shared_prefix"] = {"ms_per_step": t_grouped, "seq_steps_per_s": S / (t_grouped * 1e-3),
                                               "unique_kv_gbs": uniq / (t_grouped * 1e-3) / 1e9}

        if args.short_batches:
            extras["short_context_batches"] = short_batches(pdattn, W, dev, timed, args.short_batches)
        if args.cfg == 2 and args.num_seqs is None and not args.no_all_configs:
            extras["config2_other_seeds"] = other_seeds(pdattn, W, dev, timed, peak)
        if args.cfg == 2 and args.num_seqs is None and not args.no_all_configs:
            extras["configs"] = other_configs(pdattn, W, dev, stream, local, peak, with_oracle=not args.no_cpu_baseline)

    # ---- CPU baseline: the oracle on the host cores (rank 0, N = 1 only)
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        wc = base.to("cpu")
        t_probe, cores = oracle_pass(wc, min(S, 8))
        n = int(max(1, min(S, 20.0 / max(t_probe / min(S, 8), 1e-9))))
        dt, cores = oracle_pass(wc, n)
        passes = 1
        while dt < 12.0 and passes < 64:            # about 10-20 s of CPU work in all
            dt += oracle_pass(wc, n)[0]
            passes += 1
        cpu_baseline = {"value": n * passes / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"{passes} oracle passes over the first {n} of {S} sequences ({dt:.2f} s in all)"}
        if args.cfg <= 2:
            # single-threaded as well, on a sample sized for about 5 s
            n1 = int(max(1, min(S, 5.0 / max(t_probe / min(S, 8) * cores, 1e-9))))
            from oracle import pdattn_oracle as orc
            t0 = time.perf_counter()
            orc.decode(wc.q[:n1], wc.k_cache, wc.v_cache, wc.block_table[:n1], wc.context_lens[:n1], wc.scale, num_threads=1)
            t1 = time.perf_counter() - t0
            cpu_baseline["single_thread"] = {"value": n1 / t1, "unit": UNIT, "cores": 1,
                                             "sample": f"one oracle pass over the first {n1} of {S} sequences ({t1:.2f} s)"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms_step, "step_ms_batches": batch_timing,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if fp8 is None else "e4m3 cache, fp16 products, fp32 accumulate", "data": "synthetic",
            "config": {"workload": CFG_DESC[args.cfg] + (f" [REDUCED to {S} seqs]" if args.num_seqs else "")
                       + (" [grouped: shared prompt tiles read once per group]" if grouped else "")
                       + (" [fp8 KV cache: e4m3 codes, one scale per KV head]" if fp8 is not None else ""),
                       "num_seqs_per_gpu": S,
                       "unique_kv_bytes_per_step": uniq, "logical_kv_bytes_per_step": logical,
                       "l2": f"inputs ({uniq / 1e9:.2f} GB) larger than L2 and steps rotate over {len(copies)} "
                             "physically distinct copies of pools/tables",
                       "parallelism": f"dp{world} (independent batches, no collective)"},
            "hbm_tbs_step": uniq / (ms_step * 1e-3) / 1e12 * 1.0,
            # coefficient of the paper's decode-history term for ONE layer of this shape: seconds per
            # history token read = per-layer KV bytes per token / achieved bytes per second
            "beta_hist_s_per_token_per_layer": base.kv_bytes_per_token() / (2 if fp8 is not None else 1)
                                               / (uniq / (ms_step * 1e-3)),
            "pct_of_8tbs_nominal_step": uniq / (ms_step * 1e-3) / 8e12 * 100.0,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "traffic": traffic, "traffic_source": traffic_src,
                         "kernel": kernel_name, "kernel_ms": k1_ms, "kernel_ms_isolated": k_iso_ms,
                         "kernel_timing": kernel_note, "peak_source": peak_src,
                         "algorithmic_bytes_per_launch": uniq,
                         "pct_of_8tbs_nominal": achieved / 8000.0 * 100.0},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": ke, "note": ("bf16 step (pdattn_decode_host has no fp8 form); " if fp8 is not None else "")
                                         + "q/block_table/context_lens in pinned host memory, out in pinned host memory "
                                         "and the stream synchronised every step: the lengths and the used part of each "
                                         "block_table row are fetched by a gather kernel (bulk copies over the bus), q rows "
                                         "are fetched and out rows written over the bus by the decode kernels themselves; "
                                         "KV pools are resident state"},
            "gpu_launches": launches_per_step * K,
            "clocks": sampler.summary(),
            "cpu_baseline": cpu_baseline,
            "secondary": extras,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def other_seeds(pdattn, W, dev, timed, peak):
    """The headline configuration's length recipe (256 sequences, 512 + lognormal(median 2048, sigma 0.8) capped
    at 8192) under six other seeds: the step must not depend on the one batch the metric is quoted on.  Two
    physical copies per seed, rotated (each larger than L2)."""
    rows = []
    for seed in range(11, 17):
        lens = 512 + W.lognormal_lengths(W.host_rng(seed, W.T_LEN), 256, 2048.0, 0.8, 8192)
        cs = [W.make_custom(lens, Hq=28, Hkv=4, d=128, bs=16, seed=seed + 100 * j, device=dev, poison=False)
              for j in range(2)]
        ws = pdattn.alloc_workspace(256, 28, 4, 128, 16, device=dev)
        out = torch.empty_like(cs[0].q)
        k = [0]

        def step():
            x = cs[k[0] & 1]
            k[0] += 1
            pdattn.decode_ex(x.q, x.k_cache, x.v_cache, x.block_table, x.context_lens, x.scale, out, ws,
                             context_lens_host=x.context_lens_host)

        t = timed(step)
        assert pdattn.check(ws) == pdattn.OK
        by = cs[0].unique_kv_bytes()
        rows.append({"seed": seed, "kv_bytes": by, "ms_per_step": t, "kv_gbs": by / (t * 1e-3) / 1e9,
                     "frac_of_measured_peak": by / (t * 1e-3) / 1e9 / peak, "launches_per_step": pdattn.last_launch_count()})
        del cs, ws, out
        torch.cuda.empty_cache()
    fr = sorted(r["frac_of_measured_peak"] for r in rows)
    return {"per_seed": rows, "frac_min": fr[0], "frac_median": 0.5 * (fr[2] + fr[3]), "frac_max": fr[-1]}


def short_batches(pdattn, W, dev, timed, only="all"):
    """Batches whose pieces are one to a few tiles long: 4096 sequences of the 7B shape under the barrier
    and the chained merge of the decode kernel (and, in the default mode, with the short-piece instantiation
    switched off), and 512 GRPO groups of 8 (40 q / 8 KV heads) that share a 1024-token prompt and have
    generated 1..64 tokens, under both kernels for the shared tiles."""
    res = {}
    rng = np.random.default_rng(0)
    ragged = rng.integers(50, 400, size=4096)
    for name, lens in [("4096x64", np.full(4096, 64)), ("4096x128", np.full(4096, 128)),
                       ("4096xU[50,400]", ragged), ("4096x512", np.full(4096, 512))]:
        if only not in ("all", name):
            continue
        w = W.make_custom(lens, Hq=28, Hkv=4, d=128, bs=16, seed=3, device=dev, poison=False)
        ws = pdattn.alloc_workspace(w.num_seqs, 28, 4, 128, 16, device=dev)
        out = torch.empty_like(w.q)
        row = {"kv_bytes": w.logical_kv_bytes()}
        for mode, key in ((0, "barrier_merge_ms"), (2, "chained_merge_combine_kernel_ms"),
                          (1, "chained_merge_in_kernel_merge_ms"), (-1, "default_ms")):
            pdattn.set_merge_mode(mode)
            row[key] = timed(lambda: pdattn.decode_ex(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale,
                                                      out, ws, context_lens_host=w.context_lens_host))
        row["launches_per_step_default"] = pdattn.last_launch_count()
        pdattn.set_short_piece_path(0)
        row["default_short_piece_kernel_off_ms"] = timed(
            lambda: pdattn.decode_ex(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, ws,
                                     context_lens_host=w.context_lens_host))
        pdattn.set_short_piece_path(-1)
        pdattn.set_merge_mode(-1)
        row["default_kv_gbs"] = row["kv_bytes"] / (row["default_ms"] * 1e-3) / 1e9
        assert pdattn.check(ws) == pdattn.OK
        res[name] = row
        del w, ws, out
        torch.cuda.empty_cache()
    if only not in ("all", "grpo"):
        return res
    lens = 1024 + rng.integers(1, 65, size=4096)
    w = W.make_custom(lens, Hq=40, Hkv=8, d=128, bs=16, seed=3, device=dev, poison=False, shared_prefix_pages=64, group=8)
    gws = pdattn.alloc_grouped_workspace(w.num_seqs, 40, 8, 128, device=dev)
    out = torch.empty_like(w.q)
    pth = np.full(512, 16, dtype=np.int32)
    ptd = torch.from_numpy(pth).to(dev)
    row = {"unique_kv_bytes": w.unique_kv_bytes(), "logical_kv_bytes": w.logical_kv_bytes()}
    row["ungrouped_ms"] = timed(lambda: pdattn.decode_ex(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale,
                                                         out, gws, context_lens_host=w.context_lens_host), n=5)
    for eng, key in ((0, "grouped_warp_mma_ms"), (1, "grouped_tcgen05_ms")):
        pdattn.set_prefix_engine(eng)
        row[key] = timed(lambda: pdattn.decode_grouped(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale,
                                                       out, gws, w.context_lens_host, 8, ptd, pth), n=10)
    pdattn.set_prefix_engine(-1)
    assert pdattn.check(gws) == pdattn.OK
    res["grpo_512x8_prompt1024_resp1..64"] = row
    return res


def decode_loop(pdattn, W, dev, stream, steps=64):
    """64 consecutive growing steps of the same batch: KV append, device-side plan, decode, combine.
    Nothing in a step depends on host knowledge of the lengths.  The tokens read over the loop are
    checked against the closed form of the paper's decode-history feature (Appendix A.1.2)."""
    w = W.make_config(2, device=dev, headroom_tokens=steps + 16)
    S = w.num_seqs
    ws = pdattn.alloc_workspace(S, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size, device=dev)
    out = torch.empty_like(w.q)
    k_new = W.normal_bf16(S * w.num_kv_heads * w.head_dim, 9, 100, dev).view(S, w.num_kv_heads, w.head_dim)
    v_new = W.normal_bf16(S * w.num_kv_heads * w.head_dim, 9, 101, dev).view(S, w.num_kv_heads, w.head_dim)
    lens0 = w.context_lens.clone()
    tokens = torch.zeros((), dtype=torch.int64, device=dev)

    def step():
        pdattn.append_kv(k_new, v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens, workspace=ws,
                         stream=stream)
        pdattn.decode_ex(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, ws,
                         context_lens_host=None, stream=stream)

    # pass 1 (untimed, also the warm-up): count the tokens every step attends to
    for _ in range(steps):
        step()
        tokens += w.context_lens.sum()
    torch.cuda.synchronize()
    want = sum(W.h_dec(int(p), steps) + steps for p in lens0.cpu().tolist())
    assert int(tokens.item()) == want, (int(tokens.item()), want)
    # pass 2 (timed): the same 64 steps again, nothing but the library's launches on the stream
    w.context_lens.copy_(lens0)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(steps):
        step()
    b.record(stream)
    torch.cuda.synchronize()
    assert pdattn.check(ws) == pdattn.OK
    assert torch.equal(w.context_lens, lens0 + steps)
    ms = a.elapsed_time(b) / steps
    return {"steps": steps, "ms_per_step": ms, "seq_steps_per_s": S / (ms * 1e-3),
            "history_tokens_read": want, "launches_per_step": 4}


def _physical_copy(w, seed):
    """Same logical batch in a second, differently permuted set of physical pages."""
    import dataclasses
    NB = w.num_blocks
    dev = w.k_cache.device
    perm = torch.from_numpy(np.random.default_rng(seed).permutation(NB)).to(dev)
    inv = torch.argsort(perm)
    bt = w.block_table.clone().long()
    valid = bt >= 0
    bt[valid] = perm[bt[valid]]
    return dataclasses.replace(w, q=w.q.clone(), k_cache=w.k_cache[inv].contiguous(),
                               v_cache=w.v_cache[inv].contiguous(), block_table=bt.to(torch.int32),
                               context_lens=w.context_lens.clone())


def _reseeded(W, cfg, rank, dev, lens, rng):
    """Another batch of the same configuration for rank > 0: lengths shuffled, values reseeded; what makes the
    configuration what it is stays (config 3: the 8 rows of a group share their 64 prompt pages; config 4: per-head
    scales on K and V)."""
    lens = rng.permutation(lens)
    shapes = {2: (28, 4), 3: (40, 8), 4: (64, 8), 5: (28, 4), 1: (4, 1)}
    Hq, Hkv = shapes[cfg]
    d = 64 if cfg == 1 else 128
    kw = {}
    if cfg == 3:
        kw.update(shared_prefix_pages=1024 // 16, group=8)
    if cfg == 4:
        kw.update(head_scales=True)
    return W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, seed=1000 * cfg + rank, device=dev, **kw)


if __name__ == "__main__":
    main()
