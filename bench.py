#!/usr/bin/env python
"""Benchmark of the fused LU-KV compression path (score + allocate + select + gather).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one lukv_compress call over one batch of seeded synthetic input.  The default
workload is the Llama-3.1-8B shaped full model at 32k context (256 KV heads allocated
jointly, bf16).  Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank compresses
its own copy of the workload (sequences are independent: weak scaling, no data-path
collective) and the time is the max over ranks.

--impl reference times the CPU oracle (as it stands, single thread) on a bounded sample of
heads of the same workload and prints the same line with "impl": "reference".
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "KV-compress context tokens/s (score+allocate+select+gather)"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b_32k",
                    help="a configuration name, or 'all': one JSON line per configuration (single GPU)")
    ap.add_argument("--path", default="compress", choices=["compress", "profile", "ragged"],
                    help="compress: the headline path; profile: the offline profile build and the online "
                         "lookup front end; ragged: a batch of different context lengths in one call against one "
                         "call per sequence (secondary measurements, single GPU)")
    ap.add_argument("--sinks", type=int, default=0, help="attention sinks kept in every head (App. E uses 4)")
    ap.add_argument("--min-keep", type=float, default=0.0,
                    help="minimum retention per head (App. E uses 0.01); default off, as the headline "
                         "configuration does not name it")
    ap.add_argument("--layers", type=int, default=0,
                    help="override the workload's layer count (a reduced case for profiler captures)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-heads", type=int, default=48, help="heads in the CPU-baseline sample")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


# ---- CPU oracle leg (cpu_baseline of our arm, and the whole reference arm) --------------------

def oracle_sample_seconds(wl, heads, n_sink=0, min_keep=0.0):
    """Seconds the oracle needs for allocation (all heads) plus score/select/gather of `heads`
    sampled heads; returns (seconds, seconds extrapolated to the whole workload)."""
    import numpy as np
    from oracle import lukv_oracle as O
    from paper_2602_08585_b200 import synth
    curves = synth.gen_curves(wl)
    Bs = wl.budgets()
    total_heads = wl.S * wl.N
    heads = min(heads, total_heads)
    sample = [int(x) for x in np.linspace(0, total_heads - 1, heads).round()]
    data = []
    for u in sample:
        q, rem = divmod(u, wl.N)
        layer, h = divmod(rem, wl.H)
        qh, kh, vh = synth.gen_head(wl, q, layer, h, "cpu")
        data.append((u, synth.to_numpy_bits(qh), synth.to_numpy_bits(kh), synth.to_numpy_bits(vh)))
    t0 = time.perf_counter()
    budgets, offsets = O.allocate(curves, wl.T, wl.w, Bs, min_keep=min_keep)
    t_alloc = time.perf_counter() - t0
    t0 = time.perf_counter()
    for u, qh, kh, vh in data:
        _, pooled = O.score_head(qh, kh, wl.kp)
        b = np.array([budgets.reshape(-1)[u]], np.int32)
        off = np.array([0, b[0] + wl.w], np.int32)
        O.select_gather(pooled[None], b, off, kh[None], vh[None], wl.w, n_sink=n_sink)
    t_heads = time.perf_counter() - t0
    return t_alloc + t_heads, t_alloc + t_heads * total_heads / heads, heads


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import lukv_oracle as O
    from paper_2602_08585_b200 import synth
    O.build()
    wl = pick_workload(args)
    heads = max(1, min(4, wl.S * wl.N))
    for _ in range(args.warmup):
        oracle_sample_seconds(wl, 1, args.sinks, args.min_keep)
    full = []
    for _ in range(args.steps):
        _, extrap, used = oracle_sample_seconds(wl, heads, args.sinks, args.min_keep)
        full.append(extrap)
    sec = sum(full) / len(full)
    value = wl.S * wl.T / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded)",
        "config": {"workload": wl.name, "S": wl.S, "heads": wl.N, "T": wl.T, "w": wl.w, "keep": list(wl.keep),
                   "n_sink": args.sinks, "min_keep": args.min_keep},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "host_cores": host_cores(), "kind": "oracle",
                         "sample": f"{heads} of {wl.S * wl.N} heads per step (score+select+gather) plus the full "
                                   "allocation, single thread, extrapolated to all heads"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def host_cores() -> int:
    """Cores this process may run on (the oracle itself uses one thread)."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


# ---- clocks ------------------------------------------------------------------------------------

class ClockSampler(threading.Thread):
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, device_index: int):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception as e:  # NVML missing: the clocks object says so
            self.err = repr(e)

    def sample_once(self):
        nv = self.nv
        self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        try:
            mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
        except Exception:
            mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
        for bit, name in self.REASONS.items():
            if mask & bit:
                self.reasons.add(name)

    def run(self):
        while self.ok and not self._halt.is_set():
            self.sample_once()
            time.sleep(0.002)

    def stop(self):
        self._halt.set()
        if self.ok:
            self.join()

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "note": "NVML unavailable"}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


# ---- our arm -------------------------------------------------------------------------------------

def max_over_ranks(value, dist, device):
    """The job-level time of a step is the slowest rank's: all-reduce MAX (no-op without a process group)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def bf16_peak_tflops():
    """Measured dense bf16 rate of a kernel timed alone (burst), else the earlier measurement on this machine."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops"])
    except Exception:
        return 1590.0


def kernel_bytes(name, wl, rows):
    """Algorithmic bytes one launch of a kernel must move (inputs read once + outputs written once)."""
    es = 2 if wl.dtype == "bf16" else 4
    heads = wl.S * wl.N
    k_bytes = heads * wl.T * wl.d * es
    q_bytes = heads * wl.G * wl.w * wl.d * es
    score_bytes = heads * wl.n * 4
    row = wl.d * es
    if name.startswith("score") and "lse" not in name:
        return k_bytes + q_bytes + (score_bytes if name.endswith("2") or "fused" in name or "onepass" in name else 0)
    if name == "max_pool":
        return 2 * score_bytes
    if name == "select":
        return score_bytes + rows * 4
    if name == "gather":
        return rows * (2 * row * 2 + 4)
    return 0


def load_traffic(kernel, workload):
    """DRAM bytes per launch (read + write) from the committed ncu summary, if one is recorded there:
    lines `traffic <workload> <kernel> <bytes>` in profiles/dram_traffic.txt."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            for line in f:
                t = line.split()
                if len(t) == 4 and t[0] == "traffic" and t[1] == workload and t[2] == kernel:
                    return float(t[3])
    except Exception:
        pass
    return None


def run_ours(args):
    import numpy as np
    import torch
    from paper_2602_08585_b200 import lukv, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (the path has no CPU fallback)"
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    lukv.lib()

    wl = pick_workload(args)
    p = lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P, n_sink=args.sinks,
                         min_keep=args.min_keep)
    q, k, v = synth.gen_tensors(wl, "cuda")
    curves_np = synth.gen_curves(wl)
    curves = torch.from_numpy(curves_np).cuda()
    Bs = wl.budgets()
    ws = lukv.alloc_workspace(p)
    out = lukv.Outputs(p, Bs)

    def step():
        lukv.lukv_compress(p, q, k, v, curves, Bs, out.k_out, out.v_out, out.kept_idx, out.budgets, out.offsets,
                           out.rows, out.dev_status, ws)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 0)):
        step()
    launches_per_step = lukv.lukv_last_launch_count()
    barrier()
    sampler = ClockSampler(local)
    if sampler.ok:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    if sampler.ok and not sampler.samples:
        sampler.sample_once()
    sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    ms = max_over_ranks(ms, dist, "cuda")
    if dist is not None:
        dist.barrier()
    assert int(out.dev_status.item()) == 0
    tokens = wl.S * wl.T * world
    value = tokens / (ms * 1e-3)

    # ---- per-kernel device times (events after every kernel), dominant kernel roofline
    peak, peak_src = measured_peak()
    acc = {}
    reps = 3
    for _ in range(reps):
        for name, t_ms in lukv.lukv_compress_profile(p, q, k, v, curves, Bs, out.k_out, out.v_out, out.kept_idx,
                                                     out.budgets, out.offsets, out.rows, out.dev_status, ws):
            a = acc.setdefault(name, [0.0, 0])
            a[0] += t_ms
            a[1] += 1
    kernels = {name: {"ms_per_launch": tot / cnt, "launches_per_step": cnt // reps} for name, (tot, cnt) in acc.items()}
    total_kernel_ms = sum(kv["ms_per_launch"] * kv["launches_per_step"] for kv in kernels.values())
    for kv in kernels.values():
        kv["share"] = kv["ms_per_launch"] * kv["launches_per_step"] / total_kernel_ms
    dom = max(kernels, key=lambda nm: kernels[nm]["ms_per_launch"] * kernels[nm]["launches_per_step"])
    dom_bytes = kernel_bytes(dom, wl, out.rows)
    dom_s = kernels[dom]["ms_per_launch"] * 1e-3
    dom_gbs = dom_bytes / dom_s / 1e9
    # The bound of record is HBM: the path streams K once and copies the kept rows, and the scorer's algorithmic
    # bytes are K + Q read and the raw scores written.  `frac` = algorithmic bytes / kernel time / measured copy peak.
    roofline = {"kernel": dom, "bound": "hbm", "achieved": dom_gbs, "peak": peak, "unit": "GB/s",
                "frac": dom_gbs / peak, "frac_of_nominal_8TBs": dom_gbs / NOMINAL_HBM_GBS, "peak_source": peak_src,
                "algorithmic_bytes_per_launch": dom_bytes, "ms_per_launch": dom_s * 1e3,
                "traffic": load_traffic(dom, wl.name)}
    if roofline["traffic"]:
        roofline["traffic_gbs"] = roofline["traffic"] / dom_s / 1e9
        roofline["traffic_over_algorithmic"] = roofline["traffic"] / dom_bytes
    if dom.startswith("score") and wl.dtype == "bf16" and wl.d == 128:
        # What holds the tensor-core scorer below the HBM bound: one exp2 per (query row, key) is the method's
        # work; the two-sweep kernel evaluates every one twice (once for the row normaliser, once for the
        # probability).  The unit rate is the special-function units' (16 per clock and SM).
        sms = torch.cuda.get_device_properties(local).multi_processor_count
        exps = 1.0 * wl.S * wl.N * wl.G * wl.w * wl.T
        sweeps = 1 if "onepass" in dom else 2
        peak_exp = 16.0 * sms * (sampler.max_mhz or 1965) * 1e6 / 1e9
        roofline["exp2"] = {"algorithmic_exp2_per_launch": exps, "evaluated_exp2_per_launch": sweeps * exps,
                            "achieved_gexp2_s": exps / dom_s / 1e9,
                            "evaluated_gexp2_s": sweeps * exps / dom_s / 1e9,
                            "unit_peak_gexp2_s": peak_exp, "frac_of_unit_peak_on_algorithmic": exps / dom_s / 1e9 / peak_exp,
                            "frac_of_unit_peak_on_evaluated": sweeps * exps / dom_s / 1e9 / peak_exp,
                            "unit_peak_source": "16 exp2 per clock per SM x SM count x max SM clock; the rates the "
                                                "epilogue reaches in isolation are in profiles/exp2_epilogue_rates.md"}
    es = 2 if wl.dtype == "bf16" else 4
    path_bytes = wl.S * wl.N * wl.T * wl.d * es + 2 * out.rows * wl.d * es   # K read + kept K/V written
    path_gbs = path_bytes / (ms * 1e-3) / 1e9
    path_roofline = {"bytes_per_step": path_bytes, "achieved": path_gbs, "unit": "GB/s",
                     "frac_of_measured_peak": path_gbs / peak, "frac_of_nominal_8TBs": path_gbs / NOMINAL_HBM_GBS}

    # ---- end to end through the C ABI with host buffers (pinned): H2D inputs, compress, D2H results
    e2e = None
    if not args.no_e2e:
        try:
            host_in = [t.cpu().pin_memory() for t in (q, k, v, curves)]
            dev_in = [q, k, v, curves]
            outs = [out.k_out, out.v_out, out.kept_idx, out.budgets, out.offsets]
            host_out = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in outs]

            def e2e_step_one_call():
                for d_, h_ in zip(dev_in, host_in):
                    d_.copy_(h_, non_blocking=True)
                step()
                for h_, d_ in zip(host_out, outs):
                    h_.copy_(d_, non_blocking=True)

            # One sequence: the layers of the cache are contiguous, so layer l can be compressed (one-layer
            # calls of the same C ABI) while layer l+1 is still on its way to the device and the packed rows
            # of layer l-1 are on their way back: three streams, allocation first (it needs only the curves).
            layered = wl.S == 1 and wl.L > 1
            if layered:
                s_in, s_comp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
                p1 = lukv.make_params(1, 1, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P, n_sink=args.sinks,
                                      min_keep=args.min_keep)
                ws1 = lukv.alloc_workspace(p1)
                scores1 = torch.empty((1, wl.H, wl.n), dtype=torch.float32, device="cuda")
                hq, hk, hv, hc = host_in
                hko, hvo, hidx, hbud, hoff = host_out

            def e2e_step_layers():
                main = torch.cuda.current_stream()
                curves.copy_(hc, non_blocking=True)
                lukv.lukv_allocate(p, curves, Bs, out.budgets, out.offsets, ws)
                hbud.copy_(out.budgets, non_blocking=True)
                hoff.copy_(out.offsets, non_blocking=True)
                main.synchronize()            # the host sizes the per-layer result copies from the offsets
                offs = hoff.numpy()
                start = main.record_event()
                for st_ in (s_in, s_comp, s_out):
                    st_.wait_event(start)
                for layer in range(wl.L):
                    with torch.cuda.stream(s_in):
                        q[0, layer].copy_(hq[0, layer], non_blocking=True)
                        k[0, layer].copy_(hk[0, layer], non_blocking=True)
                        v[0, layer].copy_(hv[0, layer], non_blocking=True)
                        arrived = s_in.record_event()
                    s_comp.wait_event(arrived)
                    h0 = layer * wl.H
                    lukv.lukv_score(p1, q[0, layer], k[0, layer], scores1, ws1, stream=s_comp)
                    lukv.lukv_select_gather(p1, scores1, out.budgets[0, h0:], out.offsets[h0:], k[0, layer],
                                            v[0, layer], out.k_out, out.v_out, out.kept_idx, out.rows, ws1,
                                            stream=s_comp)
                    packed = s_comp.record_event()
                    s_out.wait_event(packed)
                    r0, r1 = int(offs[h0]), int(offs[h0 + wl.H])
                    with torch.cuda.stream(s_out):
                        hko[r0:r1].copy_(out.k_out[r0:r1], non_blocking=True)
                        hvo[r0:r1].copy_(out.v_out[r0:r1], non_blocking=True)
                        hidx[r0:r1].copy_(out.kept_idx[r0:r1], non_blocking=True)
                main.wait_stream(s_out)
                main.wait_stream(s_comp)
                main.wait_stream(s_in)

            e2e_step = e2e_step_layers if layered else e2e_step_one_call

            kept_one_call = out.kept_idx.clone()
            e2e_step()
            barrier()
            e0.record()
            for _ in range(args.e2e_steps):
                e2e_step()
            e1.record()
            torch.cuda.synchronize()
            e2e_ms = e0.elapsed_time(e1) / args.e2e_steps
            assert torch.equal(out.kept_idx, kept_one_call) and torch.equal(host_out[2], kept_one_call.cpu()), \
                "the end-to-end run did not reproduce the kept positions of the device-resident run"
            e2e_ms = max_over_ranks(e2e_ms, dist, "cuda")
            e2e = {"value": tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms, "steps": args.e2e_steps,
                   "mode": ("per layer: host-to-device copy | lukv_score + lukv_select_gather | device-to-host copy "
                            "on three streams, after one lukv_allocate") if layered else
                           "one lukv_compress call between the copies",
                   "h2d_bytes_per_step": int(sum(t.numel() * t.element_size() for t in host_in)),
                   "d2h_bytes_per_step": int(sum(t.numel() * t.element_size() for t in host_out))}
            del host_in, host_out
        except Exception as ex:  # e.g. not enough pinned host memory
            e2e = {"value": None, "unit": UNIT, "error": repr(ex)[:200]}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import lukv_oracle as O
        O.build()
        sec, extrap, used = oracle_sample_seconds(wl, args.cpu_heads, args.sinks, args.min_keep)
        cpu_baseline = {"value": wl.S * wl.T / extrap, "unit": UNIT, "cores": 1, "host_cores": host_cores(),
                        "kind": "oracle",
                        "seconds_for_sample": sec,
                        "sample": f"{used} of {wl.S * wl.N} heads (score+select+gather) plus the full allocation, "
                                  "single thread, extrapolated to all heads"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16 in / f32 accumulate" if wl.dtype == "bf16" else "f32",
            "data": "synthetic (seeded)",
            "config": {"workload": wl.name, "S": wl.S, "layers": wl.L, "kv_heads": wl.H, "gqa_group": wl.G,
                       "head_dim": wl.d, "T": wl.T, "w": wl.w, "pool": wl.kp, "curve_points": wl.P,
                       "keep": list(wl.keep), "packed_rows": out.rows, "n_sink": args.sinks,
                       "min_keep": args.min_keep,
                       "l2": "inputs (K+V %.2f GB) exceed the 126 MB L2; no explicit flush" %
                             (2 * wl.S * wl.N * wl.T * wl.d * es / 1e9),
                       "parallelism": "replicas (one full workload per GPU)" if world > 1 else "single GPU"},
            "clocks": sampler.summary(), "roofline": roofline, "path_roofline": path_roofline, "kernels": kernels,
            "e2e": e2e, "cpu_baseline": cpu_baseline, "gpu_launches": launches_per_step * args.steps,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_profile_path(args):
    """Secondary measurement (Sec. 4.3): the offline profile build at the paper's default calibration size
    (30 queries, a 4,000-token context, token-resolution curves, ratios 0.01..0.99) and the online mode
    (lookup + budgeting, scoring, selection, gather) on the headline workload."""
    import time
    import numpy as np
    import torch
    from paper_2602_08585_b200 import lukv, synth

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (the path has no CPU fallback)"
    torch.cuda.set_device(0)
    lukv.lib()
    wl = pick_workload(args)
    Mq, Tc, R = 30, 4000, 99
    ratios = (np.arange(1, R + 1) / 100.0).astype(np.float32)
    calib = lukv.make_params(1, wl.L, wl.H, 1, 64, Tc, wl.w, 1, "fp32", Tc + 1)
    U_np = synth.gen_calibration_curves(synth.BASE_SEED, Mq, wl.N, Tc)
    U = torch.from_numpy(U_np).cuda()
    pws = torch.empty(lukv.lukv_profile_workspace_bytes(calib, Mq, R), dtype=torch.uint8, device="cuda")
    phi = torch.empty((R, wl.N), dtype=torch.float32, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    # curves of the proxy ranking for all calibration queries at once (the queries are the batch)
    pc = lukv.make_params(Mq, wl.L, wl.H, 1, 64, Tc, wl.w, 1, "fp32", Tc + 1)
    g = torch.Generator(device="cuda").manual_seed(synth.BASE_SEED)
    c_scores = torch.rand((Mq, wl.N, Tc - wl.w), generator=g, device="cuda")
    c_imp = -torch.log1p(-torch.rand((Mq, wl.N, Tc - wl.w), generator=g, device="cuda"))
    c_out = torch.empty((Mq, wl.N, Tc + 1), dtype=torch.float32, device="cuda")
    curves_ms = timed(lambda: lukv.lukv_build_curves(pc, c_scores, c_imp, c_out), max(args.steps // 2, 1), 3)
    del c_scores, c_imp, c_out

    # oracle importance of one calibration query (decode queries, the cache, the output projection): 64 decode
    # steps, model width 4096, every head of the workload's shape
    Kd, Dm = 64, 4096
    pi = lukv.make_params(1, wl.L, wl.H, wl.G, wl.d, Tc, wl.w, 1, wl.dtype, Tc + 1)
    dt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    i_q = torch.randn((1, wl.L, wl.H * wl.G, Kd, wl.d), generator=g, device="cuda").to(dt)
    i_k = torch.randn((1, wl.L, wl.H, Tc, wl.d), generator=g, device="cuda").to(dt)
    i_v = torch.randn((1, wl.L, wl.H, Tc, wl.d), generator=g, device="cuda").to(dt)
    i_kd = torch.randn((1, wl.L, wl.H, Kd, wl.d), generator=g, device="cuda").to(dt)
    i_wo = (torch.randn((wl.L, wl.H * wl.G, wl.d, Dm), generator=g, device="cuda") / wl.d ** 0.5).to(dt)
    i_ws = torch.empty(lukv.lukv_importance_workspace_bytes(pi, Kd), dtype=torch.uint8, device="cuda")
    i_out = torch.empty((1, wl.N, Tc - wl.w), dtype=torch.float32, device="cuda")
    imp_ms = timed(lambda: lukv.lukv_oracle_importance(pi, Kd, Dm, i_q, i_k, i_v, i_kd, i_wo, True, i_out, i_ws), 3, 1)
    imp_launches = lukv.lukv_last_launch_count()
    imp_flops = 2.0 * wl.N * wl.G * (Tc - wl.w) * wl.d * Dm + 2.0 * 2 * wl.N * wl.G * Kd * Tc * wl.d
    del i_q, i_k, i_v, i_kd, i_wo, i_ws, i_out

    # KeyDiff proxy scores on the headline workload (a key-only scan; the anchor needs all of a head's keys before
    # its first score, and the kernel reads K from HBM twice)
    pk = lukv.make_params(wl.S, wl.L, wl.H, 1, wl.d, wl.T, 1, 1, wl.dtype, 2)
    kk = torch.randn((wl.S, wl.L, wl.H, wl.T, wl.d), generator=g, device="cuda").to(dt)
    kd_ws = lukv.alloc_workspace(pk)
    kd_out = torch.empty((wl.S, wl.N, wl.T - 1), dtype=torch.float32, device="cuda")
    kd_status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    keydiff_ms = timed(lambda: lukv.lukv_score_keydiff(pk, kk, kd_out, kd_ws, kd_status), args.steps, 3)
    keydiff_launches = lukv.lukv_last_launch_count()
    keydiff_k_bytes = kk.numel() * kk.element_size()
    keydiff_bytes = keydiff_k_bytes + kd_out.numel() * 4
    assert int(kd_status.item()) == 0, "the KeyDiff kernel gave up on a bounded wait"
    del kd_ws, kd_out
    # the whole path with KeyDiff as the proxy metric (recent window 1, no pooling), same curves and keep ratio
    pkp = lukv.make_params(wl.S, wl.L, wl.H, 1, wl.d, wl.T, 1, 1, wl.dtype, wl.P, flags=lukv.FLAG_KEYDIFF)
    kd_Bs = [int(b * (wl.T - 1) // (wl.T - wl.w)) for b in wl.budgets()]
    kd_curves = torch.from_numpy(synth.gen_curves(wl)).cuda()
    kd_vv = torch.randn((wl.S, wl.L, wl.H, wl.T, wl.d), generator=g, device="cuda").to(dt)
    kd_ws = lukv.alloc_workspace(pkp)
    kd_o = lukv.Outputs(pkp, kd_Bs)
    kd_path_ms = timed(lambda: lukv.lukv_compress(pkp, None, kk, kd_vv, kd_curves, kd_Bs, kd_o.k_out, kd_o.v_out,
                                                  kd_o.kept_idx, kd_o.budgets, kd_o.offsets, kd_o.rows,
                                                  kd_o.dev_status, kd_ws), args.steps, 3)
    kd_path_launches = lukv.lukv_last_launch_count()
    assert int(kd_o.dev_status.item()) == 0
    kd_rows = kd_o.rows
    del kk, kd_vv, kd_ws, kd_o, kd_curves

    build_ms = timed(lambda: lukv.lukv_profile_build(calib, U, Mq, ratios, phi, pws), args.steps, max(args.warmup, 3))
    build_launches = lukv.lukv_last_launch_count()

    # exact solver on the first query's curves at 70 % compression, beside the greedy on the same curves
    Bx = int(0.3 * wl.N * (Tc - wl.w))
    xws = torch.empty(lukv.lukv_exact_workspace_bytes(calib, Bx), dtype=torch.uint8, device="cuda")
    xb = torch.empty((1, wl.N), dtype=torch.int32, device="cuda")
    xo = torch.empty((wl.N + 1,), dtype=torch.int32, device="cuda")
    xv = torch.zeros(1, dtype=torch.float64, device="cuda")
    exact_ms = timed(lambda: lukv.lukv_exact_allocate(calib, U[0], [Bx], xb, xo, xv, xws), 3, 1)
    exact_launches = lukv.lukv_last_launch_count()
    gb = torch.empty((1, wl.N), dtype=torch.int32, device="cuda")
    aws = lukv.alloc_workspace(calib)
    lukv.lukv_allocate(calib, U[0], [Bx], gb, xo, aws)
    greedy_raw = float(U[0].double().gather(1, gb[0].long()[:, None]).sum().item())
    exact_val = float(xv.item())
    del xws, aws

    p = lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P)
    q, k, v = synth.gen_tensors(wl, "cuda")
    ws = lukv.alloc_workspace(p)
    sigma = np.array([1.0 - wl.keep[i % len(wl.keep)] for i in range(wl.S)], np.float32)
    budgets = torch.empty((wl.S, wl.N), dtype=torch.int32, device="cuda")
    offsets = torch.empty((wl.S * wl.N + 1,), dtype=torch.int32, device="cuda")
    lookup_ms = timed(lambda: lukv.lukv_profile_budgets(p, phi, ratios, sigma, budgets, offsets), 50, 3)
    rows = int(offsets[-1].item())
    k_out = torch.empty((rows, wl.d), dtype=k.dtype, device="cuda")
    v_out = torch.empty((rows, wl.d), dtype=k.dtype, device="cuda")
    kept = torch.empty((rows,), dtype=torch.int32, device="cuda")
    scores = torch.empty((wl.S, wl.N, wl.n), dtype=torch.float32, device="cuda")
    counts = []

    def online():
        counts.clear()
        lukv.lukv_profile_budgets(p, phi, ratios, sigma, budgets, offsets)
        counts.append(lukv.lukv_last_launch_count())
        lukv.lukv_score(p, q, k, scores, ws)
        counts.append(lukv.lukv_last_launch_count())
        lukv.lukv_select_gather(p, scores, budgets, offsets, k, v, k_out, v_out, kept, rows, ws)
        counts.append(lukv.lukv_last_launch_count())

    sampler = ClockSampler(0)
    if sampler.ok:
        sampler.start()
    online_ms = timed(online, args.steps, max(args.warmup, 3))
    if sampler.ok and not sampler.samples:
        sampler.sample_once()
    sampler.stop()

    cpu = None
    if not args.no_cpu_baseline:
        from oracle import lukv_oracle as O
        O.build()
        t0 = time.perf_counter()
        O.profile_build(U_np[:6], Tc, wl.w, ratios)
        sec = time.perf_counter() - t0
        cpu = {"value": 6 * R / sec, "unit": "(query, ratio) allocations/s", "cores": 1, "host_cores": host_cores(),
               "kind": "oracle",
               "seconds_for_sample": sec, "sample": f"6 of {Mq} calibration queries, all {R} ratios, single thread"}
    es = 2 if wl.dtype == "bf16" else 4
    print(json.dumps({
        "metric": "offline profile build: (query, ratio) allocations per second", "value": Mq * R / (build_ms * 1e-3),
        "unit": "(query, ratio) allocations/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": build_ms, "higher_is_better": True, "dtype": "f32 curves / f64 hull and mean / int64 budgets",
        "data": "synthetic (seeded)", "vs_baseline": None,
        "config": {"workload": f"profile[{wl.name}]", "queries": Mq, "calibration_tokens": Tc, "heads": wl.N,
                   "curve_points": Tc + 1, "ratios": R, "curve_bytes": int(U.numel() * 4)},
        "gpu_launches": build_launches * args.steps,
        "lookup": {"ms_per_call": lookup_ms, "sequences": wl.S, "heads": wl.N},
        "exact_allocate": {"ms_per_call": exact_ms, "heads": wl.N, "positions": Tc - wl.w, "budget": Bx,
                           "launches": exact_launches, "optimum": exact_val, "greedy_on_raw_curves": greedy_raw,
                           "relaxation_gap": (exact_val - greedy_raw) / exact_val},
        "oracle_importance": {"ms_per_call": imp_ms, "queries": 1, "heads": wl.N, "gqa_group": wl.G,
                              "positions": Tc - wl.w, "decode_steps": Kd, "d_model": Dm, "launches": imp_launches,
                              "flops": imp_flops, "tflops": imp_flops / (imp_ms * 1e-3) / 1e12,
                              "frac_of_measured_bf16_peak": imp_flops / (imp_ms * 1e-3) / 1e12 / bf16_peak_tflops()},
        "keydiff_scores": {"ms_per_call": keydiff_ms, "launches": keydiff_launches,
                           "algorithmic_bytes": keydiff_bytes, "gbs": keydiff_bytes / (keydiff_ms * 1e-3) / 1e9,
                           "frac_of_measured_hbm_peak": keydiff_bytes / (keydiff_ms * 1e-3) / 1e9 / measured_peak()[0],
                           "whole_path": {"metric": METRIC, "value": wl.S * wl.T / (kd_path_ms * 1e-3), "unit": UNIT,
                                          "ms_per_step": kd_path_ms, "launches_per_step": kd_path_launches,
                                          "packed_rows": kd_rows, "window": 1},
                           "hbm_bytes_by_design": keydiff_k_bytes + keydiff_bytes,
                           "frac_by_design": (keydiff_k_bytes + keydiff_bytes) / (keydiff_ms * 1e-3) / 1e9
                                             / measured_peak()[0]},
        "build_curves": {"ms_per_call": curves_ms, "queries": Mq, "heads": wl.N, "positions": Tc - wl.w,
                         "algorithmic_bytes": Mq * wl.N * ((Tc - wl.w) * 8 + (Tc + 1) * 4)},
        "online_mode": {"metric": METRIC, "value": wl.S * wl.T / (online_ms * 1e-3), "unit": UNIT,
                        "ms_per_step": online_ms, "packed_rows": rows, "launches_per_step": sum(counts),
                        "path_bytes_per_step": wl.S * wl.N * wl.T * wl.d * es + 2 * rows * wl.d * es},
        "clocks": sampler.summary(), "cpu_baseline": cpu}))


def run_ragged_path(args):
    """Secondary measurement (App. E deployment): the batch of configuration 4 with eight different context
    lengths, compressed by one lukv_compress_ragged call and, for comparison, by one lukv_compress call per
    sequence on the same padded cache."""
    import torch
    from paper_2602_08585_b200 import lukv, synth

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (the path has no CPU fallback)"
    torch.cuda.set_device(0)
    lukv.lib()
    wl = synth.CONFIGS["batch8_16k_mixed"]
    if args.layers > 0:
        wl = synth.scaled(wl, L=args.layers, name=f"{wl.name}[layers={args.layers}]")
    fr = [1.0, 0.5, 0.75, 0.25, 0.875, 0.375, 0.625, 0.125]
    lens = [int(wl.T * fr[q % len(fr)]) for q in range(wl.S)]         # multiples of T/8, hence of the curve grid
    p = lukv.make_params(wl.S, wl.L, wl.H, wl.G, wl.d, wl.T, wl.w, wl.kp, wl.dtype, wl.P)
    q, k, v = synth.gen_tensors(wl, "cuda")
    curves = torch.from_numpy(synth.gen_curves(wl)).cuda()
    Bs = [int(wl.keep[i % len(wl.keep)] * wl.N * (lens[i] - wl.w)) for i in range(wl.S)]
    ws = lukv.alloc_workspace(p)
    out = lukv.Outputs(p, Bs)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn):
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps

    def one_call():
        lukv.lukv_compress_ragged(p, lens, q, k, v, curves, Bs, out.k_out, out.v_out, out.kept_idx, out.budgets,
                                  out.offsets, out.rows, out.dev_status, ws)

    ragged_ms = timed(one_call)
    launches = lukv.lukv_last_launch_count()
    assert int(out.dev_status.item()) == 0
    kept_ragged = out.kept_idx.clone()

    # one call per sequence: the sequence's own parameters on contiguous copies of its part of the cache
    per = []
    row0 = 0
    for i in range(wl.S):
        pi = lukv.make_params(1, wl.L, wl.H, wl.G, wl.d, lens[i], wl.w, wl.kp, wl.dtype, wl.P)
        ki = k[i:i + 1, :, :, :lens[i]].contiguous()
        vi = v[i:i + 1, :, :, :lens[i]].contiguous()
        oi = lukv.Outputs(pi, Bs[i:i + 1])
        per.append((pi, q[i:i + 1], ki, vi, oi, lukv.alloc_workspace(pi), row0))
        row0 += oi.rows
    launches_per_seq = []

    def per_sequence():
        launches_per_seq.clear()
        for pi, qi, ki, vi, oi, wsi, _ in per:
            lukv.lukv_compress(pi, qi, ki, vi, curves, [int(oi.rows - wl.N * wl.w)], oi.k_out, oi.v_out, oi.kept_idx,
                               oi.budgets, oi.offsets, oi.rows, oi.dev_status, wsi)
            launches_per_seq.append(lukv.lukv_last_launch_count())

    seq_ms = timed(per_sequence)
    same = sum(int((kept_ragged[r0:r0 + oi.rows] == oi.kept_idx).sum().item()) for *_, oi, _w, r0 in per)
    tokens = sum(lens)
    es = 2 if wl.dtype == "bf16" else 4
    print(json.dumps({
        "metric": METRIC, "value": tokens / (ragged_ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ragged_ms, "higher_is_better": True, "vs_baseline": None,
        "dtype": "bf16 in / f32 accumulate", "data": "synthetic (seeded)",
        "config": {"workload": f"ragged[{wl.name}]", "ctx_lens": lens, "layers": wl.L, "kv_heads": wl.H,
                   "packed_rows": out.rows, "row_stride_T": wl.T},
        "gpu_launches": launches * args.steps,
        "one_call_per_sequence": {"ms_per_step": seq_ms, "launches_per_step": sum(launches_per_seq),
                                  "kept_rows_identical_to_the_ragged_call": same, "kept_rows": out.rows},
        "launches_per_step": launches,
        "path_bytes_per_step": tokens * wl.N * wl.d * es + 2 * out.rows * wl.d * es}))


def pick_workload(args):
    from paper_2602_08585_b200 import synth
    wl = synth.CONFIGS[args.workload]
    if args.layers > 0 and args.layers != wl.L:
        wl = synth.scaled(wl, L=args.layers, name=f"{wl.name}[layers={args.layers}]")
    return wl


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.path == "profile":
        if int(os.environ.get("RANK", "0")) == 0:
            run_profile_path(args)
    elif args.path == "ragged":
        if int(os.environ.get("RANK", "0")) == 0:
            run_ragged_path(args)
    elif args.workload == "all":
        # one line per configuration, each with its own roofline and clocks (single GPU; the end-to-end and CPU
        # legs only for the headline configuration)
        from paper_2602_08585_b200 import synth
        assert int(os.environ.get("WORLD_SIZE", "1")) == 1, "--workload all is a single-GPU run"
        for name in synth.CONFIGS:
            sub = argparse.Namespace(**vars(args))
            sub.workload = name
            if name != "llama8b_32k":
                sub.no_e2e = sub.no_cpu_baseline = True
            run_ours(sub)
            import gc
            import torch
            gc.collect()
            torch.cuda.empty_cache()
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
