#!/usr/bin/env python
"""Benchmark of the LUVC hot path (OIM + SPU) on B200.

One step = one pass of the whole path over one batch of a configuration: luvc_oim_merge on the
visual-encoder grid, then luvc_spu_prune on the LLM-side hidden states of the merged tokens
(configurations 2 and 3; the seeded projection between the two stands in for the projector and
is not timed), or the two stress operators back to back (configuration 4).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1|2|3|4] [--cutoff C] [--impl reference]
                    [--no-per-config] [--no-cpu-baseline] [--oim-matching bipartite]

Prints ONE JSON line (rank 0).  `value` is vision tokens per second with inputs resident in HBM,
timed with CUDA events on the launching stream; `e2e` is the same metric through the host-buffer
C-ABI entry points (host->device and device->host copies inside the timed region); `roofline`
describes the dominant kernel (the OIM chain kernel) against the measured HBM copy rate read from
MEASURED_PEAKS.json at run time: `achieved` by the algorithmic bytes of a launch, `dram` by the DRAM
bytes of the ncu capture recorded in profiles/ncu_traffic.json (null once the kernel's source has
changed since), `floor` by input-once-plus-outputs-once; `per_config` repeats the device-timed
numbers for configs[2], [3] and [4] with the OIM and SPU roofline objects and, for configs[4], all
nine (cutoff, keep) pairs of the prune; `cpu_baseline` is the CPU oracle timed on this machine's host
cores on a bounded sample (plus the single-thread time of configs[0]).
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

METRIC = "vision tokens/sec through OIM+SPU"
UNIT = "tokens/s"
L2_BYTES = 126 * 1024 * 1024
HBM_NOMINAL_GBS = 8000.0      # the figure the metric's "% of 8 TB/s" divides by
HBM_FALLBACK_GBS = 6650.0     # used only if MEASURED_PEAKS.json is absent



def ncu_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under
    profiles/ (profiles/ncu_traffic.json: kernel or kernel group -> case -> bytes, with the version of the
    source files the counters were taken on; an entry is ignored once one of those files has changed).
    A case is the workload number, for the prune followed by "@" and the cutoff ("4@0.05")."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if not os.path.exists(path):
        return {}
    import hashlib

    table = json.load(open(path))
    out = {}
    for kernel, entry in table.items():
        files = entry.get("sources") or [entry["source"]]
        h = hashlib.sha256()
        for f in files:
            src = os.path.join(ROOT, f)
            h.update(open(src, "rb").read() if os.path.exists(src) else b"missing")
        if h.hexdigest()[:16] == entry.get("source_sha256_16"):
            out[kernel] = {str(k): float(v) for k, v in entry["bytes_per_launch"].items()}
    return out


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", type=int, default=2, choices=[1, 2, 3, 4])
    ap.add_argument("--impl", default="luvc", choices=["luvc", "reference"])
    ap.add_argument("--oim-matching", default="adjacent", choices=["adjacent", "bipartite"],
                    help="bipartite: time the full-line matching variant of OIM instead (device-timed numbers only: "
                         "no end-to-end and no CPU-baseline leg)")
    ap.add_argument("--cutoff", type=float, default=0.0,
                    help="pass band of the prune as a fraction of the band (0 = the workload's own: 0.05 for "
                         "configs[4], the default 0.125 otherwise)")
    ap.add_argument("--cpu-sample", type=int, default=0, help="units of the batch the CPU oracle is timed on (0 = auto)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true",
                    help="skip the per_config object (configs[2]-[4] with the cutoff x keep sweep of configs[4])")
    return ap.parse_args()


# ----------------------------------------------------------------------------- workloads


def workload_spec(k, cutoff=0.0):
    import luvc_inputs as gi

    c = gi.CONFIGS[k]
    spec = dict(id=k, oim=(c["B"], c["H"], c["W"], c["D"]), target=c["target"], keep=c["keep"][0], cutoff=0.0)
    if k == 4:
        spec["spu"] = (c["spu_B"], c["spu_N"], c["D_llm"])
        spec["cutoff"] = c["cutoffs"][0]
        spec["tokens"] = c["B"] * c["H"] * c["W"] + c["spu_B"] * c["spu_N"]
    else:
        T = c["target"]
        spec["spu"] = (c["B"] // c.get("frames", 1), T * c.get("frames", 1), c["D_llm"])
        spec["tokens"] = c["B"] * c["H"] * c["W"]
    if cutoff > 0:
        spec["cutoff"] = cutoff
    return spec


def workload_name(spec):
    B, H, W, D = spec["oim"]
    sb, sn, sd = spec["spu"]
    cut = spec["cutoff"] if spec["cutoff"] > 0 else 0.125
    return ("configs[%d]: OIM %dx%dx%dx%d -> %d tokens/grid, then SPU %dx%dx%d keep %d at cutoff %g%s" % (
        spec["id"], B, H, W, D, spec["target"], sb, sn, sd, spec["keep"], cut,
        " (independent stress inputs)" if spec["id"] == 4 else " (merged tokens through the seeded projection)"))


def oim_iter_bytes(luvc, B, H, W, D, target, e=2):
    """Algorithmic bytes of the OIM chain: every step reads its grid and writes the compacted one,
    tokens plus the int32 size per token."""
    Hf, Wf, n_steps = luvc.oim_plan(H, W, target)
    h, w, total = H, W, 0
    while (h, w) != (Hf, Wf):
        for axis in (0, 1):
            ln, goal = (w, Wf) if axis == 0 else (h, Hf)
            m = min(2, ln - goal, (ln + 1) // 2)
            if ln < 2 or m <= 0:
                continue
            nh, nw = (h, w - m) if axis == 0 else (h - m, w)
            total += B * (h * w + nh * nw) * (D * e + 4)
            h, w = nh, nw
    return total, n_steps


def floor_bytes_oim(B, H, W, D, T, e=2):
    """What must move if the whole chain stayed on chip: the input once, the three outputs once."""
    return B * H * W * D * e + B * T * (D * e + 4) + B * H * W * 4


def spu_bytes(sb, sn, sd, keep, e=2):
    """Algorithmic bytes of one prune: the transform reads the sequence once and writes the scores, the
    select reads them and writes the indices, the gather reads and writes the kept rows."""
    transform = sb * sn * sd * e + sb * sn * 4
    select = sb * sn * 4 + sb * keep * 4
    gather = 2 * sb * keep * sd * e
    return transform, select, gather


def make_inputs(spec, device, sets):
    """`sets` independent input sets (different seeds via batch rolls) so that consecutive steps do
    not find their inputs in L2."""
    import torch

    import luvc_inputs as gi
    import paper_2512_09010_b200 as luvc

    k = spec["id"]
    x0 = gi.oim_input(k, device=device)
    xs = [x0] + [torch.roll(x0, shifts=(s, 3 * s, 5 * s), dims=(0, 1, 2)).contiguous() for s in range(1, sets)]
    if k == 4:
        y0 = gi.spu_stress_input(device=device)
        ys = [y0] + [torch.roll(y0, shifts=(s, 17 * s), dims=(0, 1)).contiguous() for s in range(1, sets)]
    else:
        ys = []
        for x in xs:
            merged = luvc.oim_merge(x, spec["target"])[0]
            ys.append(gi.spu_input_from_tokens(k, merged))
    torch.cuda.synchronize()
    return xs, ys


# ----------------------------------------------------------------------------- clocks


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, device_index):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as exc:  # no NVML: report that clocks were not sampled
            self.err = str(exc)

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for name, bit in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop_evt.wait(0.002)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


# ----------------------------------------------------------------------------- CPU oracle legs


def cpu_oracle_pass(spec, sample_units, x_host, y_host, min_seconds=0.0):
    """Times the CPU oracle (as it stands) on `sample_units` images and the matching sequences."""
    import oracle

    B = spec["oim"][0]
    sb = spec["spu"][0]
    n_img = max(1, min(sample_units, B))
    n_seq = n_img if spec["id"] == 4 else max(1, min(sb, (n_img * sb + B - 1) // B))
    n_seq = min(n_seq, len(y_host))
    cores = oracle.hardware_threads()
    sigma = oracle.spu_sigma(spec["spu"][1], spec["cutoff"])
    t_oim = t_spu = 0.0
    reps = 0
    while reps < 1 or (t_oim + t_spu < min_seconds and reps < 50):   # repeat the sample until the clock is steady
        t0 = time.perf_counter()
        oracle.oim(x_host[:n_img], target=spec["target"])
        t1 = time.perf_counter()
        for b in range(n_seq):
            e = oracle.spu_scores(y_host[b], sigma)
            idx = oracle.spu_select(e, spec["keep"])
            _ = y_host[b][idx]
        t2 = time.perf_counter()
        t_oim += t1 - t0
        t_spu += t2 - t1
        reps += 1
    if spec["id"] == 4:
        tokens = n_img * spec["oim"][1] * spec["oim"][2] + n_seq * spec["spu"][1]
    else:
        tokens = n_img * spec["oim"][1] * spec["oim"][2]      # the sequences are those same grids, merged
    return dict(seconds=t_oim + t_spu, oim_seconds=t_oim, spu_seconds=t_spu, tokens=tokens * reps, cores=cores,
                sample="%d of %d grids through the OIM oracle, %d of %d sequences through the SPU oracle (FFT method), "
                       "repeated %d times" % (n_img, B, n_seq, sb, reps))


def auto_cpu_sample(spec):
    return {1: 32, 2: 8, 3: 16, 4: 1}[spec["id"]]


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch

    import luvc_inputs as gi
    import oracle

    spec = workload_spec(args.workload, args.cutoff)
    k = spec["id"]
    sample = args.cpu_sample or max(1, auto_cpu_sample(spec) // 4)
    B = spec["oim"][0]
    n_img = min(sample, B)
    x = gi.oim_input(k, batch=n_img).float().numpy()
    if k == 4:
        y = gi.spu_stress_input(batch=1).float().numpy()
    else:
        merged = torch.from_numpy(oracle.oim(x, target=spec["target"])["tokens"]).float()
        y = gi.spu_input_from_tokens(k, merged).float().numpy()
    for _ in range(min(args.warmup, 1)):
        cpu_oracle_pass(spec, n_img, x, y)
    steps = max(1, min(args.steps, 3))
    secs, tokens, info = 0.0, 0.0, None
    for _ in range(steps):
        info = cpu_oracle_pass(spec, n_img, x, y)
        secs += info["seconds"]
        tokens += info["tokens"]
    value = tokens / secs
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * secs / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(spec) + ("" if args.oim_matching == "adjacent" else
                                                      " [OIM variant: full-line bipartite matching]"), "note": "CPU oracle on a bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": info["cores"], "kind": "oracle", "sample": info["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- multi-rank bookkeeping


def max_over_ranks(ms_local, world, device="cpu"):
    """The slowest rank's time: every rank contributes its own device-timed milliseconds."""
    if world <= 1:
        return float(ms_local)
    import torch
    import torch.distributed as dist

    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_second(tokens_per_rank, world, ms_per_step):
    """Weak scaling: every rank runs the same per-GPU batch, units are independent, no collective in
    the data path; the job's throughput is all ranks' tokens over the slowest rank's time."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


# ----------------------------------------------------------------------------- the GPU arm


def load_peak():
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        return float(json.load(open(peaks_path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return HBM_FALLBACK_GBS, "fallback"


def rate(nbytes, ms, peak):
    """GB/s and its fractions of the measured copy rate and of the nominal 8 TB/s."""
    if not ms or ms <= 0:
        return {"bytes": nbytes, "ms": ms, "achieved": None, "frac": None, "frac_of_8TBs": None}
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"bytes": nbytes, "ms": ms, "achieved": gbs, "frac": gbs / peak, "frac_of_8TBs": gbs / HBM_NOMINAL_GBS}


def timed_steps(torch, step, steps, warmup, barrier):
    """`warmup` untimed steps, then `steps` steps between two events on the current stream."""
    for i in range(warmup):
        step(i)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for i in range(steps):
        step(i)
    ev1.record()
    barrier()
    return ev0.elapsed_time(ev1)


def phase_times(luvc, step, reps):
    """The library's own events around its phases, one step at a time, averaged."""
    luvc.profile_enable(True)
    phases = {name: 0.0 for name in luvc.PHASES}
    for i in range(reps):
        step(i)
        got = luvc.profile_read()
        for name in phases:
            phases[name] += got[name] / reps
    luvc.profile_enable(False)
    return phases


def oim_roofline(luvc, spec, phases, peak, peak_src, traffic, matching):
    B, H, W, D = spec["oim"]
    iter_bytes, n_steps = oim_iter_bytes(luvc, B, H, W, D, spec["target"], 2)
    steps_ms = phases["oim_steps"]
    r = rate(iter_bytes, steps_ms, peak)
    kernel = "oim_chain_kernel" if matching == "adjacent" else "oim_bipartite_kernel"
    t = traffic.get(kernel, {}).get(str(spec["id"]))
    out = {
        "kernel": "%s (one launch runs the %d merge steps of a call)" % (kernel, n_steps),
        "bound": "hbm", "achieved": r["achieved"], "peak": peak, "unit": "GB/s", "frac": r["frac"],
        "peak_source": peak_src, "frac_of_8TBs": r["frac_of_8TBs"],
        "algorithmic_bytes_per_launch": iter_bytes, "avg_launch_ms": steps_ms, "merge_steps_per_launch": n_steps,
        "algorithmic_bytes_note": "per step: read the grid, write the compacted grid (tokens + sizes), summed over the "
                                  "schedule; this kernel keeps tokens in place, so part of those reads is served by L2 "
                                  "and the compaction write is not performed: see `dram` and `floor`",
        "traffic": t,
        "dram": rate(t, steps_ms, peak) if t else None,
        "floor": rate(floor_bytes_oim(B, H, W, D, spec["target"]), steps_ms, peak),
    }
    return out


def spu_roofline(spec, keep, phases, peak, traffic=None, cutoff=None):
    sb, sn, sd = spec["spu"]
    tb, selb, gb = spu_bytes(sb, sn, sd, keep)
    total_ms = phases["spu_transform"] + phases["spu_select"] + phases["spu_gather"]
    out = rate(tb + selb + gb, total_ms, peak)
    transform = rate(tb, phases["spu_transform"], peak)
    # DRAM bytes of the two transform kernels (forward + inverse) from the ncu capture of this case, if there is one
    cut = cutoff if cutoff is not None else spec["cutoff"]
    case = "%d@%g" % (spec["id"], cut if cut > 0 else 0.125)
    transform["traffic"] = next((v[case] for v in (traffic or {}).values() if case in v), None)
    out.update({"bound": "hbm", "unit": "GB/s", "peak": peak,
                "transform": transform,
                "select": rate(selb, phases["spu_select"], peak),
                "gather": rate(gb, phases["spu_gather"], peak)})
    return out


def per_config_report(torch, luvc, device, peak, peak_src, traffic, barrier, have):
    """configs[2], [3], [4] each timed on this machine: ms per step, the OIM chain's and the SPU's own
    roofline objects, and for configs[4] the whole cutoff x keep sweep of the prune."""
    import luvc_inputs as gi

    report = {}
    for k in (2, 3, 4):
        spec = workload_spec(k)
        if k in have:
            xs, ys, sets = have[k]
        else:
            sets = 2
            xs, ys = make_inputs(spec, device, sets)

        def step(i, spec=spec, xs=xs, ys=ys, sets=sets):
            luvc.oim_merge(xs[i % sets], spec["target"])
            luvc.spu_prune(ys[i % sets], spec["keep"], spec["cutoff"])

        ms = timed_steps(torch, step, 10, 3, barrier) / 10
        ph = phase_times(luvc, step, 10)
        entry = {"workload": workload_name(spec), "ms_per_step": ms, "tokens_per_s": spec["tokens"] / (ms * 1e-3),
                 "phases_ms": ph, "oim": oim_roofline(luvc, spec, ph, peak, peak_src, traffic, "adjacent"),
                 "spu": spu_roofline(spec, spec["keep"], ph, peak, traffic)}
        c = gi.CONFIGS[k]
        sweep = []
        cutoffs = c.get("cutoffs", (0.0,))
        for cutoff in cutoffs:
            for keep in c["keep"]:
                def prune(i, ys=ys, sets=sets, keep=keep, cutoff=cutoff):
                    luvc.spu_prune(ys[i % sets], keep, cutoff)

                timed_steps(torch, prune, 2, 3, barrier)
                ph2 = phase_times(luvc, prune, 6)
                row = spu_roofline(spec, keep, ph2, peak, traffic, cutoff)
                row.update({"cutoff": cutoff if cutoff > 0 else 0.125, "keep": keep})
                sweep.append(row)
        entry["spu_sweep"] = sweep
        report["configs[%d]" % k] = entry
        del xs, ys
        torch.cuda.empty_cache()
    return report


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    import paper_2512_09010_b200 as luvc

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    spec = workload_spec(args.workload, args.cutoff)
    k = spec["id"]
    B, H, W, D = spec["oim"]
    sb, sn, sd = spec["spu"]
    e = 2
    oim_in_bytes = B * H * W * D * e
    spu_in_bytes = sb * sn * sd * e
    sets = max(2, -(-3 * L2_BYTES // max(1, oim_in_bytes + spu_in_bytes)) if k != 4 else 2)
    sets = min(sets, 8)
    xs, ys = make_inputs(spec, device, sets)

    def step(i):
        x, y = xs[i % sets], ys[i % sets]
        a = luvc.oim_merge(x, spec["target"], matching=args.oim_matching)
        b = luvc.spu_prune(y, spec["keep"], spec["cutoff"])
        return a, b

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()

    # ---- timed region: K steps back to back, CUDA events on the launching stream
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = luvc.kernel_launches()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for i in range(args.steps):
        step(i)
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    launches = luvc.kernel_launches() - launches0
    clocks = sampler.stop()
    ms_total = max_over_ranks(ms_total, world, device)
    ms_per_step = ms_total / args.steps
    value = whole_job_tokens_per_second(spec["tokens"], world, ms_per_step)

    # ---- per-phase pass: the library's own events around its phases, one step at a time
    phases = phase_times(luvc, step, min(args.steps, 20))

    # ---- end to end: host buffers through the C ABI, copies inside the timed region
    x_host = xs[0].cpu().pin_memory()
    y_host = ys[0].cpu().pin_memory()
    T = spec["target"]
    o_tok = torch.empty((B, T, D), dtype=xs[0].dtype).pin_memory()
    o_sz = torch.empty((B, T), dtype=torch.int32).pin_memory()
    o_map = torch.empty((B, H * W), dtype=torch.int32).pin_memory()
    o_idx = torch.empty((sb, spec["keep"]), dtype=torch.int32).pin_memory()
    o_hid = torch.empty((sb, spec["keep"], sd), dtype=ys[0].dtype).pin_memory()

    # The two host entry points are independent here (the SPU input is pre-generated) and keep separate
    # staging buffers, so they run from two host threads, each on its own stream: one's device-to-host
    # copy and kernels overlap the other's host-to-device copy, as in a server whose vision and
    # language sides are separate stages.  Each call synchronises its stream before it returns.
    import concurrent.futures
    pool = concurrent.futures.ThreadPoolExecutor(max_workers=2)
    side_streams = [torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)]

    def run_on(stream, fn, *fn_args):
        torch.cuda.set_device(local)
        with torch.cuda.stream(stream):
            fn(*fn_args)

    def e2e_step():
        jobs = [pool.submit(run_on, side_streams[0], luvc.oim_merge_host, x_host, T, o_tok, o_sz, o_map),
                pool.submit(run_on, side_streams[1], luvc.spu_prune_host, y_host, spec["keep"], spec["cutoff"], o_idx,
                            o_hid)]
        for job in jobs:
            job.result()

    e2e_ms = None
    if args.oim_matching == "adjacent":
        for _ in range(3):
            e2e_step()
        barrier()
        e2e_reps = max(3, min(args.steps, 20))
        ev0.record()
        for _ in range(e2e_reps):
            e2e_step()
        ev1.record()
        barrier()
        e2e_ms = max_over_ranks(ev0.elapsed_time(ev1) / e2e_reps, world, device)
    pool.shutdown()
    h2d = x_host.numel() * 2 + y_host.numel() * 2
    d2h = sum(t_.numel() * t_.element_size() for t_ in (o_tok, o_sz, o_map, o_idx, o_hid))
    del x_host, y_host

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (the OIM chain), with the SPU's beside it
    peak, peak_src = load_peak()
    traffic = ncu_traffic()
    roofline = oim_roofline(luvc, spec, phases, peak, peak_src, traffic, args.oim_matching)
    roofline["spu"] = spu_roofline(spec, spec["keep"], phases, peak, traffic)

    per_config = None
    if not args.no_per_config and world == 1 and args.oim_matching == "adjacent":
        per_config = per_config_report(torch, luvc, device, peak, peak_src, traffic, barrier, {k: (xs, ys, sets)})

    cpu = None
    if not args.no_cpu_baseline and args.oim_matching == "adjacent":
        sample = args.cpu_sample or auto_cpu_sample(spec)
        info = cpu_oracle_pass(spec, sample, xs[0][:sample].float().cpu().numpy(),
                               ys[0][: max(1, sample)].float().cpu().numpy(), min_seconds=10.0)
        cpu = {"value": info["tokens"] / info["seconds"], "unit": UNIT, "cores": info["cores"], "kind": "oracle",
               "sample": info["sample"], "seconds": info["seconds"],
               "configs0_single_thread_seconds": config0_single_thread_seconds()}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 arithmetic on bf16 I/O", "data": "synthetic",
        "config": {"workload": workload_name(spec) + ("" if args.oim_matching == "adjacent" else
                                                      " [OIM variant: full-line bipartite matching]"), "l2": "inputs rotate over %d distinct sets (%.0f MB) > L2" % (
            sets, sets * (oim_in_bytes + spu_in_bytes) / 1e6), "parallelism": "batch split, no collective" if world > 1 else "1 GPU"},
        "clocks": clocks,
        "e2e": {"value": whole_job_tokens_per_second(spec["tokens"], world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h} if e2e_ms else None,
        "gpu_launches": launches,
        "phases_ms": phases,
        "roofline": roofline,
        "per_config": per_config,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def config0_single_thread_seconds():
    """The oracle on configs[0] (one fp32 image, then its 144 projected tokens) on ONE host thread."""
    import torch

    import luvc_inputs as gi
    import oracle

    x = gi.oim_input(0).float().numpy()
    t0 = time.perf_counter()
    r = oracle.oim(x, target=gi.CONFIGS[0]["target"], nthreads=1)
    y = gi.spu_input_from_tokens(0, torch.from_numpy(r["tokens"]).float()).float().numpy()
    t1 = time.perf_counter()
    e = oracle.spu_scores(y[0], oracle.spu_sigma(y.shape[1], 0.0), nthreads=1)
    oracle.spu_select(e, gi.CONFIGS[0]["keep"][0])
    t2 = time.perf_counter()
    return {"oim": t1 - t0, "spu": t2 - t1}


if __name__ == "__main__":
    main()
