#!/usr/bin/env python
"""Benchmark: derived tuples per second to fixpoint on one B200 (per GPU: independent replicas).

A step is one whole fixpoint (all rounds of join / project / aggregate / dedup / merge) over a seeded synthetic
workload whose facts are already loaded and indexed on the device.  The headline line is the largest single-GPU
configuration, multi-source reachability on an R-MAT scale-22 graph with 64 sources (`reach_rmat22_s64`); the same
run also measures the other four configurations and reports them under `configs`.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload reach|sssp|closure|triangles|digits|...]
  python bench.py --impl reference ...      # times the CPU oracle on the host cores instead

`--gpus N` without a torchrun environment starts N replica processes (one per device) itself.
Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import re
import socket
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "derived tuples/sec to fixpoint"
UNIT = "tuples/s"
HEADLINE = "reach"
ALL_FIVE = ["closure", "sssp", "triangles", "digits", "reach"]           # configurations 1-5


def traffic_ratios():
    """DRAM bytes per algorithmic byte of each kernel, as measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum
    over the launch's algorithmic bytes) and kept in the table of profiles/ncu_traffic_ratios.md together with the
    commands that made them.  Used only to scale a captured launch to the bench's launch size.  {(kernel, route): ratio}"""
    out = {}
    path = os.path.join(ROOT, "profiles", "ncu_traffic_ratios.md")
    if not os.path.exists(path):
        return out
    for line in open(path):
        m = re.match(r"\|\s*(k_\w+)\s*\|\s*(\w+)\s*\|\s*([0-9.]+)\s*\|", line)
        if m:
            out[(m.group(1), m.group(2))] = float(m.group(3))
    return out


def make_program(name: str, scale: int | None, sources: int | None = None):
    from paper_2609_27203_b200 import workloads as W
    if name == "sssp":
        return W.config2(scale=scale or 20), 4 << 30
    if name == "closure":
        return W.config1(), 1 << 28
    if name == "reach":
        s = scale or 22
        ns = sources or 64
        return W.config5(scale=s, n_sources=ns), (56 << 30) if s >= 21 and ns > 16 else (8 << 30)
    if name == "triangles":
        return W.config3(scale=scale or 18), 2 << 30
    if name == "wcoj":
        # the triangle-join fixture of the paper's WCOJ ablation: three relations of 2^scale rows over a hot domain
        s = scale or 16
        return W.hot_domain_triangle(n_rows=1 << s, domain=406 if s == 16 else max(int(1.4 * 2 ** (s / 2)), 8)), 2 << 30
    if name == "cycle4":
        # four-cycle join over four relations of 2^scale uniform rows, one pair in sixteen present (2^24 four-cycles at scale 16)
        s = scale or 16
        return W.uniform_four_cycle(n_rows=1 << s, domain=int(4 * 2 ** (s / 2))), 4 << 30
    if name == "digits":
        return W.config4(), 1 << 30
    if name == "nonlinear":
        # path doubling p(x,z) :- p(x,y), p(y,z): on configuration 1's graph, or (--scale) on a small R-MAT graph
        return (W.nonlinear_rmat_config(scale) if scale else W.nonlinear_config()), 24 << 30
    if name == "mutual":
        return W.mutual_config(), 2 << 30
    raise SystemExit(f"unknown workload {name}")


class ClockSampler:
    """SM clock and throttle reasons sampled while a region runs (NVML from a thread, every few ms, so
    that even a region of a few tens of milliseconds is seen; nvidia-smi at 100 ms as a fallback).
    Only reads the device's state."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None
        self.sm, self.mx, self.reasons, self.thread, self.stop = [], [], set(), None, False

    def _nvml_loop(self, nv, h):
        bits = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self.stop:
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                r = int(get_reasons(h))
                for name, b in bits.items():
                    if r & b:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        try:
            import threading
            import pynvml as nv
            nv.nvmlInit()
            # NVML orders devices by PCI bus id, like CUDA_DEVICE_ORDER=PCI_BUS_ID; honour CUDA_VISIBLE_DEVICES when it is a plain index list
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            idx = self.index
            if vis and all(x.strip().isdigit() for x in vis.split(",")):
                idx = int(vis.split(",")[self.index])
            h = nv.nvmlDeviceGetHandleByIndex(idx)
            self.mx = [float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))]
            self.thread = threading.Thread(target=self._nvml_loop, args=(nv, h), daemon=True)
            self.thread.start()
            return self
        except Exception:
            self.thread = None
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=open(self.path, "w"),
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *a):
        if self.thread:
            self.stop = True
            self.thread.join(timeout=2)
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        if self.thread:
            if not self.sm:
                return None
            return {"sm_mhz": statistics.median(self.sm), "sm_max_mhz": max(self.mx), "samples": len(self.sm),
                    "reasons": sorted(self.reasons), "how": "NVML, 2 ms period, during the timed steps"}
        if not self.path or not os.path.exists(self.path):
            return None
        sm, mx, reasons = [], [], set()
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "samples": len(sm), "reasons": sorted(reasons),
                "how": "nvidia-smi -lms 100 during the timed steps"}


def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def reduce_max(values, world, backend_device=None):
    """Element-wise max over ranks of a list of floats (torch.distributed when world > 1)."""
    if world == 1:
        return list(values)
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=backend_device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def run_oracle_once(program, mode="seminaive"):
    import oracle
    o, ids, _ = oracle.load_program(program)
    t0 = time.perf_counter()
    stats = o.run(mode)
    return time.perf_counter() - t0, stats, o


# ------------------------------------------------------------------------------------------------
MIRROR_JOIN_KERNELS = ("k_res_expand", "k_seg_expand", "k_bm_expand")


L2_PEAK_SOURCE = ("measured here: xlog_device_gather, random 4-byte reads of a 64 MB table (L2-resident), 32 bytes per read: the kernels held "
                  "against it read sorted lists or table slots at random; l2_stream_read_gbs is the library's read-only kernel on the same buffer")
_L2_PEAKS = {}


def l2_peaks():
    """The L2 rates measured on this device with the library's own probe kernels (once per process)."""
    if not _L2_PEAKS:
        from paper_2609_27203_b200 import xlog
        _L2_PEAKS["random_sector_gbs"] = xlog.gather_rate(64 << 20) * 32.0 / 1e9
        _L2_PEAKS["stream_read_gbs"] = xlog.read_bandwidth_gbs(64 << 20, 160)
    return _L2_PEAKS


def roofline_of(program, prof_all, steps, sorting_route):
    """The roofline object of the kernel that takes most of the device time, from the per-kernel CUDA-event table."""
    prof_large = {k[:-len(" (large)")]: v for k, v in prof_all.items() if k.endswith(" (large)")}
    prof = {k: v for k, v in prof_all.items() if not k.endswith(" (large)")}
    ktot = sum(v["ms"] for v in prof.values()) or 1.0
    dom = max(prof, key=lambda k: prof[k]["ms"])
    d = prof[dom]
    peak, peak_src = measured_peak_gbs()
    achieved = d["bytes"] / (d["ms"] / 1e3) / 1e9 if d["ms"] > 0 else 0.0
    mirror_kernel = dom in MIRROR_JOIN_KERNELS or (dom == "k_join_expand" and not sorting_route and "k_sort_pass" not in prof)
    ratio = traffic_ratios().get((dom, "mirror" if mirror_kernel else "sorting"))
    bound = "hbm"
    l2 = None
    probes = None
    if dom == "k_tri_edges" and "n_edges" in program.info:
        # sorted-list intersections served from L1 / L2 (both orientations of the graph fit L2): unit of work = one probe, a binary
        # search of one walked entry in the other sorted list; the launch site declares 4 bytes per probe plus 12 per edge
        probes = (d["bytes"] - 12.0 * program.info["n_edges"] * d["launches"]) / 4.0
    if dom == "k_tri_bitmap":
        # the same intersections against a shared-memory bitmap: one probe = one walked entry tested; 4 bytes declared per probe
        probes = d["bytes"] / 4.0
    if dom in ("k_cycle4", "k_cycle4_bitmap") and program.info.get("domain", 1 << 30) <= 4096:
        # one probe = one walked entry of the shorter list searched in the other (the bitmap kernel always walks t's out-list of z);
        # both launches (count, write) walk every two-path's list
        nd = program.info["domain"]
        adj = {}
        for nm in ("r", "s", "t", "u"):
            (ca, cb), _ = program.facts[nm]
            m = np.zeros((nd, nd), np.float64)
            m[ca, cb] = 1.0
            adj[nm] = m
        two_paths = adj["r"] @ adj["s"]                                            # [x, z]
        walk = np.minimum(adj["t"].sum(axis=1)[None, :], adj["u"].sum(axis=0)[:, None])     # min(out_t(z), in_u(x))
        if dom == "k_cycle4_bitmap":
            walk = np.broadcast_to(adj["t"].sum(axis=1)[None, :], two_paths.shape)
        probes = float((two_paths * walk).sum()) * d["launches"]
    if probes:
        # L2 roofline: L2 bytes per probe from the ncu capture listed in profiles/ncu_traffic_ratios.md (lts__t_bytes.sum over the
        # probes of the captured launch) times the probes per second measured here, against the L2 rate measured here
        # with the library's own random-read kernel on a table that fits L2 (a probe is a step of a binary search)
        per_probe = traffic_ratios().get((dom, "l2probe"))
        instr = traffic_ratios().get((dom, "instr"))
        if per_probe:
            l2_peak = l2_peaks()["random_sector_gbs"]
            rate = probes / (d["ms"] / 1e3)
            l2 = {"achieved": rate * per_probe / 1e9, "peak": l2_peak, "probes_per_s": rate, "l2_bytes_per_probe": per_probe}
            if instr:
                # second figure, not a roofline: share of the issue slots the kernel's own instruction count takes at this rate
                l2["issue"] = {"warp_instructions_per_probe": instr, "utilisation": rate * instr / (148 * 4 * 1.965e9),
                               "what": "instructions per probe from the same ncu capture x probes/s over 148 SMs x 4 schedulers x 1.965 GHz"}
            bound = "l2"
    roofline = {"bound": bound, "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": peak_src,
                "traffic": None if ratio is None else ratio * d["bytes"] / d["launches"],
                "algorithmic_bytes_per_launch": d["bytes"] / d["launches"], "launches_per_step": d["launches"] / steps,
                "avg_launch_us": 1e3 * d["ms"] / d["launches"], "share_of_kernel_time": d["ms"] / ktot,
                "kernels": {k: {"launches_per_step": v["launches"] / steps, "ms_per_step": v["ms"] / steps,
                                "GBps": (v["bytes"] / (v["ms"] / 1e3) / 1e9) if v["ms"] > 0 and v["bytes"] else None}
                            for k, v in sorted(prof.items(), key=lambda kv: -kv[1]["ms"])},
                "how": "second pass of the same steps with XLOG_FLAG_PROFILE (CUDA events around every launch on the ctx stream; "
                       "the resident rounds are then launched one by one instead of as one graph)"}
    big = prof_large.get(dom)
    if big and big["ms"] > 0:
        # the same kernel over its launches of at least 4 M candidates only (small rounds are launch- and latency-bound)
        g = big["bytes"] / (big["ms"] / 1e3) / 1e9
        roofline["large_launches"] = {"launches_per_step": big["launches"] / steps, "ms_per_step": big["ms"] / steps,
                                      "achieved": g, "frac": g / peak, "what": "this kernel's launches of at least 48 MB algorithmic bytes (4 M candidates x 12 B) only"}
    per_cand = traffic_ratios().get((dom, "l2cand"))
    if big and big["ms"] > 0 and per_cand and mirror_kernel:
        # second roofline of the large launches: the slots sit in L2 and every candidate reads one at random, so the bytes that
        # count are L2's.  L2 bytes per candidate from the ncu capture listed in profiles/ncu_traffic_ratios.md (lts__t_bytes.sum of a
        # large launch over its candidates) x candidates/s measured here, against the L2 bandwidth measured here.
        pk = l2_peaks()
        cps = big["bytes"] / 12.0 / (big["ms"] / 1e3)
        roofline["large_launches"]["l2"] = {"achieved": cps * per_cand / 1e9, "peak": pk["random_sector_gbs"], "frac": cps * per_cand / 1e9 / pk["random_sector_gbs"],
                                            "unit": "GB/s", "l2_bytes_per_candidate": per_cand, "candidates_per_s": cps,
                                            "peak_source": L2_PEAK_SOURCE, "l2_stream_read_gbs": pk["stream_read_gbs"]}
    if l2:
        roofline.update(achieved=l2["achieved"], peak=l2["peak"], unit="GB/s", frac=l2["achieved"] / l2["peak"], traffic=None,
                        peak_source=L2_PEAK_SOURCE, l2_stream_read_gbs=l2_peaks()["stream_read_gbs"],
                        probes_per_s=l2["probes_per_s"], l2_bytes_per_probe=l2["l2_bytes_per_probe"])
        if "issue" in l2:
            roofline["issue"] = l2["issue"]
    if dom in ("k_row_fixpoint", "k_dense_round"):
        roofline["limiter"] = ("every round runs out of shared memory with the looked-up relation in L2; the rows cross HBM once, so the HBM "
                               "fraction says nothing: read ms_per_step and the metric")
    if mirror_kernel:
        # the tag-mirror joins move few bytes per candidate by construction; what limits them is said here
        roofline["limiter"] = ("instruction issue; the table, too large for L2, is read from HBM one 128-byte line per (changed unit of 32 keys, neighbour)"
                               if dom in ("k_seg_expand", "k_bm_expand") else
                               "L2 random sector access (one tag-mirror slot per candidate); HBM carries about 8 B per candidate")
        if dom not in ("k_seg_expand", "k_bm_expand"):
            roofline["candidates_per_s"] = achieved * 1e9 / 12.0
    return roofline


def measure(name, args, steps, warmup, local_rank, world, flush, with_e2e):
    """Timed fixpoints of one workload on this rank's device: (summary dict, program).  Facts are resident and indexed
    before the timed region; L2 is flushed between steps."""
    import torch
    import torch.distributed as dist
    from paper_2609_27203_b200 import xlog
    dev = f"cuda:{local_rank}"
    headline = name == args.workload
    program, arena = make_program(name, args.scale if headline else None, args.sources if headline else None)
    base_flags = (xlog.FLAG_NO_TAG_MIRROR if args.no_tag_mirror else 0) | (xlog.FLAG_NO_GRAPH if args.no_graph else 0) | (xlog.FLAG_NO_RESIDENT_LOOP if args.no_resident_loop else 0)
    base_flags |= (xlog.FLAG_NO_BITMAP_JOIN if args.no_bitmap_join else 0)
    base_flags |= {"auto": 0, "wcoj": xlog.FLAG_FORCE_WCOJ, "chain": xlog.FLAG_FORCE_CHAIN}[args.triangle_plan]
    ctx, ids, rules = xlog.load_program(program, device=local_rank, arena_bytes=arena, device_inputs=True, flags=base_flags)

    def step(c):
        c.reset_idb()
        flush.fill_(1)                                                       # evict L2 between iterations
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        r = c.fixpoint()
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1), r

    for _ in range(warmup):
        step(ctx)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    times, launches, receipt = [], 0, None
    with ClockSampler(local_rank) as clk:
        for _ in range(steps):
            ms, receipt = step(ctx)
            times.append(ms)
            launches += receipt["kernel_launches"]
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    total_ms = reduce_max([sum(times)], world, dev)[0]
    ms_per_step = total_ms / steps
    derived = receipt["derived_tuples"]
    out = {"program": program, "ms_per_step": ms_per_step, "value": derived * world / (ms_per_step / 1e3), "times": times,
           "launches": launches, "receipt": receipt, "clocks": clk.summary(), "derived": derived}

    # per-kernel timing: the same steps again with CUDA events around every launch
    ctx.close()
    pctx, pids, _ = xlog.load_program(program, device=local_rank, arena_bytes=arena, device_inputs=True,
                                      flags=xlog.FLAG_PROFILE | base_flags)
    step(pctx)
    pctx.profile_reset()
    for _ in range(steps):
        step(pctx)
    prof_all = pctx.profile()
    pctx.close()
    out["roofline"] = roofline_of(program, prof_all, steps, args.no_tag_mirror)
    if not with_e2e:
        return out

    # end to end through the C ABI with HOST buffers: load (H2D + sort + index), fixpoint, read back (D2H)
    pinned = {}
    h2d = 0
    for rname, (cols, tags) in program.facts.items():
        pc = [torch.from_numpy(np.ascontiguousarray(c, np.int32)).pin_memory() for c in cols]
        pt = None if tags is None else torch.from_numpy(np.ascontiguousarray(tags, np.float32)).pin_memory()
        pinned[rname] = (pc, pt)
        h2d += sum(c.numel() * 4 for c in pc) + (0 if pt is None else pt.numel() * 4)
    empty = type(program)(program.name, program.relations, program.rules, {}, program.outputs)
    ectx, eids, _ = xlog.load_program(empty, device=local_rank, arena_bytes=arena, flags=base_flags)

    def e2e_step():
        t0 = time.perf_counter()
        for rname, (pc, pt) in pinned.items():
            ectx.load(eids[rname], [c.numpy() for c in pc], None if pt is None else pt.numpy())
        r = ectx.fixpoint()
        d2h = 0
        for rname in program.outputs:
            cols, tags = ectx.read(eids[rname])
            d2h += (len(cols) + 1) * 4 * len(tags)
        torch.cuda.synchronize()
        return (time.perf_counter() - t0) * 1e3, r, d2h

    for _ in range(min(warmup, 2)):
        e2e_step()
    if world > 1:
        dist.barrier()
    e_times, d2h = [], 0
    for _ in range(max(1, min(steps, 5))):
        ms, r, d2h = e2e_step()
        e_times.append(ms)
    e_ms = reduce_max([sum(e_times) / len(e_times)], world, dev)[0]
    ectx.close()
    out["e2e"] = {"value": derived * world / (e_ms / 1e3), "unit": UNIT, "ms_per_step": e_ms, "h2d_bytes_per_step": h2d,
                  "d2h_bytes_per_step": d2h, "how": "xlog_relation_load from pinned host + xlog_fixpoint + xlog_relation_read to host, wall clock"}
    return out


def config_of(args_workload, m, world):
    program, receipt = m["program"], m["receipt"]
    return {"workload": program.name, "program": args_workload, **{k: v for k, v in program.info.items()},
            "derived_tuples": m["derived"], "rounds": receipt["iterations"], "candidates": receipt["candidates"],
            "triangle_plan": {0: None, 1: "wcoj", 2: "chain"}[receipt["triangle_plan"]],
            "unique_candidates": receipt["unique_candidates"], "l2": "flushed between steps (256 MB fill)",
            "parallelism": "replicas only" if world > 1 else "1 gpu", "facts": "resident and indexed before timing"}


def run_ours(args):
    import torch
    import torch.distributed as dist

    rank, local_rank, world = dist_env()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    torch.cuda.set_device(local_rank)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=f"cuda:{local_rank}")          # > 126 MB L2

    m = measure(args.workload, args, args.steps, args.warmup, local_rank, world, flush, with_e2e=True)
    out = {"metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32 keys / f32 tags",
           "data": "synthetic", "impl": "ours", "config": config_of(args.workload, m, world),
           "clocks": m["clocks"], "e2e": m["e2e"], "gpu_launches": m["launches"], "roofline": m["roofline"],
           "step_ms_min_med_max": [min(m["times"]), statistics.median(m["times"]), max(m["times"])]}

    # the other configurations, each at its full size: a short run of the same protocol (no end-to-end leg)
    if args.workload == HEADLINE and args.scale is None and args.sources is None and not args.no_other_configs:
        others = {}
        for name in ALL_FIVE:
            if name == args.workload:
                continue
            o = measure(name, args, min(args.steps, 5), 3, local_rank, world, flush, with_e2e=False)
            r = o["roofline"]
            others[o["program"].name] = {"program": name, "ms_per_fixpoint": o["ms_per_step"], "tuples_per_s": o["value"],
                                         "derived_tuples": o["derived"], "rounds": o["receipt"]["iterations"], "candidates": o["receipt"]["candidates"],
                                         "launches_per_fixpoint": o["launches"] / min(args.steps, 5),
                                         "dominant_kernel": r["kernel"], "bound": r["bound"], "achieved": r["achieved"], "unit": r["unit"],
                                         "frac": r["frac"], "large_launches_frac": (r.get("large_launches") or {}).get("frac"),
                                         "large_launches_l2_frac": ((r.get("large_launches") or {}).get("l2") or {}).get("frac"),
                                         "clocks": o["clocks"]}
        out["configs"] = others

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # the oracle as it stands, on this machine's host cores, on a bounded sample of the same workload
        # (about 10-30 s of CPU work): the full workload where the oracle manages it, else a smaller R-MAT scale
        cpu_scale = args.cpu_scale or {"triangles": 14, "reach": 16, "wcoj": 13, "cycle4": 15}.get(args.workload)
        sample, _ = make_program(args.workload, cpu_scale) if cpu_scale else (m["program"], 0)
        sec, stats, _o = run_oracle_once(sample)
        out["cpu_baseline"] = {"value": stats["derived_tuples"] / sec, "unit": UNIT, "cores": 1, "kind": "oracle",
                               "seconds": sec, "host_cores_available": os.cpu_count(),
                               "sample": f"{sample.name}: one semi-naive fixpoint of the std::map oracle, single thread, facts pre-loaded"}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


# ------------------------------------------------------------------------------------------------
FULL_SCALE = {"sssp": 20, "reach": 22, "triangles": 18, "wcoj": 16, "cycle4": 16}
# seconds of one oracle fixpoint at the full size (host-core measurements of earlier runs; only used to size the sample)
ORACLE_SECONDS_FULL = {"sssp": 12.0, "reach": 3400.0, "closure": 3.0, "triangles": 3200.0, "digits": 3.0, "wcoj": 60.0, "cycle4": 60.0,
                       "nonlinear": 400.0, "mutual": 8.0}
REFERENCE_BUDGET_S = 420.0


def run_reference(args):
    """The oracle on the host cores, same metric and workload name as the GPU arm.  Each step is one fixpoint of the
    workload itself where (steps + warmup) of them fit the time budget, else of a smaller R-MAT scale of the same program
    (the line then says so in `sample_of` / `config.sample`)."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    n_runs = args.steps + args.warmup
    scale = args.scale
    full_name = make_name(args.workload, args.scale, args.sources)
    if args.workload in FULL_SCALE and scale is None:
        scale = FULL_SCALE[args.workload]
        while scale > 8 and n_runs * ORACLE_SECONDS_FULL[args.workload] * 2.0 ** (scale - FULL_SCALE[args.workload]) > REFERENCE_BUDGET_S:
            scale -= 1
    program, _ = make_program(args.workload, scale, args.sources)
    import oracle
    o, ids, _ = oracle.load_program(program)
    times, stats = [], None
    for i in range(n_runs):
        o.reset()
        t0 = time.perf_counter()
        stats = o.run("seminaive")
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt * 1e3)
    ms = sum(times) / len(times)
    value = stats["derived_tuples"] / (ms / 1e3)
    sample = f"{program.name}: semi-naive fixpoint of the std::map oracle, single thread, facts pre-loaded"
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int32 keys / f32 tags", "data": "synthetic", "impl": "reference",
            "config": {"workload": full_name, "program": args.workload, "sample": program.name, **program.info,
                       "derived_tuples": stats["derived_tuples"]},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    if program.name != full_name:
        line["sample_of"] = (f"{full_name}: one oracle fixpoint at full size takes about {ORACLE_SECONDS_FULL[args.workload]:.0f} s on one host core, "
                             f"so {n_runs} of them do not fit {REFERENCE_BUDGET_S:.0f} s; each step is the same program on {program.name}")
    print(json.dumps(line))


def make_name(workload, scale, sources):
    """Name of the workload make_program would build, without generating it."""
    if workload == "sssp":
        return f"sssp_rmat{scale or 20}"
    if workload == "reach":
        return f"reach_rmat{scale or 22}_s{sources or 64}"
    if workload == "triangles":
        return f"triangles_rmat{scale or 18}"
    if workload == "closure":
        return "closure_n1000_m4000"
    if workload == "digits":
        return "digits_B65536"
    return make_program(workload, scale, sources)[0].name


def spawn_replicas(n):
    """`--gpus N` outside a torchrun environment: start N ranks of this script (one per device) on this node."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE, choices=["sssp", "closure", "reach", "triangles", "digits", "wcoj", "cycle4", "nonlinear", "mutual"])
    ap.add_argument("--scale", type=int, default=None, help="R-MAT scale override (smaller cases for profiling)")
    ap.add_argument("--sources", type=int, default=None, help="reach: number of sources (fewer for a small profiling case)")
    ap.add_argument("--triangle-plan", default="auto", choices=["auto", "wcoj", "chain"], help="wcoj workload: force a join plan")
    ap.add_argument("--no-resident-loop", action="store_true", help="tag-mirror rounds driven by the host (one control read per round)")
    ap.add_argument("--no-graph", action="store_true", help="launch the resident rounds one by one (for per-launch profiling)")
    ap.add_argument("--no-tag-mirror", action="store_true", help="evaluate recursion by sort -> reduce-by-key -> merge only")
    ap.add_argument("--no-bitmap-join", action="store_true", help="grouped join from a delta row list instead of the changed bitmap")
    ap.add_argument("--no-other-configs", action="store_true", help="headline workload only (skip the `configs` object)")
    ap.add_argument("--cpu-scale", type=int, default=None, help="R-MAT scale of the cpu_baseline sample (default: the workload's)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_replicas(args.gpus))
    if args.impl == "reference":
        run_reference(args)
    else:
        if args.warmup < 3:
            print("note: fewer than 3 warm-up steps requested", file=sys.stderr)
        run_ours(args)


if __name__ == "__main__":
    main()
