#!/usr/bin/env python
"""Benchmark of the token-routing hot path (stats -> assign -> permute -> combine) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 5] [--impl reference]

One "step" is one pass of all four stages over one batch of synthetic gating output.  The
default workload is the largest benchmark config (T=131072, E=256, K=8, H=7168, 4x8 ranks).
Rank 0 prints ONE JSON line: whole-job routed (token, expert) pairs per second with inputs
resident in HBM (`value`), the same step driven from pinned host buffers (`e2e`), the HBM
roofline of the dominant kernel (`roofline`) and of every stage (`stages`), the CPU oracle
timed on a bounded sample (`cpu_baseline`), and the SM clocks seen during the timed region.
With --gpus N > 1 (launched by torchrun) every rank routes its own replica of the workload:
the path has no cross-GPU step, so scaling is weak and no collective is on the data path.
`--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "routed token-expert pairs/sec"
UNIT = "pairs/s"
FALLBACK_HBM_GBS = 6650.0          # earlier measurement on this machine, used if MEASURED_PEAKS.json is absent
def kernels_per_step(T, fused):
    """Launches of one step.  Fused: the index kernel, the row mover, the combine.  Four separate calls:
    stats 2 (clear + tile), assign 2 (clear + assign), permute 4 (hist, scan, rank, rows), combine 1; the
    statistics of a batch that fits a single cluster (at most 16 CTAs of 256 tokens) store their sums and
    need no clearing kernel."""
    if fused:
        return 3
    return 9 - (1 if 0 < T <= 4096 else 0)

TRAFFIC_JSON = os.path.join(ROOT, "profiles", "row_kernels_traffic.json")
COUNTERS_JSON = os.path.join(ROOT, "profiles", "index_kernels_counters.json")


def load_json(path):
    try:
        with open(path) as f:
            return json.load(f)
    except Exception:
        return {}


def traffic_from_ncu_csv(csv_path, tokens, K, H, command):
    """Turns `ncu -i <report> --page raw --csv` of a reduced-size capture into the per-pair DRAM
    traffic of the two row kernels and writes it where the benchmark reads it."""
    import csv
    with open(csv_path) as f:
        rows = list(csv.reader(f))
    hdr = rows[0]
    out = load_json(TRAFFIC_JSON)
    names = {"perm_rows_bulk_oneshot_kernel": "permute_rows", "combine_kernel": "combine"}
    for r in rows[2:]:
        d = dict(zip(hdr, r))
        stage = next((v for k, v in names.items() if k in d.get("Kernel Name", "")), None)
        if stage is None or "backward" in d.get("Kernel Name", ""):
            continue
        total = float(d["dram__bytes_read.sum"]) + float(d["dram__bytes_write.sum"])
        unit = hdr.index("dram__bytes_read.sum")
        scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}.get(rows[1][unit], 1.0)
        out[stage] = {"bytes_per_pair": total * scale / (tokens * K), "captured_tokens": tokens, "K": K, "H": H,
                      "kernel": d["Kernel Name"], "command": command}
    with open(TRAFFIC_JSON, "w") as f:
        json.dump(out, f, indent=1, sort_keys=True)
        f.write("\n")
    return out


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default="5")
    ap.add_argument("--step", default="fused", choices=["fused", "separate"],
                    help="the timed step: cobalt_route_index + cobalt_permute_rows + cobalt_combine (three kernels, "
                         "default) or the four stages as separate calls (nine kernels); same outputs either way, and "
                         "the other form is timed beside it")
    ap.add_argument("--tokens", type=int, default=None, help="override T (reduced-size runs for profiling)")
    ap.add_argument("--hidden", type=int, default=None, help="override H (tiny rows isolate the index stages)")
    ap.add_argument("--impl", default="cobalt", choices=["cobalt", "reference"])
    ap.add_argument("--cpu-sample-tokens", type=int, default=None,
                    help="tokens of the workload the CPU oracle is timed on (default 32768 in both legs)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="only the timed step loop (for launch lists under a profiler)")
    ap.add_argument("--clock-period-ms", type=float, default=8.0,
                    help="period of the SM clock / throttle-reason sampling during the timed region (0 = no sampling)")
    ap.add_argument("--traffic-from", default=None, metavar="CSV",
                    help="no benchmark: read `ncu -i <report> --page raw --csv` of a reduced-size capture of the row "
                         "kernels (taken with --tokens T) and write profiles/row_kernels_traffic.json")
    ap.add_argument("--counters-from", default=None, metavar="CSV",
                    help="no benchmark: read `ncu -i <report> --page raw --csv` of the index kernels and write "
                         "profiles/index_kernels_counters.json")
    ap.add_argument("--traffic-command", default="", help="the command that made the capture, recorded beside the figures")
    ap.add_argument("--summarise", nargs="+", default=None, metavar="JSON",
                    help="no benchmark: print a markdown table (per-stage times and fractions) of earlier output lines")
    return ap.parse_args()


def workload_name(w, T=None):
    T = w.T if T is None else T
    return (f"config {w.name}: T={T} E={w.E} K={w.K} H={w.H} bf16, layout {w.N} nodes x {w.Q} ranks x "
            f"{w.S} slots (D={w.D}), P={T * w.K} pairs")


def stage_bytes(w):
    """Algorithmic bytes each stage must move (ids/maps int32, rows bf16)."""
    T, K, E, H, D, P = w.T, w.K, w.E, w.H, w.D, w.P
    return {
        "coact_stats": 4 * P + 4 * E * E + 4 * E,
        "assign": 4 * P + 4 * T + 4 * P + 4 * D + T,
        "permute_index": 4 * P + 4 * P + 4 * P + 4 * (2 * D + 1),
        # one pass: ids and source ranks in; slots, both maps, remote_nodes, coact, load, counts and offsets out
        "route_index": 4 * P + 4 * T + 4 * P + 4 * P + 4 * P + T + 4 * E * E + 4 * E + 4 * (2 * D + 1),
        "permute_rows": 2 * T * H + 2 * P * H + 4 * P,
        "combine": 2 * P * H + 2 * T * H + 4 * P + 4 * P,
    }


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


# ---------------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline and --impl reference)
# ---------------------------------------------------------------------------------------------
def oracle_step(w, x_bits):
    """All four stages of the oracle, as it stands, on the host. Returns seconds."""
    import oracle as O
    t0 = time.perf_counter()
    O.coact_stats(w.topk_ids, w.E)
    r = O.assign(w.N, w.Q, w.S, w.E, w.slot_expert, w.primary_slot, w.topk_ids, w.src_rank, w.seed)
    p = O.permute(r["assigned_slot"], w.D, x_bits)
    O.combine(p["send"], p["row_of_pair"], w.gate_w)
    return time.perf_counter() - t0


CPU_SAMPLE_TOKENS = 32768          # the oracle is timed on the first tokens of the workload, in both legs


def cpu_sample(config, tokens, hidden=None):
    import workloads as W
    w = W.make_config(config, T=tokens)
    if hidden is not None:
        w.H = hidden
    return w, w.hidden_rows()


def cpu_sample_text(ws, extra=""):
    return (f"first {ws.T} tokens of the workload ({ws.P} pairs), all four stages of the oracle as it stands, "
            f"single thread{extra}")


def config_dict(name_T, w):
    """The `config` object of the JSON line: the same for both arms (the reference arm describes the
    workload it samples, not the sample; that is in cpu_baseline.sample)."""
    cold = name_T * w.K * w.H * 2 > (1 << 28)
    return {"workload": workload_name(w, T=name_T), "seed": int(w.seed),
            "l2": ("no explicit flush: each step streams the send buffer (larger than L2) through L2 twice, "
                   "so every stage starts cold") if cold else "inputs smaller than L2: stages run warm",
            "parallelism": "replicas only (no cross-GPU step on this path)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    full_T = args.tokens or _default_T(args.config)
    w, x_bits = cpu_sample(args.config, min(args.cpu_sample_tokens or CPU_SAMPLE_TOKENS, full_T), args.hidden)
    budget_s = 150.0
    t_begin = time.perf_counter()
    warm = 0
    for _ in range(max(0, args.warmup)):
        oracle_step(w, x_bits)
        warm += 1
        if time.perf_counter() - t_begin > budget_s / 2:
            break
    times = []
    for _ in range(max(1, args.steps)):
        times.append(oracle_step(w, x_bits))
        if time.perf_counter() - t_begin > budget_s:
            break
    sec = sum(times) / len(times)
    value = w.P / sec
    sample = cpu_sample_text(w, f", mean of {len(times)} runs, {sec:.2f} s each")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": len(times), "warmup": warm, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "dtype_detail": "bf16 rows moved bit-exactly, fp32 accumulation in the combine, u32 counts, i32 indices",
        "data": "synthetic", "config": config_dict(full_T, w),
        "cpu_baseline": dict({"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
                             **host_description()),
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def _default_T(config):
    return {"1": 4096, "1a": 4096, "2": 16384, "3": 32768, "4": 65536, "5": 131072}[str(config)]


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    """SM clock, power and throttle reasons of one GPU, sampled while the timed region runs: through
    NVML from a thread every few milliseconds (reads only), or, without the NVML module, from an
    nvidia-smi loop."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
    PERIOD_S = 0.008

    def __init__(self, device_id):
        self.proc = None
        self.thread = None
        self.rows = []                      # (epoch seconds, sm MHz, max sm MHz, watts, [reason strings])
        self.device_index = device_id       # an index or a "GPU-<uuid>" string
        self.how = None

    def _nvml_loop(self, handle, nv):
        bits = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        try:
            max_sm = float(nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM))
        except Exception:
            max_sm = float("nan")
        n_taken, watts = 0, float("nan")
        while not self._stop:
            try:
                sm = float(nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM))
                reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(handle))
                n_taken += 1
                if n_taken % 8 == 1:                       # the power reading is the slow one
                    watts = nv.nvmlDeviceGetPowerUsage(handle) / 1000.0
                self.rows.append((time.time(), sm, max_sm, watts,
                                  ["Active" if reasons & bits[n] else "Not Active" for n in self.NAMES]))
            except Exception:
                pass
            time.sleep(self.PERIOD_S)

    def start(self):
        try:
            import threading

            import pynvml as nv
            nv.nvmlInit()
            dev = str(self.device_index)
            handle = nv.nvmlDeviceGetHandleByUUID(dev) if dev.startswith("GPU-") else nv.nvmlDeviceGetHandleByIndex(int(dev))
            self._stop = False
            self.thread = threading.Thread(target=self._nvml_loop, args=(handle, nv), daemon=True)
            self.thread.start()
            self.how = f"NVML every {self.PERIOD_S * 1e3:.0f} ms"
            return
        except Exception:
            self.thread = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.device_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.how = "nvidia-smi every 20 ms"
        except Exception:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Median SM clock and throttle reasons over the samples taken inside [t_begin, t_end]
        (wall-clock seconds since the epoch); all samples if no window is given or none fall in it."""
        rows = []
        if self.thread is not None:
            time.sleep(0.02)
            self._stop = True
            self.thread.join(timeout=2)
            rows = list(self.rows)
        elif self.proc is not None:
            time.sleep(0.1)
            self.proc.terminate()
            try:
                out, _ = self.proc.communicate(timeout=5)
            except Exception:
                self.proc.kill()
                out = ""
            for line in out.splitlines():
                f = [v.strip() for v in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(f[1]), float(f[2]), float(f[3]), f[4:8]))
                except ValueError:
                    continue
        else:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        inside = [r for r in rows if t_begin is not None and t_begin <= r[0] <= t_end]
        window = "timed region" if inside else "whole run (no sample fell inside the timed region)"
        use = inside or rows
        reasons = set()
        for r in use:
            for name, v in zip(self.NAMES, r[4]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(r[1] for r in use) if use else None,
                "sm_min_mhz": min(r[1] for r in use) if use else None,
                "sm_max_mhz": max(r[2] for r in use) if use else None,
                "power_w_max": max((r[3] for r in use if r[3] == r[3]), default=None),
                "reasons": sorted(reasons), "samples": len(use), "window": window, "sampler": self.how}


def host_description():
    """The host the CPU oracle is timed on: logical CPUs, model name, the threads the oracle uses."""
    model = None
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"nproc": os.cpu_count(), "cpu_model": model, "threads_used": 1}


# ---------------------------------------------------------------------------------------------
# aggregation over ranks (every rank routes its own replica; nothing crosses GPUs on the data path)
# ---------------------------------------------------------------------------------------------
def max_over_ranks(ms: float, device) -> float:
    """Slowest rank's time: all-reduce(MAX) when a process group is up, else the value itself."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, pairs_per_rank: int, ms_per_step: float) -> float:
    """Pairs routed by all ranks per second of the slowest rank's step time (weak scaling)."""
    return world * pairs_per_rank / (ms_per_step * 1e-3)


# ---------------------------------------------------------------------------------------------
# secondary measurements (rank 0): a same-run copy, the index stages warm and launch-free, and the
# traffic model on a layout whose co-activation clusters share a node
# ---------------------------------------------------------------------------------------------
def extra_measurements(args, w, step, cb, torch):
    import numpy as np
    out = {}

    def timed(fn, n, warm=3):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    # device-to-device copy of half the send buffer into the other half, in this very run
    half = step.send.shape[0] // 2
    if half > 0 and half * w.H * 2 > (1 << 27):
        ms = timed(lambda: step.send[half:2 * half].copy_(step.send[:half]), 5)
        out["same_run_copy_gbs"] = 2 * half * w.H * 2 / (ms * 1e-3) / 1e9
        step.permute()                       # restore the send buffer

    # stats + assign + permutation index replayed from a CUDA graph: inputs L2-resident (warm),
    # no per-launch host latency; compare with the cold per-stage times of the step loop
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            def index_stages():
                step.stats()
                step.assign(w.seed)
                cb.permute_index(step.assigned_slot, w.D, step.dest_counts, step.dest_offsets, step.row_of_pair,
                                 step.pair_of_row, step.workspace)
            for _ in range(3):
                index_stages()
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                index_stages()
            ms = timed(graph.replay, 50)
        torch.cuda.current_stream().wait_stream(side)
        out["index_stages_graph_replay_warm_us"] = ms * 1e3
    except Exception as exc:          # capture is best effort; the step loop numbers stand on their own
        out["index_stages_graph_replay_warm_us"] = None
        out["graph_replay_error"] = str(exc)[:200]

    # each index stage warm: 50 calls back to back between one pair of events, inputs L2-resident,
    # launches queued ahead of the GPU (what a stage costs when the gating kernel has just written the ids)
    try:
        out["index_stages_warm_us"] = {
            "coact_stats": timed(step.stats, 50) * 1e3,
            "assign": timed(lambda: step.assign(w.seed), 50) * 1e3,
            "permute_index": timed(lambda: cb.permute_index(step.assigned_slot, w.D, step.dest_counts,
                                                            step.dest_offsets, step.row_of_pair, step.pair_of_row,
                                                            step.workspace), 50) * 1e3,
        }
    except Exception as exc:
        out["index_stages_warm_us"] = None
        out["index_stages_warm_error"] = str(exc)[:200]

    # What the timing method itself costs: a pair of events around nothing, around one kernel that
    # only clears 257 KB (coact_stats with an empty batch), and around the statistics call at this
    # batch size, each behind a 256 MB fill so that the launches are queued before the GPU gets to them
    try:
        fill = torch.empty(256 << 20, dtype=torch.uint8, device=step.x.device)
        none = torch.empty((0, w.K), dtype=torch.int32, device=step.x.device)

        def cold_us(fn, n=30):
            best = []
            for _ in range(n + 3):
                fill.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn()
                e1.record()
                torch.cuda.synchronize()
                best.append(e0.elapsed_time(e1) * 1e3)
            return float(np.median(best[3:]))

        out["timing_floor_us"] = {
            "event_pair_alone": cold_us(lambda: None),
            "one_clearing_kernel": cold_us(lambda: cb.coact_stats(none, w.E, step.coact, step.load)),
            "coact_stats": cold_us(step.stats),
        }
        del fill
    except Exception as exc:
        out["timing_floor_us"] = None
        out["timing_floor_error"] = str(exc)[:200]

    # What binds the statistics and the assignment is not HBM: the rate of shared-memory atomic adds and
    # of instruction issue, measured here on this device by the measurement kernels of cobalt_peaks.h
    try:
        from paper_2609_36959_b200 import peaks
        out["sm_peaks"] = {
            "shared_atomic_adds_per_clk_sm_conflict_free": peaks.shared_atomics_conflict_free(),
            "shared_atomic_adds_per_clk_sm_stats_pattern": (peaks.shared_atomics_stats_pattern(step.topk_ids, w.E)
                                                            if w.K in (1, 2, 4, 6, 8) and w.E <= 600 else None),
            "warp_instructions_per_clk_sm": peaks.issue_rate(0),
            "warp_instructions_per_clk_sm_hash_mix": peaks.issue_rate(1),
            "how": "one CTA of 1024 threads per SM, SM cycle counter over the slowest CTA, warm; "
                   "stats pattern = the K(K+1)/2 adds per token of this workload's ids into the 16-bit triangle, nothing else",
        }
    except Exception as exc:
        out["sm_peaks"] = {"error": str(exc)[:200]}

    # the same step with stages 1, 2 and the permutation index fused into one pass over the ids
    try:
        n = max(5, min(args.steps, 30))
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n)]
        for _ in range(3):
            step.route_fused(w.seed)
        torch.cuda.synchronize()
        for i in range(n):
            ev[i][0].record()
            cb.route_index(step.layout, step.topk_ids, step.src_rank, w.seed, step.coact, step.load,
                           step.assigned_slot, step.dest_counts, step.dest_offsets, step.row_of_pair, step.workspace,
                           remote_nodes=step.remote_nodes, totals=step.totals, pair_of_row=step.pair_of_row)
            ev[i][1].record()
            cb.permute_rows(step.x, step.row_of_pair, w.K, step.send)
            step.combine()
            ev[i][2].record()
        torch.cuda.synchronize()
        out["fused_route_index_us"] = sum(e[0].elapsed_time(e[1]) for e in ev) / n * 1e3
        out["fused_step_ms"] = ev[0][0].elapsed_time(ev[-1][2]) / n
        out["fused_step_pairs_per_s"] = w.P / (out["fused_step_ms"] * 1e-3)
    except Exception as exc:
        out["fused_route_index_us"] = None
        out["fused_error"] = str(exc)[:200]

    # the four-stage step with the statistics on a side stream beside the other stages
    try:
        n = max(5, min(args.steps, 30))
        for _ in range(3):
            step.route(w.seed, overlap_stats=True)
        out["stats_overlapped_step_ms"] = timed(lambda: step.route(w.seed, overlap_stats=True), n)
        out["stats_overlapped_step_pairs_per_s"] = w.P / (out["stats_overlapped_step_ms"] * 1e-3)
        out["sequential_step_ms_same_loop"] = timed(lambda: step.route(w.seed), n)
    except Exception as exc:
        out["stats_overlapped_step_ms"] = None
        out["stats_overlap_error"] = str(exc)[:200]

    # the four-stage step replayed from a CUDA graph (seed read from a device word at run time)
    try:
        n = max(5, min(args.steps, 30))
        step.capture()
        out["graph_step_ms"] = timed(lambda: step.replay(w.seed), n)
        out["graph_step_pairs_per_s"] = w.P / (out["graph_step_ms"] * 1e-3)
        step.capture(fused=True)
        out["graph_fused_step_ms"] = timed(lambda: step.replay(w.seed), n)
    except Exception as exc:
        out["graph_step_ms"] = None
        out["graph_step_error"] = str(exc)[:200]

    # the next two blocks allocate one more buffer of the send buffer's size: only with room to spare
    send_bytes = step.send.numel() * 2

    def has_room():
        free, _ = torch.cuda.mem_get_info()
        return free > 1.5 * send_bytes + (2 << 30)

    # backward of the two row stages (adjoints), same buffers: grad_send := send, grad_y := y
    try:
        if not has_room():
            raise RuntimeError("skipped: not enough free device memory for another send-sized buffer")
        peak, _ = hbm_peak()
        grad_x = torch.empty_like(step.x)
        grad_out = torch.empty_like(step.send)
        grad_w = torch.empty_like(step.gate_w)
        T, K, H, P = w.T, w.K, w.H, w.P
        ms = timed(lambda: cb.permute_backward(step.send, step.row_of_pair, K, grad_x), 10)
        b = 2 * P * H + 2 * T * H + 4 * P
        out["permute_backward"] = {"ms": ms, "bytes": b, "gbs": b / ms / 1e6, "frac": b / ms / 1e6 / peak}
        ms = timed(lambda: cb.combine_backward(step.y, step.send, step.row_of_pair, step.gate_w, grad_out, grad_w), 10)
        b = 2 * T * H + 4 * P * H + 12 * P
        out["combine_backward"] = {"ms": ms, "bytes": b, "gbs": b / ms / 1e6, "frac": b / ms / 1e6 / peak}
        del grad_x, grad_out, grad_w
    except Exception as exc:
        out["backward_error"] = str(exc)[:200]

    # node-deduplicated send layout: one row per (token, destination node) instead of per pair
    try:
        torch.cuda.empty_cache()
        if not has_room():
            raise RuntimeError("skipped: not enough free device memory for another send-sized buffer")
        peak, _ = hbm_peak()
        T, K, H, P, N = w.T, w.K, w.H, w.P, w.N
        node_counts = torch.zeros(N, dtype=torch.int32, device="cuda")
        node_offsets = torch.zeros(N + 1, dtype=torch.int32, device="cuda")
        node_row = torch.zeros(T * N, dtype=torch.int32, device="cuda")
        fwd = torch.zeros(P, dtype=torch.int32, device="cuda")
        cross = torch.zeros(1, dtype=torch.int64, device="cuda")
        ws = torch.empty(cb.dedup_workspace_bytes(T, K, N), dtype=torch.uint8, device="cuda")

        def index():
            cb.dedup_index(step.assigned_slot, step.src_rank, N, w.Q, w.S, node_counts, node_offsets, node_row, fwd, ws,
                           cross_node_rows=cross)
        ms_index = timed(index, 20)
        rows = int(node_offsets[-1])
        dedup_send = torch.empty((rows, H), dtype=torch.bfloat16, device="cuda")
        ms_rows = timed(lambda: cb.dedup_rows(step.x, node_row, N, dedup_send), 10)
        recv = torch.empty_like(step.send)
        ms_fwd = timed(lambda: cb.forward_rows(dedup_send, fwd, step.row_of_pair, recv), 10)
        b_rows = 2 * T * H + 2 * rows * H + 4 * T * N
        b_fwd = 2 * rows * H + 2 * P * H + 8 * P      # every buffer row read once, every pair row written
        out["dedup_layout"] = {
            "n_rows": rows, "pairs": P, "rows_per_pair": rows / P, "cross_node_rows": int(cross[0]),
            "buffer_bytes": rows * H * 2, "plain_buffer_bytes": P * H * 2, "bytes_saved_frac": 1 - rows / P,
            "index_us": ms_index * 1e3,
            "fill": {"ms": ms_rows, "gbs": b_rows / ms_rows / 1e6, "frac": b_rows / ms_rows / 1e6 / peak},
            "forward": {"ms": ms_fwd, "gbs": b_fwd / ms_fwd / 1e6, "frac": b_fwd / ms_fwd / 1e6 / peak},
            "recv_equals_send": bool(torch.equal(recv.view(torch.int16), step.send.view(torch.int16)))}
        del dedup_send, recv
    except Exception as exc:
        out["dedup_layout"] = {"error": str(exc)[:200]}

    # Stage 2 of the planner closed on one box: this step's w_er -> greedy intra-node rebalancing ->
    # the same tokens assigned over the new layout (rank-load imbalance = max / mean, as in the paper)
    try:
        load = step.slot_load.cpu().numpy().astype(np.float32)
        new_layout, moved, kept = cb.rebalance_intra_node(w.N, w.Q, w.S, w.E, w.slot_expert.tolist(), load.tolist())
        lay2 = cb.Layout(w.N, w.Q, w.S, w.E, new_layout)
        slots2 = torch.zeros_like(step.assigned_slot)
        load2 = torch.zeros_like(step.slot_load)
        cb.assign(lay2, step.topk_ids, step.src_rank, w.seed, slots2, slot_load=load2)
        before = load.reshape(w.G, w.S).sum(axis=1)
        after = load2.cpu().numpy().astype(np.float64).reshape(w.G, w.S).sum(axis=1)
        out["stage2_rebalance"] = {"imbalance_before": float(before.max() / before.mean()),
                                   "imbalance_after": float(after.max() / after.mean()), "nodes_kept": kept}
    except Exception as exc:
        out["stage2_rebalance"] = {"error": str(exc)[:200]}

    # Eq. 1 under a layout that co-locates each co-activation cluster (what the paper's global
    # planner aims for), same ids: reported as context
    try:
        import workloads as W
        wc = W.make_config(args.config, clustered=True, T=min(w.T, 32768))
        lay = cb.Layout(wc.N, wc.Q, wc.S, wc.E, wc.slot_expert.tolist(), wc.primary_slot.tolist())
        ids = torch.from_numpy(wc.topk_ids).cuda()
        src = torch.from_numpy(wc.src_rank).cuda()
        slots = torch.zeros((wc.T, wc.K), dtype=torch.int32, device="cuda")
        totals = torch.zeros(2, dtype=torch.int64, device="cuda")
        cb.assign(lay, ids, src, wc.seed, slots, totals=totals)
        v, vn = totals.cpu().tolist()
        out["traffic_model_clustered_layout"] = {
            "tokens": wc.T, "V_cobalt": v, "V_naive": vn,
            "remote_nodes_per_token_cobalt": v / wc.T, "remote_nodes_per_token_naive": vn / wc.T,
            "cross_node_reduction": (1 - v / vn) if vn else None}
    except Exception as exc:
        out["traffic_model_clustered_layout"] = {"error": str(exc)[:200]}
    return out


# ---------------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------------
def run_cobalt(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2609_36959_b200 as cb
    import workloads as W
    from paper_2609_36959_b200.router import RouteStep

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the routing path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    distributed = world > 1 or "TORCHELASTIC_RUN_ID" in os.environ   # under torchrun: always through NCCL
    if distributed:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()

    w = W.make_config(args.config, T=args.tokens)
    if args.hidden is not None:
        w.H = args.hidden
    need = 2 * w.P * w.H + 4 * w.T * w.H + 64 * w.P + (1 << 28)     # send + x + y + index arrays + slack
    free, _ = torch.cuda.mem_get_info()
    if free < need:
        raise SystemExit(f"bench.py: {workload_name(w)} needs about {need / 2**30:.1f} GiB of device memory, "
                         f"only {free / 2**30:.1f} GiB are free on cuda:{local_rank}")
    layout = cb.Layout(w.N, w.Q, w.S, w.E, w.slot_expert.tolist(), w.primary_slot.tolist())
    step = RouteStep(layout, w.T, w.K, w.H)

    # pinned host copies of the inputs (the e2e leg reads them every step)
    ids_h = torch.from_numpy(w.topk_ids).pin_memory()
    w_h = torch.from_numpy(w.gate_w).pin_memory()
    src_h = torch.from_numpy(w.src_rank).pin_memory()
    x_h = torch.empty((w.T, w.H), dtype=torch.bfloat16).pin_memory()
    blk = 16384
    for t0 in range(0, w.T, blk):
        t1 = min(w.T, t0 + blk)
        x_h[t0:t1].copy_(torch.from_numpy(w.hidden_rows(t0, t1).view(np.int16)).view(torch.bfloat16))
    step.topk_ids.copy_(ids_h); step.gate_w.copy_(w_h); step.src_rank.copy_(src_h); step.x.copy_(x_h)
    torch.cuda.synchronize()

    names = ["coact_stats", "assign", "permute_index", "permute_rows", "combine"]
    fused_names = ["route_index", "permute_rows", "combine"]

    def separate_step(events=None):
        """The four stages as four calls (cobalt_permute split into its two halves so that the row mover is
        timed on its own): nine kernels."""
        def mark(i):
            if events is not None:
                events[i].record()
        mark(0)
        step.stats()
        mark(1)
        step.assign(w.seed)
        mark(2)
        cb.permute_index(step.assigned_slot, w.D, step.dest_counts, step.dest_offsets, step.row_of_pair,
                         step.pair_of_row, step.workspace)
        mark(3)
        cb.permute_rows(step.x, step.row_of_pair, w.K, step.send)
        mark(4)
        step.combine()
        mark(5)

    def fused_step(events=None):
        """The same outputs from three kernels: stages 1, 2 and the index half of 3 in one (cobalt_route_index)."""
        def mark(i):
            if events is not None:
                events[i].record()
        mark(0)
        cb.route_index(step.layout, step.topk_ids, step.src_rank, w.seed, step.coact, step.load, step.assigned_slot,
                       step.dest_counts, step.dest_offsets, step.row_of_pair, step.workspace,
                       remote_nodes=step.remote_nodes, totals=step.totals, pair_of_row=step.pair_of_row)
        mark(1)
        cb.permute_rows(step.x, step.row_of_pair, w.K, step.send)
        mark(2)
        step.combine()
        mark(3)

    headline_fused = args.step == "fused"
    one_step = fused_step if headline_fused else separate_step
    n_marks = 4 if headline_fused else 6

    def timed_loop(fn, marks, n_steps):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(marks)] for _ in range(n_steps)]
        for i in range(n_steps):
            fn(evs[i])
        torch.cuda.synchronize()
        return evs

    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:
        gpu_id = local_rank
    sampler = ClockSampler(gpu_id)
    sampler.PERIOD_S = args.clock_period_ms * 1e-3
    if rank == 0 and args.clock_period_ms > 0:
        sampler.start()
    for _ in range(max(3, args.warmup)):
        one_step()
    barrier()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(n_marks)] for _ in range(args.steps)]
    barrier()
    t_epoch0 = time.time()
    t_wall0 = time.perf_counter()
    for i in range(args.steps):
        one_step(ev[i])
    barrier()
    t_wall = time.perf_counter() - t_wall0
    clocks = sampler.stop(t_epoch0, t_epoch0 + t_wall) if rank == 0 else None

    total_ms = ev[0][0].elapsed_time(ev[-1][n_marks - 1])
    head_names = fused_names if headline_fused else names
    per_step = {n: [e[i].elapsed_time(e[i + 1]) for e in ev] for i, n in enumerate(head_names)}
    err_bits = cb.read_and_clear_device_error()
    # the other form of the step, same number of steps, for the stages the headline loop does not separate
    other_total_ms = None
    if rank == 0 and not args.no_extras:
        if headline_fused:
            ev2 = timed_loop(separate_step, 6, args.steps)
            other = {n: [e[i].elapsed_time(e[i + 1]) for e in ev2] for i, n in enumerate(names)}
            other_total_ms = ev2[0][0].elapsed_time(ev2[-1][5]) / args.steps
            for n in ("coact_stats", "assign", "permute_index"):
                per_step[n] = other[n]
        else:
            ev2 = timed_loop(fused_step, 4, args.steps)
            per_step["route_index"] = [e[0].elapsed_time(e[1]) for e in ev2]
            other_total_ms = ev2[0][0].elapsed_time(ev2[-1][3]) / args.steps
    stage_ms = {n: sum(v) / len(v) for n, v in per_step.items()}

    ms_per_step = max_over_ranks(total_ms, "cuda") / args.steps
    value = whole_job_value(world, w.P, ms_per_step)

    extras = {}
    if rank == 0:
        extras = {} if args.no_extras else extra_measurements(args, w, step, cb, torch)

    # end to end from pinned host buffers: H2D of the inputs, four stages, D2H of the results
    e2e = None
    if not args.no_e2e:
        y_h = torch.empty((w.T, w.H), dtype=torch.bfloat16).pin_memory()
        coact_h = torch.empty((w.E, w.E), dtype=torch.int32).pin_memory()
        load_h = torch.empty((w.E,), dtype=torch.int32).pin_memory()
        sl_h = torch.empty((w.D,), dtype=torch.int32).pin_memory()
        tot_h = torch.empty((2,), dtype=torch.int64).pin_memory()
        n_e2e = max(3, min(args.steps, 30))
        for _ in range(2):
            step.route_host(w.seed, ids_h, w_h, src_h, x_h, y_h, coact_h, load_h, sl_h, tot_h)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        # the steps are queued back to back without joining the copy-out stream in between, so a
        # step's inputs start moving in while the previous step's last results move out; the
        # closing event is recorded after the last copy out has been joined
        e0.record()
        for i in range(n_e2e):
            step.route_host(w.seed, ids_h, w_h, src_h, x_h, y_h, coact_h, load_h, sl_h, tot_h,
                            join=(i == n_e2e - 1))
        e1.record()
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), "cuda") / n_e2e
        e2e = {"value": whole_job_value(world, w.P, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": step.h2d_bytes(), "d2h_bytes_per_step": step.d2h_bytes(), "steps": n_e2e}

    if rank == 0:
        peak, peak_src = hbm_peak()
        sb = stage_bytes(w)
        stages = {}
        for n in [m for m in ["coact_stats", "assign", "permute_index", "route_index", "permute_rows", "combine"] if m in stage_ms]:
            gbs = sb[n] / (stage_ms[n] * 1e-3) / 1e9
            stages[n] = {"ms": stage_ms[n], "ms_median": statistics.median(per_step[n]), "ms_min": min(per_step[n]),
                         "bytes": sb[n], "gbs": gbs, "frac": gbs / peak,
                         "frac_of_nominal_8TBs": gbs / 8000.0,
                         "frac_of_same_run_copy": (gbs / extras["same_run_copy_gbs"]
                                                   if extras.get("same_run_copy_gbs") else None),
                         "pairs_per_s": w.P / (stage_ms[n] * 1e-3)}
        # second roofline of the two small stages: the SM resource that binds them
        pk = extras.get("sm_peaks") or {}
        counters = load_json(COUNTERS_JSON).get(f"config{w.name}", {}) if w.T == _default_T(w.name) else {}
        n_sm = torch.cuda.get_device_properties(local_rank).multi_processor_count
        sm_hz = (clocks.get("sm_mhz") or 1965.0) * 1e6 if clocks else 1965.0e6
        if pk.get("shared_atomic_adds_per_clk_sm_conflict_free"):
            adds = w.T * w.K * (w.K + 1) // 2
            rate = adds / (stage_ms["coact_stats"] * 1e-3 * sm_hz * n_sm)
            stages["coact_stats"]["second_bound"] = {
                "bound": "shared-memory atomic adds", "adds": adds, "unit": "adds per clock per SM", "achieved": rate,
                "peak_conflict_free": pk["shared_atomic_adds_per_clk_sm_conflict_free"],
                "frac_of_conflict_free": rate / pk["shared_atomic_adds_per_clk_sm_conflict_free"],
                "peak_this_pattern": pk.get("shared_atomic_adds_per_clk_sm_stats_pattern"),
                "frac_of_this_pattern": (rate / pk["shared_atomic_adds_per_clk_sm_stats_pattern"]
                                         if pk.get("shared_atomic_adds_per_clk_sm_stats_pattern") else None),
                "note": "whole stage (clearing kernel, launch, merge) against the adds alone"}
        instr = (counters.get("assign_kernel") or {}).get("warp_instructions")
        if pk.get("warp_instructions_per_clk_sm") and instr:
            rate = instr / (stage_ms["assign"] * 1e-3 * sm_hz * n_sm)
            stages["assign"]["second_bound"] = {
                "bound": "instruction issue", "warp_instructions": instr, "unit": "warp instructions per clock per SM",
                "achieved": rate, "peak": pk["warp_instructions_per_clk_sm"], "frac": rate / pk["warp_instructions_per_clk_sm"],
                "note": "instruction count from the ncu capture in profiles/index_kernels_counters.json; whole stage "
                        "(clearing kernel, launch) against issue alone"}
        dom = max(("permute_rows", "combine"), key=lambda n: stage_ms[n])
        # DRAM bytes per pair from the ncu capture of a reduced token count on this row shape
        # (profiles/row_kernels_traffic.json); traffic grows in proportion to the pairs of a launch
        captured = load_json(TRAFFIC_JSON).get(dom, {})
        traffic = captured.get("bytes_per_pair") if (captured.get("H"), captured.get("K")) == (w.H, w.K) else None
        roofline = {"bound": "hbm", "kernel": dom, "achieved": stages[dom]["gbs"], "peak": peak,
                    "unit": "GB/s", "frac": stages[dom]["frac"], "peak_source": peak_src,
                    "traffic": None if traffic is None else traffic * w.P,
                    "traffic_source": None if traffic is None else
                    f"ncu dram__bytes_read+write per pair at T={captured.get('captured_tokens')}, scaled to {w.P} pairs",
                    "algorithmic_bytes": sb[dom], "ms_per_launch": stage_ms[dom]}
        totals = step.totals.cpu().tolist()
        load = step.slot_load.cpu().numpy().astype(np.int64).reshape(w.G, w.S).sum(axis=1)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "dtype_detail": "bf16 rows moved bit-exactly, fp32 accumulation in the combine, u32 counts, i32 indices",
            "data": "synthetic",
            "config": config_dict(w.T, w),
            "step": ("cobalt_route_index (stages 1, 2 and the index half of 3 in one kernel) + cobalt_permute_rows + "
                     "cobalt_combine; the four separate calls are timed beside it (stages, four_stage_step_ms)"
                     if headline_fused else "cobalt_coact_stats + cobalt_assign + cobalt_permute + cobalt_combine"),
            "e2e": e2e, "gpu_launches": kernels_per_step(w.T, headline_fused) * args.steps,
            "roofline": roofline, "stages": stages, "clocks": clocks,
            "traffic_model": {"V_cobalt": totals[0], "V_naive": totals[1],
                              "remote_nodes_per_token_cobalt": totals[0] / max(w.T, 1),
                              "remote_nodes_per_token_naive": totals[1] / max(w.T, 1),
                              "cross_node_reduction": (1 - totals[0] / totals[1]) if totals[1] else None,
                              "rank_load_imbalance": float(load.max() / load.mean()) if load.sum() else None},
            "four_stage_step_ms": other_total_ms if headline_fused else ms_per_step,
            "fused_step_ms": ms_per_step if headline_fused else other_total_ms,
            "device_error_bits": err_bits, "wall_s_timed_region": t_wall, "extras": extras,
        }
        if not args.no_cpu_baseline and world == 1:
            ws, xs = cpu_sample(args.config, min(args.cpu_sample_tokens or CPU_SAMPLE_TOKENS, w.T), args.hidden)
            runs = [oracle_step(ws, xs) for _ in range(3)]
            sec = min(runs[1:])                      # the first run warms the page cache and the allocator
            line["cpu_baseline"] = dict({"value": ws.P / sec, "unit": UNIT, "cores": 1, "kind": "oracle",
                                         "sample": cpu_sample_text(ws, f", best of 2 runs after one warm-up, {sec:.2f} s each")},
                                        **host_description())
        print(json.dumps(line))
    if distributed:
        dist.destroy_process_group()


def counters_from_ncu_csv(csv_path, config, command):
    """Turns `ncu -i <report> --page raw --csv` of the index kernels (full token count, tiny rows) into
    profiles/index_kernels_counters.json: warp instructions, shared-memory atomics and their wavefronts,
    kernel time."""
    import csv
    import re
    with open(csv_path) as f:
        rows = list(csv.reader(f))
    hdr = rows[0]
    out = load_json(COUNTERS_JSON)
    entry = out.setdefault(f"config{config}", {})
    want = {"smsp__inst_executed.sum": "warp_instructions", "smsp__thread_inst_executed.sum": "thread_instructions",
            "smsp__inst_executed_op_shared_atom.sum": "shared_atomic_instructions",
            "l1tex__data_pipe_lsu_wavefronts_mem_shared_op_atom.sum": "shared_atomic_wavefronts",
            "l1tex__data_pipe_lsu_wavefronts_mem_shared.sum": "shared_wavefronts",
            "gpu__time_duration.sum": "time_under_ncu", "launch__grid_size": "grid", "launch__block_size": "block",
            "launch__registers_per_thread": "registers", "sm__cycles_active.avg": "sm_cycles_active_avg"}
    for r in rows[2:]:
        d = dict(zip(hdr, r))
        name = re.sub(r"^void ", "", d.get("Kernel Name", "")).split("(")[0]
        short = name.split("<")[0]
        rec = {"kernel": name, "command": command}
        for metric, key in want.items():
            if metric in d and d[metric] not in ("", "nan"):
                rec[key] = float(d[metric])
                if metric == "gpu__time_duration.sum":
                    rec["time_unit"] = rows[1][hdr.index(metric)]
        entry[short] = rec
    with open(COUNTERS_JSON, "w") as f:
        json.dump(out, f, indent=1, sort_keys=True)
        f.write("\n")
    return entry


def summarise(paths):
    """Markdown table of benchmark lines written earlier (one file per config)."""
    rows = []
    for path in paths:
        with open(path) as f:
            d = json.loads(f.read().strip().splitlines()[-1])
        st, ex, tm = d["stages"], d.get("extras") or {}, d["traffic_model"]
        e2e = d.get("e2e") or {}
        rows.append("| {} | {} | {} | {} | {} | {} | {:.3f} | {:.1f} | {} | {:.1f} | {} | {:.1f} % | {:.2f} | {} |".format(
            d["config"]["workload"].split(":")[0].replace("config ", ""),
            *("{:.1f} ({:.1f} %)".format(st[n]["ms"] * 1e3, 100 * st[n]["frac"]) for n in
              ("coact_stats", "assign", "permute_index", "permute_rows", "combine")),
            d["ms_per_step"], d["value"] / 1e6,
            "{:.1f}".format(ex["fused_route_index_us"]) if ex.get("fused_route_index_us") else "-",
            (e2e.get("ms_per_step") or float("nan")), "{:.1f}".format(e2e["value"] / 1e6) if e2e.get("value") else "-",
            100 * (tm["cross_node_reduction"] or 0.0), tm["rank_load_imbalance"] or float("nan"),
            "{:.0f}".format(d["clocks"]["sm_mhz"]) if d.get("clocks") and d["clocks"].get("sm_mhz") else "-"))
    print("| config | coact_stats us (of HBM peak) | assign us | permute_index us | permute_rows us | combine us | step ms | "
          "M pairs/s | fused index pass us | e2e ms | e2e M pairs/s | cross-node reduction | rank-load imbalance | SM MHz |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        print(r)


def main():
    args = parse_args()
    if args.summarise:
        summarise(args.summarise)
        return
    if args.counters_from:
        print(json.dumps(counters_from_ncu_csv(args.counters_from, args.config, args.traffic_command)))
        return
    if args.traffic_from:
        import workloads as W
        w = W.make_config(args.config, T=16)
        tokens = args.tokens or _default_T(args.config)
        print(json.dumps(traffic_from_ncu_csv(args.traffic_from, tokens, w.K, args.hidden or w.H, args.traffic_command)))
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cobalt(args)


if __name__ == "__main__":
    main()
