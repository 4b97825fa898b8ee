#!/usr/bin/env python
"""Benchmark of the fused-subgraph executor on B200.

One *step* = one pass of the whole hot path over one batch of synthetic input: for every chain of the workload, R
launches of the fused subgraph kernel, each on its own resident buffer set (R chosen so that the sets together
exceed 4x the L2 capacity, so every launch reads its inputs from HBM). The launches of a chain are captured once
into a CUDA graph; a step replays the graphs in order, with a CUDA event between chains, so the per-kernel launch
durations behind `roofline` are measured inside the timed region.

The default workload is the largest configuration, `bert_layer_384`: the attention chain (`attn_384`) and then the
feed-forward chain (`ffn_12288`) on the same 32 sequences of 384 tokens. `--workload NAME` times one chain alone.
Prints ONE JSON line (rank 0); `workloads` in it holds the full record of every other configuration.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--mode fused|per_mini_subgraph|per_op|auto]
    python bench.py --impl reference ...      # the CPU oracle on the host cores, same metric

Multi-GPU (torchrun): every rank runs an independent replica on its own batch (weak scaling, no data-path
collective); time = max over ranks.
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

from paper_2212_01005_b200 import workloads as WL  # noqa: E402

# config 4 of the benchmark definition: both chains of a BERT-base encoder layer on the same 32 x 384 tokens
COMPOSITES = {"bert_layer_384": ["attn_384", "ffn_12288"]}
DEFAULT_WORKLOAD = "bert_layer_384"
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # 148 SMs x 128 FMA lanes x 2 flop x max SM clock
SFU_PEAK_TOPS = 148 * 16 * 1.965e9 / 1e12               # 16 transcendental results / clk / SM
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}     # data-sheet figures, for context only


def parts_of(name):
    return COMPOSITES.get(name, [name])


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


def load_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of each kernel, from the ncu captures summarised
    under profiles/ (a profiler figure: it cannot be measured inside a timed run)."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    table = {}
    if os.path.exists(path):
        with open(path) as f:
            for ln in f:
                col = ln.split()
                if len(col) >= 3 and not ln.startswith("#"):
                    table[col[0]] = {"bytes": int(col[1]), "source": col[2]}
    return table


def roofline(wl, peaks, seconds_per_launch, traffic, clocks=None, extra_bytes=0):
    """The roofline that bounds one launch set of `wl`: the slowest of HBM (inputs + weights + output, plus
    `extra_bytes` of intermediates for an unfused chain), tensor cores (dense contractions) and plain ALUs
    (depthwise FMAs). `achieved` / `peak` are in that bound's unit."""
    fl = WL.flops(wl)
    io = WL.io_bytes(wl) + extra_bytes
    t_hbm = io / (peaks["hbm_gbs"] * 1e9)
    # tensor peak: the burst measurement, unless the clocks sampled during the timed region show the power cap at
    # work (median SM clock below 90 % of the maximum): then the sustained measurement is the one that applies
    capped = bool(clocks) and clocks.get("sm_mhz") and clocks["sm_mhz"] < 0.9 * (clocks.get("sm_max_mhz") or 0)
    tensor_peak = (peaks.get("bf16_tflops_sustained") if capped else None) or peaks["bf16_tflops"]
    t_tensor = fl["tensor"] / (tensor_peak * 1e12)
    t_alu = fl["cuda"] / (FP32_PEAK_TFLOPS * 1e12)
    bound = max((t_hbm, "hbm"), (t_tensor, "tensor"), (t_alu, "alu"))[1]
    if bound == "hbm":
        achieved, peak, unit = io / seconds_per_launch / 1e9, peaks["hbm_gbs"], "GB/s"
    elif bound == "tensor":
        achieved, peak, unit = fl["tensor"] / seconds_per_launch / 1e12, tensor_peak, "TFLOP/s"
    else:
        achieved, peak, unit = fl["cuda"] / seconds_per_launch / 1e12, FP32_PEAK_TFLOPS, "TFLOP/s"
    t_roof = max(t_hbm, t_tensor, t_alu)
    src = "of measured" if peaks["_source"] == "measured" else "of fallback"
    if bound == "tensor" and capped:
        src += " (sustained bf16 figure: SM clocks were power-capped during the timed region)"
    if bound == "alu":
        src = "derived: 148 SM x 128 lanes x 2 x 1.965 GHz"
    t_nominal = max(io / (NOMINAL_PEAKS["hbm_gbs"] * 1e9), fl["tensor"] / (NOMINAL_PEAKS["bf16_tflops"] * 1e12), t_alu)
    return {
        "bound": bound, "achieved": round(achieved, 3), "peak": round(peak, 3), "unit": unit,
        "frac": round(achieved / peak, 4), "traffic": traffic, "peak_source": src,
        "us_per_launch": round(seconds_per_launch * 1e6, 3), "roofline_us": round(t_roof * 1e6, 3),
        "t_hbm_us": round(t_hbm * 1e6, 3), "t_tensor_us": round(t_tensor * 1e6, 3), "t_alu_us": round(t_alu * 1e6, 3),
        "t_sfu_us": round(fl["sfu"] / (SFU_PEAK_TOPS * 1e12) * 1e6, 3),
        "algorithmic_bytes": io, "algorithmic_tensor_flops": fl["tensor"], "algorithmic_alu_flops": fl["cuda"],
        "frac_of_nominal_roofline": round(t_nominal / seconds_per_launch, 4),
    }


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception as e:  # NVML missing: report that, never guess
            self.err = repr(e)

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._halt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def finish(self):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2)
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "note": "NVML unavailable"}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_pass(parts, data):
    from oracle import oracle
    for wl, d in zip(parts, data):
        oracle.run_chain(wl.ops, d["inputs"], d["weights"])


def cpu_baseline(name, budget_s):
    """The oracle as it stands, timed on this host's cores on a bounded sample of the workload: n of the samples
    of one launch set (all chains of the workload), repeated until about `budget_s` seconds of CPU work are done."""
    from oracle import oracle
    names = parts_of(name)
    full = [WL.get(n) for n in names]
    one = [WL.get(n, batch=1) for n in names]
    d1 = [WL.generate(w) for w in one]
    t0 = time.perf_counter()
    oracle_pass(one, d1)
    t1 = time.perf_counter() - t0
    n = max(1, min(full[0].samples, int(budget_s / max(t1, 1e-4))))
    big = [WL.get(nm, batch=n) for nm in names]
    d = [WL.generate(w) for w in big]
    calls, t0 = 0, time.perf_counter()
    while True:
        oracle_pass(big, d)
        calls += 1
        t = time.perf_counter() - t0
        if t >= budget_s or calls >= 10000:
            break
    return {"value": n * calls / t, "unit": "samples/s", "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{calls} pass(es) of the oracle over {n} of the {full[0].samples} samples of one {name} launch set, {t:.2f} s wall"}


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the host cores; --steps / --warmup are honoured, each
    step a bounded sample of the workload sized so that the whole run ends within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle
    names = parts_of(args.workload)
    full = [WL.get(n) for n in names]
    one = [WL.get(n, batch=1) for n in names]
    d1 = [WL.generate(w) for w in one]
    t_probe = time.perf_counter()
    oracle_pass(one, d1)
    t_probe = time.perf_counter() - t_probe
    steps, warm = max(1, args.steps), max(0, args.warmup)
    n = max(1, min(full[0].samples, int(150.0 / (steps + warm) / max(t_probe, 1e-3))))
    big = [WL.get(nm, batch=n) for nm in names]
    d = [WL.generate(w) for w in big]
    for _ in range(warm):
        oracle_pass(big, d)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_pass(big, d)
    t = (time.perf_counter() - t0) / steps
    v = n / t
    sample = f"{n} of {full[0].samples} samples of {args.workload} per step (bounded sample), {steps} steps after {warm} warm-up"
    print(json.dumps({
        "impl": "reference", "metric": "fused-subgraph samples/s", "value": v, "unit": "samples/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": warm, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "chains": names, "samples_per_step": n},
        "cpu_baseline": {"value": v, "unit": "samples/s", "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(COMPOSITES) + list(WL.ALL))
    ap.add_argument("--mode", default="fused", choices=["fused", "per_mini_subgraph", "per_op", "auto"])
    ap.add_argument("--no-graph", action="store_true", help="launch directly instead of replaying CUDA graphs")
    ap.add_argument("--sets", type=int, default=0, help="rotating buffer sets per step (0 = enough to exceed 4x L2)")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-unfused", action="store_true")
    ap.add_argument("--headline-only", action="store_true", help="skip the records of the other configurations")
    args = ap.parse_args()

    if args.impl == "reference":
        run_reference(args)
        return
    args.warmup = max(args.warmup, 3)

    import torch
    from paper_2212_01005_b200 import binding as B

    B.load()                                    # fails loudly when the CUDA library is missing
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the executor has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    peaks = load_peaks()
    traffic = load_traffic()
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    stream = torch.cuda.Stream(dev)
    mode_names = {B.AGO_MODE_FUSED: "fused", B.AGO_MODE_PER_MINI_SUBGRAPH: "per_mini_subgraph", B.AGO_MODE_PER_OP: "per_op"}

    def timed(step_fn, steps, warmup, sampler=None):
        """K steps between two events on the launching stream, barrier + synchronize on both sides, max over ranks."""
        with torch.cuda.stream(stream):
            for _ in range(warmup):
                step_fn(None)
            stream.synchronize()
            if dist is not None:
                dist.barrier()
            torch.cuda.synchronize()
            if sampler is not None:
                sampler.start()
            marks = []
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(steps):
                step_fn(marks)
            e1.record(stream)
            stream.synchronize()
            torch.cuda.synchronize()
            if dist is not None:
                dist.barrier()
        ms = e0.elapsed_time(e1)
        if dist is not None:
            t = torch.tensor([ms], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        # per-chain time inside the timed region: events recorded around each chain's launches in every step
        per_part = None
        if marks:
            per_part = [0.0] * (len(marks[0]) - 1)
            for ev in marks:
                for i in range(len(ev) - 1):
                    per_part[i] += ev[i].elapsed_time(ev[i + 1])
            per_part = [x / steps for x in per_part]
        return ms / steps, per_part

    class Bench:
        """Handles, resident buffer sets and launch graphs of one workload (one or more chains) in one mode."""

        def __init__(self, name, mode):
            self.name, self.mode = name, mode
            self.wls = [WL.get(n) for n in parts_of(name)]
            self.sgs = []
            for wl in self.wls:
                h = B.Subgraph(wl.ops, wl.input_shapes, mode=mode)
                h.ensure_workspace(dev)
                self.sgs.append(h)
            self.per_set = sum(WL.io_bytes(wl) + sg.workspace_bytes for wl, sg in zip(self.wls, self.sgs))
            self.nsets = args.sets or max(2, int(np.ceil(4.0 * l2 / self.per_set)))
            # resident buffer sets: set r holds its own inputs, weights and output of every chain (seeded, one draw per set)
            self.sets = []
            for r in range(self.nsets):
                per_chain = []
                for wl, sg in zip(self.wls, self.sgs):
                    d = WL.generate(wl, list(wl.seed_seq) + [1000 + r + 10000 * rank])
                    ins = [torch.from_numpy(a).to(dev, torch.bfloat16) for a in d["inputs"]]
                    ws = [torch.from_numpy(a).to(dev, torch.float32 if k == "bias" else torch.bfloat16)
                          for a, k in zip(d["weights"], wl.weight_kinds)]
                    per_chain.append((ins, ws, sg.empty_output(dev)))
                self.sets.append(per_chain)
            self.launches = [int(sg.query(B.AGO_Q_NUM_LAUNCHES)) for sg in self.sgs]
            self.effective = [mode_names[int(sg.query(B.AGO_Q_MODE))] for sg in self.sgs]
            self.graphs = [self._graph_of(lambda c=c: self.chain_pass(c)) for c in range(len(self.wls))]

        def chain_pass(self, c, one_set=None):
            for r in range(self.nsets):
                ins, ws, out = self.sets[r if one_set is None else one_set][c]
                self.sgs[c].run(ins, ws, out=out, stream=stream.cuda_stream)

        def _graph_of(self, fn):
            with torch.cuda.stream(stream):
                fn()                                # first run: status block, attributes, tensor maps
            stream.synchronize()
            if args.no_graph:
                return fn
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                fn()
            return g.replay

        def step(self, marks):
            ev = None
            if marks is not None:
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(len(self.graphs) + 1)]
                ev[0].record(stream)
            for i, g in enumerate(self.graphs):
                g()
                if ev is not None:
                    ev[i + 1].record(stream)
            if marks is not None:
                marks.append(ev)

        def status_ok(self):
            for sg in self.sgs:
                assert sg.status() == B.AGO_OK, B.ago_last_error()

        def close(self):
            for sg in self.sgs:
                sg.close()
            self.sets = None
            torch.cuda.empty_cache()

    def run_mode(name, mode, steps, warmup, sampler=None):
        """Time one workload in one mode; returns the record shared by the headline and the per-configuration entries."""
        b = Bench(name, mode)
        ms_step, per_part = timed(b.step, steps, warmup, sampler)
        clocks = sampler.finish() if sampler is not None else None
        b.status_ok()
        chains = []
        for c, wl in enumerate(b.wls):
            sec = per_part[c] * 1e-3 / b.nsets
            eff = b.effective[c]
            inter = int(b.sgs[c].query(B.AGO_Q_INTERMEDIATE_BYTES)) if eff != "fused" else 0
            key = f"{wl.name}/{eff}"
            rf = roofline(wl, peaks, sec, traffic.get(key, {}).get("bytes"), clocks, extra_bytes=inter)
            if key in traffic:
                rf["traffic_source"] = traffic[key]["source"]
            ws_traffic = int(b.sgs[c].query(B.AGO_Q_WORKSPACE_TRAFFIC))
            if ws_traffic:
                # partial sums a split-reduction kernel adds into and reads back from device memory (through L2): real
                # traffic that the roofline's algorithmic bytes (inputs + weights + output) do not contain
                rf["workspace_traffic_bytes"] = ws_traffic
            chains.append({"chain": wl.name, "mode": eff, "us_per_launch_set": round(sec * 1e6, 3), "kernels_per_launch_set": b.launches[c],
                           "tile_rows": int(b.sgs[c].query(B.AGO_Q_TILE_ROWS)), "smem_bytes": int(b.sgs[c].query(B.AGO_Q_SMEM_BYTES)),
                           "roofline": rf})
        rec = {"value": b.wls[0].samples * b.nsets * world / (ms_step * 1e-3), "unit": "samples/s", "ms_per_step": ms_step,
               "us_per_launch_set": round(ms_step * 1e3 / b.nsets, 3), "chains": chains, "clocks": clocks,
               "buffer_sets": b.nsets, "bytes_per_set": b.per_set, "launches_per_step": b.nsets * sum(b.launches)}
        return b, rec

    def e2e_of(b, steps):
        """End to end through the C-ABI with HOST buffers: every launch set copies its inputs from pinned host memory,
        runs, and copies its output back, inside the timed region. Calls rotate over a few streams (each with its own
        pinned buffers), so the copy in of one call overlaps the kernel and the copy out of earlier ones."""
        k_streams = 4
        n_e2e = min(b.nsets, 8)
        h_in = [[[t.cpu().pin_memory() for t in b.sets[k][c][0]] for c in range(len(b.wls))] for k in range(min(k_streams, b.nsets))]
        h_out = [[torch.empty(wl.output_shape, dtype=torch.bfloat16).pin_memory() for wl in b.wls] for _ in range(len(h_in))]
        extra = [torch.cuda.Stream(dev) for _ in range(len(h_in) - 1)]
        lanes = [stream] + extra

        def e2e_pass(_marks):
            ev = torch.cuda.Event()
            ev.record(stream)
            for s in extra:
                s.wait_event(ev)
            for r in range(n_e2e):
                k = r % len(lanes)
                for c in range(len(b.wls)):
                    ins, ws, out = b.sets[r][c]
                    b.sgs[c].run_host(h_in[k][c], ws, h_out[k][c], ins, out, stream=lanes[k].cuda_stream)
            for s in extra:
                ev2 = torch.cuda.Event()
                ev2.record(s)
                stream.wait_event(ev2)

        ms, _ = timed(e2e_pass, max(3, min(steps, 10)), 3)
        in_bytes = sum(2 * int(np.prod(sh)) for wl in b.wls for sh in wl.input_shapes)
        out_bytes = sum(2 * int(np.prod(wl.output_shape)) for wl in b.wls)
        return {"value": b.wls[0].samples * n_e2e * world / (ms * 1e-3), "unit": "samples/s",
                "h2d_bytes_per_step": in_bytes * n_e2e, "d2h_bytes_per_step": out_bytes * n_e2e,
                "launch_sets_per_step": n_e2e, "streams": len(lanes)}

    def record_of(name, steps, warmup, headline):
        """The full record of one configuration: fused run (clocks sampled during its timed region), end to end,
        the per-mini-subgraph chain of the same library with ITS roofline, and what AGO_MODE_AUTO picks."""
        sampler = ClockSampler(local)
        b, rec = run_mode(name, args.mode if headline else "fused", steps, warmup, sampler)
        rec["e2e"] = e2e_of(b, steps)
        if headline:
            # context, none of it the reported value: five more repetitions, one buffer set (inputs hot in L2), the same
            # launches dealt alternately to two streams, and the floor of an empty kernel launched the same way
            ctx = {}
            reps = sorted(timed(b.step, max(3, steps // 5), 1)[0] * 1e3 / b.nsets for _ in range(5))
            ctx["repeats_us_per_launch_set"] = {"median": round(reps[2], 3), "best": round(reps[0], 3), "n": 5}
            hot = b._graph_of(lambda: [b.chain_pass(c, one_set=0) for c in range(len(b.wls))])
            ctx["hot_l2_us_per_launch_set"] = round(timed(lambda m: hot(), max(3, steps // 5), 3)[0] * 1e3 / b.nsets, 3)
            n_launch = b.nsets * sum(b.launches)
            empty = b._graph_of(lambda: [B.ago_launch_empty(128, 1024, 0, stream.cuda_stream) for _ in range(n_launch)])
            ctx["empty_kernel_us_per_launch"] = round(timed(lambda m: empty(), max(3, steps // 5), 3)[0] * 1e3 / n_launch, 3)
            rec["context"] = ctx
        b.close()
        if not args.skip_unfused and (not headline or args.mode == "fused"):
            try:
                b2, r2 = run_mode(name, "per_mini_subgraph", max(3, steps // 5), 3)
                b2.close()
                rec["per_mini_subgraph"] = {"value": r2["value"], "unit": "samples/s", "us_per_launch_set": r2["us_per_launch_set"],
                                            "chains": r2["chains"]}
                rec["fused_speedup_vs_per_mini_subgraph"] = round(rec["value"] / r2["value"], 3)
            except B.AgoError as e:
                rec["per_mini_subgraph"] = {"error": str(e)}
            picks = []
            for wl in [WL.get(n) for n in parts_of(name)]:
                h = B.Subgraph(wl.ops, wl.input_shapes, mode="auto")
                picks.append(mode_names[int(h.query(B.AGO_Q_MODE))])
                h.close()
            rec["auto_mode_picks"] = picks
        if not args.skip_cpu_baseline and rank == 0:
            rec["cpu_baseline"] = cpu_baseline(name, 12.0 if headline else 3.0)
        return rec

    head = record_of(args.workload, args.steps, args.warmup, True)

    # the other configurations, each with its full record (fewer steps; same timing method)
    others = {}
    if not args.headline_only and world == 1 and args.mode == "fused":
        done = set(parts_of(args.workload)) | {args.workload}
        for name in WL.ALL:
            if name in done:
                continue
            others[name] = record_of(name, max(3, min(args.steps, 10)), 3, False)
        for name in parts_of(args.workload):      # the chains of a composite headline also appear on their own
            if name != args.workload:
                others[name] = record_of(name, max(3, min(args.steps, 10)), 3, False)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    dominant = max(head["chains"], key=lambda c: c["us_per_launch_set"])
    line = {
        "metric": "fused-subgraph samples/s", "value": head["value"], "unit": "samples/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": args.workload, "chains": parts_of(args.workload), "mode": args.mode,
            "samples_per_launch_set": WL.get(parts_of(args.workload)[0]).samples,
            "launches_per_step": head["launches_per_step"], "buffer_sets": head["buffer_sets"],
            "l2_policy": f"inputs larger than L2: {head['buffer_sets']} rotating buffer sets x {head['bytes_per_set'] / 1e6:.2f} MB >= 4 x L2 ({l2 / 1e6:.0f} MB)",
            "cuda_graph": not args.no_graph, "parallelism": f"replicas x{world}",
            "us_per_launch_set": head["us_per_launch_set"],
        },
        # the dominant kernel of the step (the chain with the longest launches); every chain's roofline is in `chains`
        "roofline": dict(dominant["roofline"], kernel_of=dominant["chain"]),
        "chains": head["chains"],
        "e2e": head["e2e"], "gpu_launches": args.steps * head["launches_per_step"], "clocks": head["clocks"],
        "context": head.get("context", {}),
    }
    for k in ("per_mini_subgraph", "fused_speedup_vs_per_mini_subgraph", "auto_mode_picks", "cpu_baseline"):
        if k in head:
            line[k] = head[k]
    line["workloads"] = others
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
