#!/usr/bin/env python
"""Benchmark of the fused-subgraph executor on B200.

One *step* = one pass of the whole hot path over one batch of synthetic input:
R launches of the fused subgraph kernel, each on its own resident buffer set
(R chosen so that the sets together exceed 4x the L2 capacity, so every launch
reads its inputs from HBM). The R launches are captured once into a CUDA graph
and a step replays it. Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--mode fused|per_mini_subgraph|per_op]
    python bench.py --impl reference ...      # the CPU oracle on the host cores, same metric

Multi-GPU (torchrun): every rank runs an independent replica on its own batch
(weak scaling, no data-path collective); time = max over ranks.
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

DEFAULT_WORKLOAD = "mbv2_56"
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # 148 SMs x 128 FMA lanes x 2 flop x max SM clock
SFU_PEAK_TOPS = 148 * 16 * 1.965e9 / 1e12               # 16 transcendental results / clk / SM
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}     # data-sheet figures, for context only

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (None until a capture exists for that workload and mode).
NCU_TRAFFIC_BYTES = {
    ("mbv2_56", "fused"): 4906752 + 0,            # profiles/mbv2_fused_kernel__mbv2_56.txt (output still dirty in L2)
    ("attn_384", "fused"): 56796672 + 2367232,    # profiles/attention_fused_kernel__attn_384.txt
    ("resnet_56", "fused"): 13343744 + 3328,      # profiles/conv3x3_pair_kernel__resnet_56.txt
    ("ffn_12288", "fused"): 28403712 + 0,         # profiles/ffn_cluster_kernel__ffn_12288.txt (output still dirty in L2)
    ("ffn_512", "fused"): 11877632 + 0,           # profiles/ffn_fused_kernel__ffn_512.txt
    ("pw_dw_56", "fused"): 4894464 + 1280,        # profiles/mbv2_fused_kernel__pw_dw_56.txt
    ("dw_pw_56", "fused"): 28972288 + 256,        # profiles/mbv2_fused_kernel__dw_pw_56.txt
    ("dw_dw_56", "fused"): 28976640 + 1269504,    # profiles/dwdw_fused_kernel__dw_dw_56.txt
    ("pw_pw_56", "fused"): 28948992 + 112384,     # profiles/pwpw_fused_kernel__pw_pw_56.txt
    ("unfold_96", "fused"): 12671232 + 0,         # profiles/pwpw_fused_kernel__unfold_96.txt
}


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


def roofline(wl, peaks, seconds_per_launch, traffic, clocks=None):
    """The roofline that bounds one fused launch: the slowest of HBM (inputs +
    weights + output), tensor cores (dense contractions) and plain ALUs
    (depthwise FMAs). `achieved` / `peak` are in that bound's unit."""
    fl = WL.flops(wl)
    io = WL.io_bytes(wl)
    t_hbm = io / (peaks["hbm_gbs"] * 1e9)
    # tensor peak: the burst measurement, unless the clocks sampled during the timed region show the power cap at
    # work (median SM clock below 90 % of the maximum): then the sustained measurement is the one that applies
    capped = bool(clocks) and clocks.get("sm_mhz", 0) and clocks["sm_mhz"] < 0.9 * clocks.get("sm_max_mhz", 0)
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
    return {
        "bound": bound, "achieved": round(achieved, 3), "peak": round(peak, 3), "unit": unit,
        "frac": round(achieved / peak, 4), "traffic": traffic,
        "peak_source": (("of measured" if peaks["_source"] == "measured" else "of fallback") +
                        (" (sustained bf16 figure: SM clocks were power-capped during the timed region)" if bound == "tensor" and capped else ""))
        if bound != "alu"
        else "derived: 148 SM x 128 lanes x 2 x 1.965 GHz",
        "roofline_us": round(t_roof * 1e6, 3),
        "t_hbm_us": round(t_hbm * 1e6, 3), "t_tensor_us": round(t_tensor * 1e6, 3), "t_alu_us": round(t_alu * 1e6, 3),
        "t_sfu_us": round(fl["sfu"] / (SFU_PEAK_TOPS * 1e12) * 1e6, 3),
        "algorithmic_bytes": io, "algorithmic_tensor_flops": fl["tensor"], "algorithmic_alu_flops": fl["cuda"],
        "frac_of_whole_roofline": round(t_roof / seconds_per_launch, 4),
        # the same roofline against the data-sheet peaks (8 TB/s, 2250 TFLOP/s bf16), for context
        "frac_of_nominal_roofline": round(max(io / (NOMINAL_PEAKS["hbm_gbs"] * 1e9), fl["tensor"] / (NOMINAL_PEAKS["bf16_tflops"] * 1e12),
                                              t_alu) / seconds_per_launch, 4),
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


def cpu_baseline(wl, name, budget_s=12.0):
    """The oracle as it stands, timed on this host's cores on a bounded sample:
    whole launches' worth of samples (or fewer when one launch takes longer than
    the budget), repeated until about `budget_s` seconds of CPU work are done."""
    from oracle import oracle
    per = WL.get(name, batch=1)
    d = WL.generate(per)
    t0 = time.perf_counter()
    oracle.run_chain(per.ops, d["inputs"], d["weights"])
    t1 = time.perf_counter() - t0
    n = max(1, min(wl.samples, int(budget_s / max(t1, 1e-4))))
    big = WL.get(name, batch=n)
    d = WL.generate(big)
    calls, t0 = 0, time.perf_counter()
    while True:
        oracle.run_chain(big.ops, d["inputs"], d["weights"])
        calls += 1
        t = time.perf_counter() - t0
        if t >= budget_s or calls >= 10000:
            break
    return {"value": n * calls / t, "unit": "samples/s", "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{calls} oracle.run_chain call(s) on {n} of the {wl.samples} samples of one {name} launch, {t:.2f} s wall"}


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle
    wl = WL.get(args.workload)
    t_probe = time.perf_counter()
    per = WL.get(args.workload, batch=1)
    d = WL.generate(per)
    oracle.run_chain(per.ops, d["inputs"], d["weights"])
    t_probe = time.perf_counter() - t_probe
    steps, warm = max(1, min(args.steps, 5)), max(0, min(args.warmup, 1))
    n = max(1, min(wl.samples, int(120.0 / (steps + warm) / max(t_probe, 1e-3))))
    big = WL.get(args.workload, batch=n)
    d = WL.generate(big)
    for _ in range(warm):
        oracle.run_chain(big.ops, d["inputs"], d["weights"])
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.run_chain(big.ops, d["inputs"], d["weights"])
    t = (time.perf_counter() - t0) / steps
    v = n / t
    sample = f"{n} of {wl.samples} samples of {args.workload} per step (bounded sample), {steps} steps"
    print(json.dumps({
        "impl": "reference", "metric": "fused-subgraph samples/s", "value": v, "unit": "samples/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": warm, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "samples_per_step": n},
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
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=WL.ALL)
    ap.add_argument("--mode", default="fused", choices=["fused", "per_mini_subgraph", "per_op"])
    ap.add_argument("--no-graph", action="store_true", help="launch directly instead of replaying a CUDA graph")
    ap.add_argument("--sets", type=int, default=0, help="rotating buffer sets per step (0 = enough to exceed 4x L2)")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-unfused", action="store_true")
    ap.add_argument("--headline-only", action="store_true", help="skip the summary of the other configurations")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    if args.impl == "reference":
        run_reference(args)
        return

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
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    stream = torch.cuda.Stream(dev)

    def timed(step_fn, steps, warmup, sampler=None):
        with torch.cuda.stream(stream):
            for _ in range(warmup):
                step_fn()
            stream.synchronize()
            if dist is not None:
                dist.barrier()
            torch.cuda.synchronize()
            if sampler is not None:
                sampler.start()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(steps):
                step_fn()
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
        return ms / steps

    def measure(name, mode, steps, warmup, with_e2e, unfused_modes, sampler=None):
        """Time one workload: fused (or `mode`) step, optional end-to-end and unfused modes, same buffers."""
        wl = WL.get(name)
        io = WL.io_bytes(wl)

        def make_handle(m):
            h = B.Subgraph(wl.ops, wl.input_shapes, mode=m)
            h.ensure_workspace(dev)
            return h

        sg = make_handle(mode)
        per_set = io + sg.workspace_bytes
        nsets = args.sets or max(2, int(np.ceil(4.0 * l2 / per_set)))
        # Resident buffer sets: set r holds its own inputs, weights and output (seeded, one draw per set).
        sets = []
        for r in range(nsets):
            d = WL.generate(wl, list(wl.seed_seq) + [1000 + r + 10000 * rank])
            ins = [torch.from_numpy(a).to(dev, torch.bfloat16) for a in d["inputs"]]
            ws = [torch.from_numpy(a).to(dev, torch.float32 if k == "bias" else torch.bfloat16)
                  for a, k in zip(d["weights"], wl.weight_kinds)]
            sets.append((ins, ws, sg.empty_output(dev)))

        def one_pass(handle):
            for ins, ws, out in sets:
                handle.run(ins, ws, out=out, stream=stream.cuda_stream)

        def build_step(handle):
            with torch.cuda.stream(stream):
                one_pass(handle)                    # first run: status word, attributes, tensor maps
            stream.synchronize()
            if args.no_graph:
                return lambda: one_pass(handle)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                one_pass(handle)
            return g.replay

        step = build_step(sg)
        ms_step = timed(step, steps, warmup, sampler)
        clocks = sampler.finish() if sampler is not None else None
        context = {}
        if with_e2e:
            # context figures of the headline workload, none of them the reported value: five more repetitions
            # (median / best), the same launches on ONE buffer set (inputs hot in L2), and the floor of an empty
            # kernel launched the same way (same grid, block and shared memory, same CUDA-graph replay)
            reps = sorted(timed(step, max(3, steps // 5), 1) * 1e3 / nsets for _ in range(5))
            context["repeats_us_per_launch"] = {"median": round(reps[2], 3), "best": round(reps[0], 3), "n": 5}
            ins0, ws0, out0 = sets[0]

            def hot_pass():
                for _ in range(nsets):
                    sg.run(ins0, ws0, out=out0, stream=stream.cuda_stream)

            def graph_of(fn):
                with torch.cuda.stream(stream):
                    fn()
                stream.synchronize()
                if args.no_graph:
                    return fn
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    fn()
                return g.replay

            context["hot_l2_us_per_launch"] = round(timed(graph_of(hot_pass), max(3, steps // 5), 3) * 1e3 / nsets, 3)
            # the same launches dealt alternately to two streams: independent batches overlap, so the SMs one grid
            # leaves idle (and its tail) are taken by the next grid -- throughput of concurrent requests, not the
            # latency of one
            side = torch.cuda.Stream(dev)

            def two_stream_pass():
                side.wait_stream(stream)
                for r, (ins, ws, out) in enumerate(sets):
                    sg.run(ins, ws, out=out, stream=(stream if r % 2 == 0 else side).cuda_stream)
                stream.wait_stream(side)

            context["two_streams_us_per_launch"] = round(timed(graph_of(two_stream_pass), max(3, steps // 5), 3) * 1e3 / nsets, 3)
            grid = max(1, int(sg.query(B.AGO_Q_NUM_LAUNCHES)))
            smem = int(sg.query(B.AGO_Q_SMEM_BYTES)) if mode == "fused" else 0

            def empty_pass():
                for _ in range(nsets * grid):
                    B.ago_launch_empty(128, 1024, smem, stream.cuda_stream)

            context["empty_kernel_us_per_launch"] = round(timed(graph_of(empty_pass), max(3, steps // 5), 3) * 1e3 / (nsets * grid), 3)
        assert sg.status() == B.AGO_OK, B.ago_last_error()
        res = {"wl": wl, "nsets": nsets, "per_set": per_set, "ms_step": ms_step, "clocks": clocks,
               "launches_per_pass": sg.query(B.AGO_Q_NUM_LAUNCHES),
               "sec_per_launch": ms_step * 1e-3 / nsets,
               "value": wl.samples * nsets * world / (ms_step * 1e-3),
               "tile_rows": sg.query(B.AGO_Q_TILE_ROWS), "smem_bytes": sg.query(B.AGO_Q_SMEM_BYTES), "context": context}

        if with_e2e:
            # end to end: pinned host buffers, H2D + run + D2H inside the timed region
            kStreams = 4
            h_in = [[t.cpu().pin_memory() for t in ins] for ins, _, _ in sets[:kStreams]]
            h_out = [torch.empty(wl.output_shape, dtype=torch.bfloat16).pin_memory() for _ in range(len(h_in))]
            e2e_sets = min(nsets, 8)

            # Calls rotate over a few streams (each with its own pinned buffers), so the host->device copy of one
            # call overlaps the kernel and the device->host copy of earlier ones (the link is full duplex); the
            # extra streams are fenced into the timed stream at both ends of a pass.
            extra = [torch.cuda.Stream(dev) for _ in range(len(h_in) - 1)]
            lanes = [stream] + extra

            def e2e_pass():
                ev = torch.cuda.Event()
                ev.record(stream)
                for s in extra:
                    s.wait_event(ev)
                for r in range(e2e_sets):
                    ins, ws, out = sets[r]
                    k = r % len(lanes)
                    sg.run_host(h_in[k], ws, h_out[k], ins, out, stream=lanes[k].cuda_stream)
                for s in extra:
                    ev2 = torch.cuda.Event()
                    ev2.record(s)
                    stream.wait_event(ev2)

            ms_e2e = timed(e2e_pass, max(3, min(steps, 10)), 3)
            in_bytes = sum(2 * int(np.prod(sh)) for sh in wl.input_shapes)
            out_bytes = 2 * int(np.prod(wl.output_shape))
            res["e2e"] = {"value": wl.samples * e2e_sets * world / (ms_e2e * 1e-3), "unit": "samples/s",
                          "h2d_bytes_per_step": in_bytes * e2e_sets, "d2h_bytes_per_step": out_bytes * e2e_sets,
                          "launches_per_step": e2e_sets, "streams": len(lanes)}

        # the unfused modes of the same library, same buffers (context for the fusion speedup)
        unfused = {}
        for m in unfused_modes:
            try:
                h2 = make_handle(m)
                st2 = build_step(h2)
                ms2 = timed(st2, max(3, steps // 5), 3)
                unfused[m] = {"value": wl.samples * nsets * world / (ms2 * 1e-3), "unit": "samples/s",
                              "us_per_launch_set": ms2 * 1e3 / nsets, "kernels_per_pass": h2.query(B.AGO_Q_NUM_LAUNCHES)}
                h2.close()
            except B.AgoError as e:
                unfused[m] = {"error": str(e)}
        for m in unfused_modes:
            if "value" in unfused.get(m, {}):
                unfused["speedup_vs_" + m] = round(res["value"] / unfused[m]["value"], 3)
        res["unfused"] = unfused
        sg.close()
        del sets
        torch.cuda.empty_cache()
        return res

    sampler = ClockSampler(local)
    head_unfused = [] if (args.skip_unfused or args.mode != "fused") else ["per_mini_subgraph", "per_op"]
    head = measure(args.workload, args.mode, args.steps, args.warmup, True, head_unfused, sampler)
    wl, nsets, per_set, ms_step = head["wl"], head["nsets"], head["per_set"], head["ms_step"]
    clocks, launches_per_pass, sec_per_launch, value = head["clocks"], head["launches_per_pass"], head["sec_per_launch"], head["value"]
    e2e, unfused = head["e2e"], head["unfused"]

    # the other benchmark configurations, fused, against their own rooflines and per-mini-subgraph chains
    others = {}
    if not args.headline_only and world == 1 and args.mode == "fused":
        for name in WL.ALL:
            if name == args.workload:
                continue
            r = measure(name, "fused", max(3, min(args.steps, 10)), 3, False,
                        [] if args.skip_unfused else ["per_mini_subgraph"])
            rf = roofline(r["wl"], peaks, r["sec_per_launch"], NCU_TRAFFIC_BYTES.get((name, "fused")))
            others[name] = {"value": r["value"], "unit": "samples/s", "us_per_launch": round(r["sec_per_launch"] * 1e6, 3),
                            "roofline_bound": rf["bound"], "roofline_us": rf["roofline_us"],
                            "roofline_frac": rf["frac_of_whole_roofline"],
                            "speedup_vs_per_mini_subgraph": r["unfused"].get("speedup_vs_per_mini_subgraph"),
                            "tile_rows": r["tile_rows"]}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    line = {
        "metric": "fused-subgraph samples/s", "value": value, "unit": "samples/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": args.workload, "mode": args.mode, "samples_per_launch": wl.samples,
            "launches_per_step": nsets * launches_per_pass, "buffer_sets": nsets,
            "l2_policy": f"inputs larger than L2: {nsets} rotating buffer sets x {per_set / 1e6:.2f} MB >= 4 x L2 ({l2 / 1e6:.0f} MB)",
            "cuda_graph": not args.no_graph, "parallelism": f"replicas x{world}",
            "us_per_launch": round(sec_per_launch * 1e6, 3),
        },
        "roofline": roofline(wl, peaks, sec_per_launch, NCU_TRAFFIC_BYTES.get((args.workload, args.mode)), clocks),
        "e2e": e2e, "gpu_launches": args.steps * nsets * launches_per_pass, "clocks": clocks,
        "unfused": unfused,
        "context": head["context"],
        "other_workloads": others,
    }
    if not args.skip_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl, args.workload)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
