#!/usr/bin/env python
"""Benchmark of the EoRA compensated linear layer on B200.

Default workload (one "step" = one decoded token through the linear layers of a LLaMA3-8B-shaped
model): 32 blocks x 7 layers (q, k, v, o, gate, up, down), 3-bit asymmetric group-128 backbone,
fp16 rank-128 EoRA adapter, X fp16 with M = 1 -- 224 fused-layer launches on distinct weights
(3.4 GB, far larger than L2, so every launch streams from HBM).  Reports tokens/s (linear layers
only: no attention, norms or sampling), the achieved HBM bandwidth on algorithmic bytes against
the measured copy bandwidth, an end-to-end number through the host-buffer entry point, the
tensor-core prefill throughput at M = 2048 as an extra, and the CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import eora_inputs as gen  # noqa: E402
from paper_2410_21271_b200 import traffic  # noqa: E402

METRIC = "decode tokens/s, LLaMA3-8B linear layers (224 EoRA-compensated layers per token), M=1"
UNIT = "tokens/s"
WORKLOAD = "llama3-8b-layer-set/w3-g128/eora-fp16-r128/M1"
W_FMT, AB_FMT, RANK, M_DECODE = "q3", "f16", 128, 1
LAYERS = list(gen.LLAMA3_8B_SHAPES.items())
NOMINAL_HBM_GBS = 8000.0


def measured_peaks() -> tuple[dict, str]:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return json.load(open(p)), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


# Layers of a block that read the same activations are fused into one launch (q|k|v and gate|up).
FUSE_GROUPS = (("q", "k", "v"), ("o",), ("gate", "up"), ("down",))


def step_bytes(blocks: int, fused: bool = True) -> int:
    """Algorithmic bytes of a step; a fused group reads its X once."""
    shapes = dict(LAYERS)
    per_block = sum(traffic.forward_bytes(W_FMT, AB_FMT, K, N, RANK, M_DECODE) for _, (K, N) in LAYERS)
    if fused:
        per_block -= sum((len(g) - 1) * 2 * M_DECODE * shapes[g[0]][0] for g in FUSE_GROUPS)
    return blocks * per_block


# --------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self) -> dict:
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------------------------
def build_layer_set(blocks: int, device: str, seed0: int = 1000, fused: bool = True):
    """blocks x 7 layers with distinct seeded weights as launch units (names, K, Ns, object): with `fused` the
    layers of a block that share their input sit behind one handle (one launch), otherwise every layer has
    its own.  Returns (units, x buffers, y buffers)."""
    import torch
    import paper_2410_21271_b200 as eora
    shapes = dict(LAYERS)
    index = {name: li for li, (name, _) in enumerate(LAYERS)}
    groups = FUSE_GROUPS if fused else tuple((name,) for name, _ in LAYERS)
    units = []
    for b in range(blocks):
        for names in groups:
            parts = []
            for name in names:
                K, N = shapes[name]
                seed = seed0 + 16 * b + index[name]
                wf = gen.make_backbone_quant(seed, K, N, 3 if W_FMT == "q3" else 4, 128)
                af, bf = gen.make_ab_f16(seed, K, N, RANK)
                parts.append((wf, af, bf))
            K = shapes[names[0]][0]
            Ns = tuple(shapes[n][1] for n in names)
            if len(names) == 1:
                obj = eora.Layer(*parts[0], max_m=M_DECODE, device=device)
            else:
                obj = eora.FusedLayers(parts, max_m=M_DECODE, device=device)
            units.append((names, K, Ns, obj))
    xs, ys = {}, {}
    for name, (K, N) in LAYERS:
        xs[name] = torch.from_numpy(gen.make_x(7, M_DECODE, K)).to(device)
        ys[name] = torch.empty((M_DECODE, N), dtype=torch.float16, device=device)
    return units, xs, ys


# Inside a transformer block q, k, v read the same hidden state and gate, up the same one, so (when they are
# not fused into one launch) those launches do not depend on each other: they go to side streams and join
# before o / down.  Everything else is in stream order (each layer's input is the previous layer's output in
# the real model).
CONCURRENT_WITH_PREVIOUS = {"k", "v", "up"}


def launch_unit(unit, xs, ys, stream):
    import paper_2410_21271_b200 as eora
    names, K, Ns, obj = unit
    if len(names) == 1:
        eora.eora_linear_forward(obj.handle, xs[names[0]], M_DECODE, ys[names[0]], stream)
    else:
        eora.eora_linear_forward_fused(obj.handle, xs[names[0]], M_DECODE, [ys[n] for n in names], stream)


def run_step(units, xs, ys, side=None):
    import torch
    main = torch.cuda.current_stream()
    pending = []
    i = 0
    while i < len(units):
        group = [units[i]]
        while i + len(group) < len(units) and units[i + len(group)][0][0] in CONCURRENT_WITH_PREVIOUS:
            group.append(units[i + len(group)])
        i += len(group)
        if side is None or len(group) == 1:
            for u in group:
                launch_unit(u, xs, ys, main)
            continue
        fork = main.record_event()
        for j, u in enumerate(group):
            st = main if j == 0 else side[(j - 1) % len(side)]
            if j:
                st.wait_event(fork)
            launch_unit(u, xs, ys, st)
            if j:
                pending.append(st.record_event())
        for ev in pending:
            main.wait_event(ev)
        pending = []


def time_decode(layers, xs, ys, steps: int, warmup: int, device_index: int, use_graph: bool = True,
                use_streams: bool = True):
    """Device-timed steps (CUDA events on the launching stream).  Returns (ms per step, clocks)."""
    import torch
    stream = torch.cuda.Stream()
    side = [torch.cuda.Stream(), torch.cuda.Stream()] if use_streams else None
    graph = None
    with torch.cuda.stream(stream):
        run_step(layers, xs, ys, side)
        torch.cuda.synchronize()
        if use_graph:
            try:
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=stream):
                    run_step(layers, xs, ys, side)
            except Exception:
                graph = None
        launch = graph.replay if graph is not None else (lambda: run_step(layers, xs, ys, side))
        for _ in range(warmup):
            launch()
        stream.synchronize()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(device_index) as cs:
            torch.cuda.synchronize()
            e0.record(stream)
            for _ in range(steps):
                launch()
            e1.record(stream)
            stream.synchronize()
            torch.cuda.synchronize()
        barrier()
        ms = e0.elapsed_time(e1) / steps
    for _, _, _, obj in layers:
        assert obj.device_status() == 0, "a device-side wait ran out"
    return ms, cs.summary(), graph is not None


def time_e2e(layers, steps: int, warmup: int):
    """The same step through eora_linear_forward_host: pinned host X in, host Y out, per layer."""
    import torch
    hx = {name: torch.from_numpy(gen.make_x(7, M_DECODE, K)).pin_memory() for name, (K, N) in LAYERS}
    hy = {name: torch.empty((M_DECODE, N), dtype=torch.float16).pin_memory() for name, (K, N) in LAYERS}
    def step():
        for names, K, Ns, obj in layers:
            if len(names) == 1:
                obj.forward_host(hx[names[0]], hy[names[0]])
            else:
                obj.forward_host(hx[names[0]], [hy[n] for n in names])
    for _ in range(max(1, warmup)):
        step()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    torch.cuda.synchronize()
    sec = (time.perf_counter() - t0) / steps
    h2d = sum(2 * M_DECODE * K for _, K, Ns, _ in layers)
    d2h = sum(2 * M_DECODE * N for _, K, Ns, _ in layers for N in Ns)
    return sec, h2d, d2h


def _time_prefill_layer(device: str, K: int, N: int, r: int, M: int, steps: int, warmup: int, flush):
    import torch
    import paper_2410_21271_b200 as eora
    wf = gen.make_backbone_quant(5, K, N, 4, 128)
    af, bf = gen.make_ab_f16(5, K, N, r)
    L = eora.Layer(wf, af, bf, max_m=M, device=device)
    path = L.path(M)
    x = torch.from_numpy(gen.make_x(6, M, K)).to(device)
    y = torch.empty((M, N), dtype=torch.float16, device=device)
    if path == eora.EORA_PATH_GENERIC:
        steps, warmup = 2, 1
    for _ in range(warmup):
        L.forward(x, y)
    times = []
    for _ in range(steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); L.forward(x, y); e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    L.close()
    return float(np.median(times)), path


def time_prefill(device: str, steps: int = 10, warmup: int = 3, layer_set: bool = False):
    """Extra: tensor-core prefill, 4-bit g128, fp16 r=128, M=2048: the q-shaped layer (the workload of the
    committed profile) and, with layer_set, every distinct shape of the LLaMA3-8B block."""
    import torch
    K = N = 4096
    M, r = 2048, 128
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=device)
    ms, path = _time_prefill_layer(device, K, N, r, M, steps, warmup, flush)
    fl = traffic.forward_flops(K, N, r, M)
    out = {"workload": "q 4096x4096/w4-g128/eora-fp16-r128/M2048", "ms": ms, "tflops": fl / ms / 1e9,
           "path": {0: "generic", 1: "decode", 2: "prefill"}[path], "l2": "flushed between iterations"}
    if layer_set:
        shapes = {"q,o": (4096, 4096, 2), "k,v": (4096, 1024, 2), "gate,up": (4096, 14336, 2), "down": (14336, 4096, 1)}
        per, tot_ms, tot_fl = {}, 0.0, 0.0
        for name, (k, n, count) in shapes.items():
            ms_s = ms if (k, n) == (K, N) else _time_prefill_layer(device, k, n, r, M, 6, warmup, flush)[0]
            fl_s = traffic.forward_flops(k, n, r, M)
            per[name] = {"ms": ms_s, "tflops": fl_s / ms_s / 1e9}
            tot_ms += count * ms_s
            tot_fl += count * fl_s
        out["layer_set"] = {"per_shape": per, "ms_block": tot_ms, "tflops": tot_fl / tot_ms / 1e9,
                            "note": "seven layers of a block, one launch unit per layer, times summed"}
    return out


# dram__bytes_read.sum + dram__bytes_write.sum of k_decode over the seven layers of one block, from the ncu
# capture summarised in profiles/k_decode_llama3-8b-w3g128-r128-M1.md (traffic grows with the number of
# blocks in proportion; fusing layers changes the number of launches, not the bytes).  Set to None when the
# kernel's memory behaviour changes until the capture is redone.
DRAM_BYTES_PER_BLOCK = 108.52e6


def cpu_oracle_sample(blocks_sample: int = 1):
    """The CPU oracle, as it stands, on `blocks_sample` block(s) of the decode workload."""
    from oracle import eora_oracle as orc
    x = {K: gen.make_x(7, M_DECODE, K) for _, (K, N) in LAYERS}
    data = []
    for li, (name, (K, N)) in enumerate(LAYERS):
        wf = gen.make_backbone_quant(1000 + li, K, N, 3 if W_FMT == "q3" else 4, 128)
        af, bf = gen.make_ab_f16(1000 + li, K, N, RANK)
        data.append((K, wf, af, bf))
    t0 = time.perf_counter()
    for _ in range(blocks_sample):
        for K, wf, af, bf in data:
            orc.forward(x[K], "f16", wf, af, bf)
    sec = time.perf_counter() - t0
    sec_per_token = sec / blocks_sample * gen.LLAMA3_8B_BLOCKS
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    return {"value": 1.0 / sec_per_token, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{blocks_sample} of {gen.LLAMA3_8B_BLOCKS} blocks (7 layers each) of the same workload, "
                      f"{sec:.1f} s of CPU work, scaled to a whole token"}, sec


# --------------------------------------------------------------------------------------------
_DIST = {"on": False}


def barrier():
    if _DIST["on"]:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(v: float) -> float:
    if not _DIST["on"]:
        return v
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([v], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate(ms_local: float, tokens_per_step_per_rank: int, world: int) -> tuple[float, float]:
    """Whole-job throughput: units of all ranks / max-over-ranks time.  Replicas only: no collective
    on the data path."""
    ms = max_over_ranks(ms_local)
    return world * tokens_per_step_per_rank / (ms / 1e3), ms


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--blocks", type=int, default=gen.LLAMA3_8B_BLOCKS, help=argparse.SUPPRESS)
    ap.add_argument("--no-extras", action="store_true", help="skip the prefill / e2e / cpu legs")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--unfused", action="store_true", help="one launch per layer (224 per token) instead of fusing q|k|v and gate|up")
    ap.add_argument("--only-prefill", action="store_true", help="run the prefill leg alone (for profiling) and print its result")
    ap.add_argument("--single-stream", action="store_true", help="launch all layers of a block in stream order")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    config = {"workload": WORKLOAD, "blocks": args.blocks, "layers_per_block": 7, "M": M_DECODE,
              "l2": "weights of one step (3.4 GB) exceed L2, no flush needed", "parallelism": f"replicas x{world}",
              "launches_per_token": 224 if args.unfused else 128,
              "fusion": ("none: one launch per layer" if args.unfused else
                         "q|k|v and gate|up of a block share their input and run as one launch each"),
              "streams": ("stream order" if (args.single_stream or not args.unfused) else
                          "q,k,v and gate,up of a block are independent and run on 3 / 2 streams; the rest in stream order")}

    if args.impl == "reference":
        if rank != 0:
            return
        warm = max(0, min(args.warmup, 1))
        for _ in range(warm):
            cpu_oracle_sample(1)
        vals = [cpu_oracle_sample(1) for _ in range(max(1, min(args.steps, 3)))]
        base = min(vals, key=lambda v: v[1])[0]
        line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 / base["value"],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                "data": "synthetic", "config": config, "cpu_baseline": base,
                "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    import torch
    import paper_2410_21271_b200 as eora
    eora.lib()                                   # fail loudly if the CUDA library is missing
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(device))
        _DIST["on"] = True

    if args.only_prefill:
        if rank == 0:
            print(json.dumps({"prefill": time_prefill(device)}))
        return
    fused = not args.unfused
    layers, xs, ys = build_layer_set(args.blocks, device, fused=fused)
    n_launch_step = sum(obj.launches(M_DECODE) for _, _, _, obj in layers)
    ms_local, clocks, graphed = time_decode(layers, xs, ys, args.steps, args.warmup, local_rank, not args.no_graph,
                                             not args.single_stream)
    value, ms = aggregate(ms_local, M_DECODE, world)
    peaks, peak_kind = measured_peaks()
    bytes_step = step_bytes(args.blocks, fused)
    achieved = bytes_step / (ms_local / 1e3) / 1e9
    roofline = {"bound": "hbm", "kernel": "k_decode", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}",
                "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "traffic": DRAM_BYTES_PER_BLOCK * args.blocks / n_launch_step,
                "bytes_per_launch": bytes_step / n_launch_step, "us_per_launch": ms_local * 1e3 / n_launch_step}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16", "data": "synthetic", "config": config, "clocks": clocks,
            "gpu_launches": n_launch_step * args.steps, "cuda_graph": graphed, "roofline": roofline}

    if not args.no_extras:
        sec, h2d, d2h = time_e2e(layers, max(2, min(args.steps, 10)), 1)
        sec = max_over_ranks(sec)
        line["e2e"] = {"value": world * M_DECODE / sec, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                       "note": "per launch unit: pinned host X -> device, the layer(s), Y -> host, stream sync"}
    for _, _, _, obj in layers:
        obj.close()
    if not args.no_extras and rank == 0:
        if world == 1:
            line["cpu_baseline"] = cpu_oracle_sample(8)[0]
        try:
            line["prefill"] = time_prefill(device, layer_set=True)
            line["prefill"]["frac_of_measured_bf16_burst"] = line["prefill"]["tflops"] / peaks["bf16_tflops"]
            line["prefill"]["layer_set"]["frac_of_measured_bf16_burst"] = line["prefill"]["layer_set"]["tflops"] / peaks["bf16_tflops"]
        except Exception as e:  # the decode line must still be printed
            line["prefill"] = {"error": repr(e)}
    if rank == 0:
        print(json.dumps(line))
    if _DIST["on"]:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
