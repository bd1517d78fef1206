#!/usr/bin/env python
"""Benchmark of the routed quantized-linear path on B200.

One *step* is one pass of the whole hot path over one synthetic batch of a
workload: route (arg-max of resident logits) -> expand ids -> stable sort by
expert -> the routed dequant-GEMM of every linear layer of the block, each fed
its own resident activations, outputs written back in original row order.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is tokens/s over all N GPUs with inputs
resident in HBM; `e2e` is the same metric with host buffers (pinned host ->
device copies of logits and activations and device -> host copies of the outputs
inside the timed region); `roofline` describes the dominant kernel; and
`cpu_baseline` is the CPU oracle timed on this machine's cores on a bounded
sample.  `--impl reference` times that oracle alone.
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

import moqe_workloads as wl  # noqa: E402

METRIC = "routed_qgemm_tokens_per_s"
UNIT = "tokens/s"

# DRAM traffic of the dominant kernel comes from the tracked table profiles/dram_traffic.txt: one line per ncu capture,
#   workload  kernel source file  git blob hash of that file when captured  dram bytes per launch  algorithmic bytes of that launch
# The ratio of the last two is applied to the average launch of the block (traffic grows with the bytes streamed).
# A line whose hash no longer matches the source file is ignored: `traffic` is then null.
TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "dram_traffic.txt")


def git_blob_hash(path: str) -> str:
    import hashlib
    with open(path, "rb") as f:
        data = f.read()
    return hashlib.sha1(b"blob %d\0" % len(data) + data).hexdigest()


def traffic_ratio(workload: str):
    try:
        with open(TRAFFIC_TABLE) as f:
            lines = [l.split() for l in f if l.strip() and not l.startswith("#")]
    except OSError:
        return None
    for name, src, blob, dram, alg in lines:
        if name == workload:
            path = os.path.join(ROOT, src)
            if os.path.exists(path) and git_blob_hash(path) == blob:
                return float(dram) / float(alg)
    return None


# --------------------------------------------------------------------------- helpers
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the GPU is under load."""

    def __init__(self, index: int, period_s: float = 0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if bit and (r & bit):
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2.0)
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def workload_logits(w, seed, pooled_from=None):
    if w.routing == "router_mlp":
        layer = w.layers[0]
        X = wl.activations_bf16(f"{w.name}/{layer.name}/X", w.M_of(layer), layer.K, w.relu_inputs, seed)
        return wl.router_logits(w, seed, pooled=wl.mean_pool(X, w.row_offsets(layer)))
    return wl.router_logits(w, seed)


# --------------------------------------------------------------------------- CPU oracle legs
def oracle_sample_plan(w):
    """Distinct layer shapes with their multiplicity inside the block: timing one of each and
    weighting by the multiplicity reproduces the block's work exactly."""
    shapes = {}
    for l in w.layers:
        key = (l.N, l.K, l.rows_per_sample)
        if key not in shapes:
            shapes[key] = [l, 0]
        shapes[key][1] += 1
    return list(shapes.values())


def run_oracle_once(w, prepared, rows_per_layer):
    """-> seconds of oracle routed GEMM for the block (distinct shapes x multiplicity), rows sampled."""
    import oracle
    total = 0.0
    for (layer, mult, X, row_ids, What, rows) in prepared:
        t0 = time.perf_counter()
        oracle.routed_gemm(X, row_ids, What, rows=rows)
        dt = time.perf_counter() - t0
        M = X.shape[0]
        total += dt * mult * (M / float(len(rows)))          # linear in rows: extrapolated to all M rows
    return total


def prepare_oracle(w, seed, max_rows):
    import oracle
    ids = oracle.route(workload_logits(w, seed))
    prepared, t_quant, t_deq = [], 0.0, 0.0
    for layer, mult in oracle_sample_plan(w):
        W, X = wl.layer_inputs(w, layer, seed)
        row_ids = oracle.expand_ids(ids, w.row_offsets(layer))
        What = []
        for sp in w.experts:
            t0 = time.perf_counter()
            c, s, z = oracle.quantize_rtn(W, sp.bits, sp.group, sp.sym)
            t1 = time.perf_counter()
            What.append(oracle.dequantize(c, s, z, sp.group))
            t2 = time.perf_counter()
            t_quant += (t1 - t0) * mult
            t_deq += (t2 - t1) * mult
        M = X.shape[0]
        _, offsets, perm, _ = oracle.permutation(row_ids, w.n_experts)
        if M <= max_rows:
            rows = np.arange(M, dtype=np.int32)
        else:                                                 # first/last row of every expert + evenly spaced rows
            per = max(1, max_rows // w.n_experts)
            pick = []
            for e in range(w.n_experts):
                lo, hi = int(offsets[e]), int(offsets[e + 1])
                if hi > lo:
                    pick.extend(perm[np.unique(np.linspace(lo, hi - 1, num=min(per, hi - lo)).astype(np.int64))])
            rows = np.array(sorted(set(int(v) for v in pick)), dtype=np.int32)
        prepared.append((layer, mult, X, row_ids, What, rows))
    return prepared, t_quant, t_deq


def oracle_sample_text(w, prepared):
    parts = [f"{layer.name} x{mult} ({len(rows)}/{X.shape[0]} rows, all N, full K)" for (layer, mult, X, _, _, rows) in prepared]
    return "oracle routed GEMM on one layer of each distinct shape, weighted by its count in the block: " + "; ".join(parts)


def reference_arm(args, w):
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    tokens = sum(w.sample_rows) if w.layers[0].rows_per_sample is None else w.n_samples
    budget_s = 150.0
    max_rows = 16
    prepared, t_quant, t_deq = prepare_oracle(w, args.seed, max_rows)
    probe = 0.0
    t0 = time.perf_counter()
    run_oracle_once(w, prepared, None)
    probe = time.perf_counter() - t0
    if probe * (args.steps + args.warmup) > budget_s and max_rows > 3:
        max_rows = max(3, int(max_rows * budget_s / (probe * (args.steps + args.warmup))))
        prepared, t_quant, t_deq = prepare_oracle(w, args.seed, max_rows)
    for _ in range(args.warmup):
        run_oracle_once(w, prepared, None)
    times = [run_oracle_once(w, prepared, None) for _ in range(args.steps)]
    step_s = float(np.mean(times))
    value = tokens / step_s
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "tokens_per_step": tokens, "note": "CPU oracle (plain C, fp32 sequential accumulation), extrapolated linearly to the block"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": oracle_sample_text(w, prepared), "dequant_s": t_deq, "quantize_s": t_quant},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- the CUDA arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b_decode", choices=list(wl.WORKLOAD_ORDER))
    ap.add_argument("--path", type=int, default=0, help="0 auto, 1 streaming kernel, 2-4 tcgen05 kernel")
    ap.add_argument("--seed", type=int, default=wl.BASE_SEED)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-fuse", action="store_true", help="one launch per layer (no q/k/v, gate/up grouping)")
    ap.add_argument("--tune", action="append", default=[], help="key=value passed to moqe_tune (measurement knob)")
    ap.add_argument("--repeats", type=int, default=5, help="timings of --steps steps each; the median is reported")
    ap.add_argument("--no-workloads", action="store_true", help="skip the sub-records of the other workloads")
    ap.add_argument("--force-expert", type=int, default=None, help="route every sample to this expert (per-format timing)")
    ap.add_argument("--experts", default=None, help="replace the workload's expert formats: 'bits,group,sym;...' (same count), "
                                                    "e.g. '8,0,1;2,128,0;3,128,0' (measurement of other formats on the same shapes)")
    ap.add_argument("--fused-block", action="store_true",
                    help="decode workloads: gate/up as ONE gated launch (silu(gate) * up), residual add in the o / down stores")
    args = ap.parse_args()
    w = wl.get(args.workload)
    heavy = w.kind in ("prefill", "mixed", "conv")
    if args.steps is None:
        args.steps = 20 if heavy else 2000
    if args.warmup is None:
        args.warmup = 3 if heavy else 200
    args.warmup = max(args.warmup, 3)

    if args.impl == "reference":
        reference_arm(args, w)
        return

    import torch
    import torch.distributed as dist
    import paper_2508_09204_b200 as moqe
    from paper_2508_09204_b200 import replicas

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the routed path has no CPU fallback")
    moqe.lib()                                              # fails loudly if the CUDA library is not built
    for kv in args.tune:
        k, v = kv.split("=")
        moqe.moqe_tune(k, int(v))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    heavy = w.kind in ("prefill", "mixed", "conv")
    peaks = load_peaks()
    seed = replicas.shard_seed(args.seed, rank)             # every rank owns its own shard of samples (weak scaling)
    stream = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(stream)
    ctx = dict(torch=torch, moqe=moqe, replicas=replicas, dev=dev, stream=stream, world=world, rank=rank, local=local,
               peaks=peaks, seed=seed, args=args, experts={})

    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    if args.experts:
        import dataclasses
        sp = tuple(wl.ExpertSpec(int(b), int(g), bool(int(y))) for b, g, y in (t.split(",") for t in args.experts.split(";")))
        if len(sp) != len(w.experts):
            raise SystemExit(f"--experts: workload {w.name} has {len(w.experts)} experts")
        w = dataclasses.replace(w, experts=sp)
        args.no_workloads = True
    line = bench_workload(ctx, w, steps=args.steps, warmup=args.warmup, repeats=args.repeats, with_e2e=True, force_expert=args.force_expert)
    line["clocks"] = sampler.stop()

    # ---- the other workloads of the metric, as sub-records (resident inputs, fewer steps) -------
    if args.workload == "llama7b_decode" and not args.no_workloads and world == 1:
        subs = {}
        for name in ("llama7b_prefill", "qwen7b_mixed", "resnet50_1x1", "tiny"):
            w2 = wl.get(name)
            heavy2 = w2.kind in ("prefill", "mixed", "conv")
            sm = ClockSampler(physical_gpu_index(local))
            sm.start()
            rec = bench_workload(ctx, w2, steps=5 if heavy2 else 200, warmup=3 if heavy2 else 20, repeats=3, with_e2e=False)
            if name == "llama7b_prefill":
                # the seeded mix is mostly 8-bit rows: time every format alone as well (all sequences to one expert)
                rec["per_format"] = {}
                for e, sp in enumerate(w2.experts):
                    r = bench_workload(ctx, w2, steps=5, warmup=3, repeats=3, with_e2e=False, force_expert=e)
                    rec["per_format"][sp.tag] = {"ms_per_step": r["ms_per_step"], "roofline": r["roofline"]}
            rec["clocks"] = sm.stop()
            subs[name] = {k: rec[k] for k in ("ms_per_step", "value", "unit", "config", "roofline", "gpu_launches", "clocks",
                                              "device_status", "ms_per_step_repeats") if k in rec}
            if "per_format" in rec:
                subs[name]["per_format"] = rec["per_format"]
            ctx["experts"] = {k: v for k, v in ctx["experts"].items() if k[0] == "llama"}   # free what the next one cannot reuse
            torch.cuda.empty_cache()
        line["workloads"] = subs

    # ---- the oracle on this machine's cores (rank 0, single-GPU runs only) ----------------------
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        max_rows = 16 if not heavy else 6
        prepared, t_quant, t_deq = prepare_oracle(w, args.seed, max_rows)
        sec = run_oracle_once(w, prepared, None)
        tokens_per_step = line["config"]["tokens_per_step"]
        line["cpu_baseline"] = {"value": tokens_per_step / sec, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                                "sample": oracle_sample_text(w, prepared), "gemm_s_extrapolated": sec,
                                "dequant_s": t_deq, "quantize_s": t_quant}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def bench_workload(ctx, w, steps, warmup, repeats, with_e2e, force_expert=None):
    """Times one workload: experts built (or reused), inputs resident, one step = route -> expand -> sort -> the routed
    GEMM of every layer; returns the record (top-level keys of the JSON line)."""
    import ctypes as C
    torch, moqe, replicas = ctx["torch"], ctx["moqe"], ctx["replicas"]
    dev, stream, world, peaks, seed, args = ctx["dev"], ctx["stream"], ctx["world"], ctx["peaks"], ctx["seed"], ctx["args"]
    heavy = w.kind in ("prefill", "mixed", "conv")
    E = w.n_experts

    # ---- experts (replicated on every rank) and resident inputs ---------------------------------
    family = w.name.split("7b")[0] if "7b" in w.name else w.name
    layers = []
    for layer in w.layers:
        key = (family, layer.name, layer.N, layer.K, tuple(sp.tag for sp in w.experts))
        if key not in ctx["experts"]:                       # (workloads of one model share shapes and formats: one set of experts)
            Wd = torch.from_numpy(wl.weights_f32(f"{w.name}/{layer.name}/W", layer.N, layer.K, 0.02, args.seed)).to(dev)
            ctx["experts"][key] = [moqe.moqe_quantize_rtn(Wd, sp.bits, sp.group, sp.sym) for sp in w.experts]
            del Wd
        experts = ctx["experts"][key]
        M = w.M_of(layer)
        Xh = torch.from_numpy(wl.activations_bf16(f"{w.name}/{layer.name}/X", M, layer.K, w.relu_inputs, seed).view(np.int16)).view(torch.bfloat16)
        if with_e2e:
            Xh = Xh.pin_memory()
        X = Xh.to(dev)
        Y = torch.empty((M, layer.N), dtype=torch.bfloat16, device=dev)
        Yh = torch.empty((M, layer.N), dtype=torch.bfloat16).pin_memory() if with_e2e else None
        ws = moqe.alloc_workspace(moqe.moqe_routed_qgemm_workspace(M, layer.N, layer.K, E), dev)
        moqe.moqe_routed_qgemm_workspace_clear(ws, M, layer.N, layer.K, E)
        off_h = torch.from_numpy(w.row_offsets(layer)).pin_memory()
        arr = (C.c_void_p * E)(*[e.handle for e in experts])
        layers.append(dict(spec=layer, experts=experts, M=M, X=X, Xh=Xh, Y=Y, Yh=Yh, ws=ws, arr=arr,
                           row_off=off_h.to(dev), row_off_h=off_h))
    # Layers of a block that read the same input and do not depend on one another (q/k/v, gate/up) go to the GPU as ONE
    # call when the decode kernel takes the batch; every other layer is a call of its own.
    siblings = [("q_proj", "k_proj", "v_proj"), ("gate_proj", "up_proj")]
    groups, used = [], set()
    for i, L in enumerate(layers):
        if i in used:
            continue
        g = [i]
        for sib in siblings:
            if L["spec"].name in sib and not args.no_fuse and L["M"] <= 16:
                g = [j for j, L2 in enumerate(layers) if L2["spec"].name in sib and L2["M"] == L["M"] and L2["spec"].K == L["spec"].K]
        for j in g:
            used.add(j)
        groups.append(g)
    fused_block = bool(args.fused_block) and max(L["M"] for L in layers) <= 16
    for g in groups:
        Ls = [layers[j] for j in g]
        names = tuple(L["spec"].name for L in Ls)
        if fused_block and names == ("gate_proj", "up_proj"):
            Ls[0]["gated"] = ((C.c_void_p * E)(*[e.handle for e in Ls[0]["experts"]]), (C.c_void_p * E)(*[e.handle for e in Ls[1]["experts"]]))
        elif fused_block and names in (("o_proj",), ("down_proj",)):
            Ls[0]["resid"] = torch.randn((Ls[0]["M"], Ls[0]["spec"].N), device=dev).to(torch.bfloat16)
        if len(g) > 1:
            layers[g[0]]["multi"] = ((C.c_void_p * len(g))(*[L["X"].data_ptr() for L in Ls]),
                                     (C.c_void_p * len(g))(*[L["Y"].data_ptr() for L in Ls]),
                                     (C.c_void_p * (len(g) * E))(*[e.handle for L in Ls for e in L["experts"]]))
    on_device_router = w.routing == "router_mlp" and force_expert is None
    if on_device_router:
        # the router front end runs on the device inside the step: mean-pool of the first layer's input -> MLP -> ids
        W1h, W2h = wl.router_weights(w, seed)
        rW1, rW2 = torch.from_numpy(W1h).to(dev), torch.from_numpy(W2h).to(dev)
        r_ws = moqe.alloc_workspace(moqe.lib().moqe_router_mlp_workspace(w.n_samples, w.layers[0].K, 256), dev)
        logits_h = torch.zeros((w.n_samples, E), dtype=torch.float32).pin_memory()
    else:
        lg = workload_logits(w, seed)
        if force_expert is not None:                        # every sample to one expert
            lg = np.full_like(lg, -1.0)
            lg[:, force_expert] = 1.0
        logits_h = torch.from_numpy(lg).pin_memory()
    logits = logits_h.to(dev)
    torch.cuda.synchronize()

    def run_group(g, perm, offsets):
        Ls = [layers[j] for j in g]
        if "gated" in Ls[0]:
            moqe.moqe_routed_qgemm_sorted_gated(Ls[0]["X"], perm, offsets, Ls[0]["experts"], Ls[1]["experts"], Ls[0]["Y"],
                                                Ls[0]["ws"], _arrs=Ls[0]["gated"])
        elif "resid" in Ls[0]:
            L = Ls[0]
            moqe.moqe_routed_qgemm_sorted_residual(L["X"], perm, offsets, L["experts"], L["resid"], L["Y"], L["ws"], _arr=L["arr"])
        elif len(g) > 1:
            moqe.moqe_routed_qgemm_sorted_multi([L["X"] for L in Ls], perm, offsets, [L["experts"] for L in Ls],
                                                [L["Y"] for L in Ls], Ls[0]["ws"], _arrs=Ls[0]["multi"])
        else:
            L = Ls[0]
            moqe.moqe_routed_qgemm_sorted(L["X"], perm, offsets, L["experts"], L["Y"], L["ws"], path=args.path, _arr=L["arr"])

    one_launch_routing = (not on_device_router and len({L["spec"].rows_per_sample for L in layers}) == 1
                          and layers[0]["M"] <= 1024 and w.n_samples <= 1024)

    # Host buffers: the inputs of every call go up on one copy stream and the results come down on another, so that the
    # copies of a call overlap the kernels of its neighbours (PCIe is full duplex); a step begins when the previous one
    # has completely finished and ends when its last result has landed.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    # groups of layers that share one row structure share one sort
    def hot_path(from_host: bool):
        lgd = logits
        ev_in = []
        if from_host:
            fork = torch.cuda.Event()
            fork.record(stream)
            s_in.wait_event(fork)
            s_out.wait_event(fork)
            with torch.cuda.stream(s_in):
                if not on_device_router:
                    lgd.copy_(logits_h, non_blocking=True)
                for g in groups:
                    for j in g:
                        layers[j]["X"].copy_(layers[j]["Xh"], non_blocking=True)
                    ev = torch.cuda.Event()
                    ev.record(s_in)
                    ev_in.append(ev)
            stream.wait_event(ev_in[0])                     # (recorded after the logits and the first call's inputs)
        if on_device_router:
            _, ids = moqe.moqe_router_mlp(layers[0]["X"], layers[0]["row_off"], rW1, rW2, workspace=r_ws)
        else:
            if one_launch_routing:                          # a decode step: arg-max, expansion and sort in one launch
                L0 = layers[0]
                _, _, perm, offsets = moqe.moqe_route_permute(lgd, L0["row_off"], L0["M"])
                sorted_for = {L0["spec"].rows_per_sample: (perm, offsets)}
            else:
                ids = moqe.moqe_route(lgd)
        if not one_launch_routing:
            sorted_for = {}
        for gi, g in enumerate(groups):
            Ls = [layers[j] for j in g]
            if from_host:
                stream.wait_event(ev_in[gi])
            key = Ls[0]["spec"].rows_per_sample
            if key not in sorted_for:
                row_ids = moqe.moqe_expand_ids(ids, Ls[0]["row_off"], Ls[0]["M"])
                _, perm, offsets = moqe.moqe_permute(None, row_ids, E)
                sorted_for[key] = (perm, offsets)
            perm, offsets = sorted_for[key]
            run_group(g, perm, offsets)
            if from_host:
                done = torch.cuda.Event()
                done.record(stream)
                s_out.wait_event(done)
                with torch.cuda.stream(s_out):
                    for L in Ls:
                        L["Yh"].copy_(L["Y"], non_blocking=True)
        if from_host:
            join = torch.cuda.Event()
            join.record(s_out)
            stream.wait_event(join)
        return sorted_for

    def make_runner(from_host: bool):
        """Warm up eagerly, then capture one step in a CUDA graph (the launch-bound inner loop)."""
        for _ in range(2):
            hot_path(from_host)
        stream.synchronize()
        if args.no_graph:
            return (lambda: hot_path(from_host)), 0
        before = moqe.moqe_launch_count()
        g = torch.cuda.CUDAGraph()
        try:
            with torch.cuda.graph(g, stream=stream):
                hot_path(from_host)
        except Exception as ex:                                # capture refused: run eagerly
            print(f"[bench] graph capture failed ({type(ex).__name__}: {ex}); running eagerly", file=sys.stderr)
            stream.synchronize()
            return (lambda: hot_path(from_host)), 0
        per_step = moqe.moqe_launch_count() - before
        return g.replay, per_step

    def timed(run, n_steps, n_warmup):
        for _ in range(n_warmup):
            run()
        stream.synchronize()
        replicas.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n_steps):
            run()
        e1.record(stream)
        torch.cuda.synchronize()
        replicas.barrier()
        return replicas.max_over_ranks(e0.elapsed_time(e1), dev)

    tokens_per_step = sum(w.sample_rows) if w.layers[0].rows_per_sample is None else w.n_samples

    # ---- 1. resident inputs: the median of `repeats` timings of `steps` steps each --------------
    run, graph_launches = make_runner(False)
    l0 = moqe.moqe_launch_count()
    rep_ms = []
    for r in range(max(1, repeats)):
        rep_ms.append(timed(run, steps, warmup if r == 0 else 1) / steps)
    launches_eager = moqe.moqe_launch_count() - l0
    launches = (graph_launches * steps) if graph_launches else launches_eager // max(1, repeats)
    ms_per_step = float(np.median(rep_ms))
    value = replicas.whole_job_value(tokens_per_step, world, ms_per_step)

    # ---- 2. per-launch duration of the dominant kernel (events round every routed-GEMM call) ----
    sorted_for = hot_path(False)
    stream.synchronize()
    counts = {k: np.diff(v[1].cpu().numpy()) for k, v in sorted_for.items()}
    reps = max(3, min(steps, 200 if not heavy else 10))
    per_layer_ms = []
    for g in groups:
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        per_layer_ms.append(evs)
    for r in range(reps):
        for g, evs in zip(groups, per_layer_ms):
            perm, offsets = sorted_for[layers[g[0]]["spec"].rows_per_sample]
            evs[r][0].record(stream)
            run_group(g, perm, offsets)
            evs[r][1].record(stream)
    stream.synchronize()
    layer_ms = [float(np.mean([a.elapsed_time(b) for a, b in evs[1:]])) for evs in per_layer_ms]

    # ---- 2b. the same launches back to back, as the step issues them, between ONE pair of events: an event pair round a
    # single launch adds the ~6 us an empty kernel measures that way on this part, and keeps a launch's prologue from
    # overlapping the previous launch's tail (programmatic dependent launch), which the timed step does.  One block's
    # weights exceed L2 for the headline workload, so cycling through the block's launches re-reads them from HBM.
    def gemm_block():
        for g in groups:
            perm, offsets = sorted_for[layers[g[0]]["spec"].rows_per_sample]
            run_group(g, perm, offsets)
    run_block = gemm_block
    if not args.no_graph:
        gb = torch.cuda.CUDAGraph()
        try:
            with torch.cuda.graph(gb, stream=stream):
                gemm_block()
            run_block = gb.replay
        except Exception as ex:
            print(f"[bench] graph capture of the GEMM-only block failed ({type(ex).__name__}: {ex}); running eagerly", file=sys.stderr)
            stream.synchronize()
    for _ in range(3):
        run_block()
    eb0, eb1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    eb0.record(stream)
    for _ in range(reps):
        run_block()
    eb1.record(stream)
    stream.synchronize()
    block_ms = eb0.elapsed_time(eb1) / reps
    status = moqe.moqe_async_status()

    alg_bytes, act_bytes, flops = [], [], []
    for L in layers:
        cnt = counts[L["spec"].rows_per_sample]
        b = 0
        for e, ex in enumerate(L["experts"]):
            if cnt[e] > 0:
                b += ex.code_bytes + ex.meta_bytes
        a = L["M"] * L["spec"].K * 2 + L["M"] * L["spec"].N * 2
        if fused_block and L["spec"].name == "up_proj":
            a -= L["M"] * L["spec"].N * 2                    # the gated launch writes one output for the pair
        if "resid" in L:
            a += L["M"] * L["spec"].N * 2                    # the residual is read
        alg_bytes.append(b + a)
        act_bytes.append(a)
        flops.append(2.0 * L["M"] * L["spec"].N * L["spec"].K)
    iso_ms = sum(layer_ms)
    tot_ms = block_ms
    n_launch = len(groups)
    ratio = traffic_ratio(w.name) if args.path == 0 and not args.tune and force_expert is None and not args.experts else None
    traffic = None if ratio is None else ratio * sum(alg_bytes) / n_launch
    hbm_time = sum(alg_bytes) / (peaks["hbm_gbs"] * 1e9)
    tensor_time = sum(flops) / (peaks["bf16_tflops"] * 1e12)
    hbm = {"achieved": sum(alg_bytes) / (tot_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    hbm["frac"] = hbm["achieved"] / hbm["peak"]
    hbm["frac_of_nominal_8000"] = hbm["achieved"] / 8000.0
    tens = {"achieved": sum(flops) / (tot_ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    tens["frac"] = tens["achieved"] / tens["peak"]
    tens["frac_of_nominal_2250"] = tens["achieved"] / 2250.0
    tens["frac_of_sustained"] = tens["achieved"] / peaks["bf16_tflops_sustained"]   # the library GEMM's rate under the power cap
    if tensor_time > hbm_time:
        roofline = {"bound": "tensor", **tens, "traffic": traffic,
                    "frac_whole_step": sum(flops) / (ms_per_step * 1e-3) / 1e12 / peaks["bf16_tflops"]}
        if w.kind == "mixed":                               # the other fraction of a mixed batch: expert bytes streamed once
            roofline["hbm"] = hbm
    else:
        roofline = {"bound": "hbm", **hbm, "traffic": traffic,
                    "frac_whole_step": sum(alg_bytes) / (ms_per_step * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    max_m = max(L["M"] for L in layers)
    small = all(L["spec"].N <= 1024 and L["spec"].K <= 1024 for L in layers)     # the library's dense-weights rule
    kernel = (("qgemm_dense_kernel" if small and args.path == 0 else "qgemm_tc_kernel") if max_m > 128
              else ("qgemm_decode_kernel" if max_m <= 16 else "qgemm_stream_kernel"))
    roofline.update({"peak_source": peaks["source"],
                     "kernel": kernel + f": average of the {n_launch} routed-GEMM launches of one block" +
                               (" (q/k/v and gate/up each in one launch)" if any(len(g) > 1 for g in groups) else ""),
                     "launches_per_step": n_launch, "algorithmic_bytes_per_launch": sum(alg_bytes) / n_launch,
                     "traffic_unit": "bytes per launch",
                     "algorithmic_bytes_per_step": int(sum(alg_bytes)), "activation_bytes_per_step": int(sum(act_bytes)),
                     "flops_per_step": float(sum(flops)),
                     "avg_launch_ms": block_ms / n_launch,
                     "avg_launch_ms_method": "events round `reps` repetitions of the block's routed-GEMM launches back to back "
                                             "(no route/sort kernels inside), divided by the launches",
                     "launch_ms_isolated": {"+".join(layers[j]["spec"].name for j in g): round(t, 5) for g, t in zip(groups, layer_ms)},
                     "frac_isolated": roofline["frac"] * block_ms / iso_ms,
                     "isolated_note": "one event pair round every single call: includes ~6 us of event/launch overhead per call "
                                      "(what an empty kernel measures that way) and no overlap between consecutive launches"})

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "ms_per_step_repeats": [round(v, 6) for v in rep_ms], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "layers": [f"{l.name}:{l.N}x{l.K}" for l in w.layers],
                   "experts": [sp.tag for sp in w.experts], "tokens_per_step": tokens_per_step,
                   "rows_per_expert": {str(k): v.tolist() for k, v in counts.items()},
                   "routing": "every sample to expert %d" % force_expert if force_expert is not None else
                              (w.routing + (" (computed on the device inside the step)" if on_device_router else "")),
                   "parallelism": f"replicas x{world} (samples sharded, experts replicated, no collective)",
                   "l2": "weights of one block exceed L2 (inputs larger than L2, no flush)" if sum(alg_bytes) > 126e6
                         else "working set fits L2", "cuda_graph": bool(graph_launches), "path": args.path,
                   "timing": f"median of {max(1, repeats)} repeats of {steps} steps",
                   "fused_block": ({"gate_up": "one gated launch, silu(gate) * up", "o_down": "residual added in the store",
                                    "bytes_not_moved_per_step": int(sum(3 * L["M"] * L["spec"].N * 2 for L in layers if L["spec"].name == "up_proj")),
                                    "note": "the [M][N] bf16 outputs of gate and up are never written nor re-read by a separate "
                                            "silu-mul kernel, which would also write its own output"} if fused_block else False),
                   "launch_groups": ["+".join(layers[j]["spec"].name for j in g) for g in groups]},
        "roofline": roofline, "gpu_launches": int(launches), "device_status": moqe.status_str(status),
    }

    # ---- 3. end to end through the public API with host buffers ---------------------------------
    if with_e2e:
        run_h, _ = make_runner(True)
        e2e_steps = max(3, steps // 4)
        ms_h = timed(run_h, e2e_steps, 3) / e2e_steps
        h2d = int(logits_h.numel() * 4 + sum(L["Xh"].numel() * 2 for L in layers))
        d2h = int(sum(L["Yh"].numel() * 2 for L in layers))
        line["e2e"] = {"value": replicas.whole_job_value(tokens_per_step, world, ms_h), "unit": UNIT, "h2d_bytes_per_step": h2d,
                       "d2h_bytes_per_step": d2h, "ms_per_step": ms_h}
    return line


if __name__ == "__main__":
    main()
