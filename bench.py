#!/usr/bin/env python
"""Benchmark of the GRASS layer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--rank r]
    python bench.py --impl reference ...      # the fp64 CPU oracle, timed on the host cores

--gpus N (N > 1) runs N independent replicas, one process per GPU: under a launcher
(torch.distributed.run sets WORLD_SIZE) this process is one of them; without one it starts
them itself.

A step is one iteration of the paper's Algorithm 1 over every layer of the
workload: on a refresh iteration (t = 0 mod K) the dense gradient, its row
norms and the selection, then for every layer projected gradient, Adam and
the row-sparse apply.  The timed region starts at t = 0, so it contains one
refresh per K steps and exercises all five library calls.  One JSON line is
printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "TFLOP/s per layer-step (select+project+Adam+scatter)"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from one ncu
# capture of the default workload at T = 8192 (1717.6 MB over the three GEMM launches of a step)
# scaled by 4 to T = 32768 (every operand is streamed once per launch, so traffic grows in
# proportion to the tokens), averaged over the three launches.  The kernel gathers the selected
# dY columns itself, so this includes every 128-byte line of dY that holds one.  None where
# nothing was captured.
NCU_TRAFFIC_BYTES = {"llama7b_block_r1024": 2290e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap,clocks.mem,clocks.max.mem")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20", "-i", str(self.gpu)], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons, power, mem, mem_mx = [], [], set(), [], [], []
        for line in self.file:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            try:
                mem.append(float(parts[7]))
                mem_mx.append(float(parts[8]))
            except (ValueError, IndexError):
                pass
            for name, val in zip(self.NAMES, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(power))
            if mem:
                out.update(mem_mhz=statistics.median(mem), mem_max_mhz=max(mem_mx))
        return out


# ----------------------------------------------------------------------------- oracle arm
def oracle_sample_step(wl, host_inputs, states, T_s):
    """One regular layer-step of the oracle per projection of one block on the first T_s tokens."""
    from oracle import grass_oracle as oracle
    for (name, m, n), (dY, X) in zip(wl.shapes, host_inputs):
        st = states[name]
        Gc = oracle.project_grad(dY[:T_s], X[:T_s], st["sigma"], st["rho"])
        st["M"], st["V"], U = oracle.adam_update(st["M"], st["V"], Gc, wl.lr, wl.beta1, wl.beta2,
                                                 wl.eps, st["step"])
        st["step"] += 1
        st["W"] = oracle.scatter_update(st["W"], U, st["sigma"], st["rho"], wl.alpha,
                                        w_is_bf16=wl.notes.get("w_is_bf16", True))
    return sum(2.0 * min(wl.r, m) * T_s * n for _, m, n in wl.shapes)


def make_oracle_states(wl, host_W):
    import numpy as np
    states = {}
    for (name, m, n), W in zip(wl.shapes, host_W):
        r = min(wl.r, m)
        rng = np.random.default_rng(m * 31 + n)
        sigma = np.sort(rng.choice(m, r, replace=False))
        states[name] = dict(sigma=sigma, rho=np.ones(r), M=np.zeros((r, n)), V=np.zeros((r, n)),
                            W=W.astype(np.float64), step=1)
    return states


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def time_oracle(wl, host_inputs, host_W, budget_s, steps=1, warmup=0):
    """Time `steps` sample steps of the oracle; the sample length is chosen from a calibration
    run so that warmup + steps fit in budget_s.  Returns dict(value TFLOP/s, sample, seconds)."""
    T_cal = min(256, wl.T)
    states = make_oracle_states(wl, host_W)
    t0 = time.perf_counter()
    oracle_sample_step(wl, host_inputs, states, T_cal)
    cal1 = time.perf_counter() - t0
    t0 = time.perf_counter()
    oracle_sample_step(wl, host_inputs, states, min(2 * T_cal, wl.T))
    cal2 = time.perf_counter() - t0
    per_token = max(cal2 - cal1, 0.05 * cal1) / T_cal      # cost that grows with the tokens
    fixed = max(cal1 - per_token * T_cal, 0.0)              # copies of W and of the state
    T_s = T_cal
    while T_s * 2 <= wl.T and (per_token * T_s * 2 + fixed) * (steps + warmup) <= budget_s:
        T_s *= 2
    states = make_oracle_states(wl, host_W)
    for _ in range(warmup):
        oracle_sample_step(wl, host_inputs, states, T_s)
    t0 = time.perf_counter()
    flops = 0.0
    for _ in range(steps):
        flops += oracle_sample_step(wl, host_inputs, states, T_s)
    sec = time.perf_counter() - t0
    return dict(value=flops / sec / 1e12, seconds=sec, T_sample=T_s, steps=steps,
                sample=f"{steps} regular layer-step(s) of one block ({len(wl.shapes)} projections) "
                       f"on the first {T_s} of {wl.T} tokens, r={wl.r}")


def host_block_inputs(wl, device):
    """float32 numpy copies of one block's inputs (exact widening of the bf16 bits)."""
    import torch
    from paper_2406_17660_b200 import synthetic as syn
    ins, Ws = [], []
    for pi, (name, m, n) in enumerate(wl.shapes):
        dY = syn.make_dY(wl.T, m, wl.dtype, proj=pi, device=device)
        X = syn.make_X(wl.T, n, wl.dtype, proj=pi, device=device)
        W = syn.make_W(m, n, wl.dtype, proj=pi, device=device)
        ins.append((syn.to_f32_numpy(dY), syn.to_f32_numpy(X)))
        Ws.append(syn.to_f32_numpy(W))
    return ins, Ws


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from paper_2406_17660_b200 import workloads
    wl = workloads.get(args.workload, r=args.rank, T=args.tokens, layers=args.layers)
    T_gen = min(wl.T, 8192)                      # the sample never reads more tokens than this
    gen = workloads.get(args.workload, r=args.rank, T=T_gen, layers=args.layers)
    ins, Ws = host_block_inputs(gen, "cpu")
    gen.T = T_gen
    res = time_oracle(gen, ins, Ws, budget_s=150.0, steps=args.steps, warmup=args.warmup)
    cores = blas_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": res["value"], "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * res["seconds"] / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "T": wl.T, "r": wl.r, "sample_tokens": res["T_sample"]},
        "cpu_baseline": {"value": res["value"], "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "sample": res["sample"]},
        "e2e": {"value": res["value"], "unit": "TFLOP/s", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- GPU arm
def aggregate_max(local_ms: float, dist_mod=None) -> float:
    """Max over ranks of a duration (the slowest replica bounds the job)."""
    if dist_mod is None or not dist_mod.is_initialized():
        return local_ms
    import torch
    dev = "cuda" if dist_mod.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    dist_mod.all_reduce(t, op=dist_mod.ReduceOp.MAX)
    return float(t.item())


def measure_workload(ctx, name, r, steps, warmup, want_e2e, want_cpu, args):
    """Run one workload on this rank's GPU and return its result line (rank 0; None elsewhere)."""
    import torch
    import torch.distributed as dist
    import paper_2406_17660_b200 as grass
    from paper_2406_17660_b200 import synthetic as syn
    from paper_2406_17660_b200 import workloads
    from paper_2406_17660_b200.step import GrassLayer, GrassLayerGroup, GrassWorkspace

    world, rank, local_rank, dev, peaks = (ctx["world"], ctx["rank"], ctx["local_rank"], ctx["dev"],
                                           ctx["peaks"])
    wl = workloads.get(name, r=r, T=args.tokens, layers=args.layers)
    K = args.refresh_every or wl.K
    # ---- inputs: one block of distinct tensors, shared by all blocks (replicas are independent:
    # every rank holds its own full copy of the workload, no data-path collective) ----
    block_in = []
    for pi, (pname, m, n) in enumerate(wl.shapes):
        dY = syn.make_dY(wl.T, m, wl.dtype, proj=pi, device=dev, ld=syn.pad_to(m, 8))
        X = syn.make_X(wl.T, n, wl.dtype, proj=pi, device=dev, ld=syn.pad_to(n, 8))
        block_in.append((dY, X))
    # Layers are independent, so consecutive layers go to alternating streams (each with its own
    # scratch): the HBM-bound kernels of one layer (Adam, apply, split-K reduce) then run beside
    # the GEMM of its neighbour.  --streams 1 puts everything on one stream.
    n_streams = max(1, args.streams)
    main_stream = torch.cuda.current_stream()
    streams = [main_stream] + [torch.cuda.Stream() for _ in range(n_streams - 1)]
    wss = [GrassWorkspace([(m, n) for _, m, n in wl.shapes], wl.T, wl.r, wl.dtype, wl.method,
                          device=dev) for _ in range(n_streams)]
    layers = []
    for i, (li, pi, pname, m, n) in enumerate(wl.layer_list()):
        W = syn.make_W(m, n, wl.dtype, layer=li, proj=pi, device=dev, ld=syn.pad_to(n, 8))
        layer = GrassLayer(W, min(wl.r, m), wl.method, K, wl.alpha, wl.lr, wl.beta1, wl.beta2,
                           wl.eps, reset_state=wl.reset_state, seed=0,
                           layer_id=li * len(wl.shapes) + pi, workspace=wss[i % n_streams],
                           fused_update=not args.unfused, keep_U=False)
        layer.stream = streams[i % n_streams]
        layers.append((pi, layer))
    in_bytes = sum(d.numel() * d.element_size() + x.numel() * x.element_size() for d, x in block_in)

    # units of work: a single layer, or (--batched, bf16) a run of consecutive layers of one
    # shape inside a block (q,k,v,o / gate,up / down) stepped by one set of launches.  A unit has
    # one stream and one scratch; consecutive units alternate over the streams.
    units = []
    i = 0
    while i < len(layers):
        j = i + 1
        if args.batched and wl.dtype == torch.bfloat16:
            while (j < len(layers) and j - i < 8 and layers[j][1].W.shape == layers[i][1].W.shape
                   and j // len(wl.shapes) == i // len(wl.shapes)):
                j += 1
        members = layers[i:j]
        obj = members[0][1] if len(members) == 1 else GrassLayerGroup([l for _, l in members], wl.T,
                                                                      device=dev)
        units.append({"obj": obj, "pis": [pi for pi, _ in members], "layers": [l for _, l in members]})
        i = j
    # Within a step the units are independent, so their order is free: start with the unit whose
    # dY is smallest (layers x m) and keep the rest in block order.
    if len(units) > 2:
        first = min(range(len(units)), key=lambda u: len(units[u]["layers"]) * units[u]["layers"][0].m)
        units.insert(0, units.pop(first))
    for u, unit in enumerate(units):
        unit["stream"] = streams[u % n_streams]
        for l in unit["layers"]:
            l.stream = unit["stream"]
            l.ws = wss[u % n_streams]

    def run_unit(unit, stream):
        with torch.cuda.stream(stream):
            if len(unit["layers"]) == 1:
                unit["obj"].step(*block_in[unit["pis"][0]])
            else:
                unit["obj"].step([block_in[p][0] for p in unit["pis"]],
                                 [block_in[p][1] for p in unit["pis"]])

    single_stream = [False]

    def one_step():
        for st in streams[1:]:
            st.wait_stream(main_stream)
        for unit in units:
            run_unit(unit, main_stream if single_stream[0] else unit["stream"])
        for st in streams[1:]:
            main_stream.wait_stream(st)

    def rewind():
        for _, layer in layers:
            layer.t = 0

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(warmup, 3)):
        one_step()
    grass.grass_device_status()

    # ---- pass A: the timed region ----
    rewind()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.1)
    barrier()
    ev[0].record()
    for i in range(steps):
        one_step()
        ev[i + 1].record()
    barrier()
    total_ms = aggregate_max(ev[0].elapsed_time(ev[-1]), dist if world > 1 else None)
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    grass.grass_device_status()

    # ---- pass B: the same steps with every kernel launch bracketed by events ----
    rewind()
    n_refresh = (steps + K - 1) // K
    cap = steps * len(layers) * 5 + n_refresh * len(layers) * 8 + 16
    # one stream for this pass: an event pair must bracket one kernel running alone, not a kernel
    # sharing the GPU with another layer's kernels
    single_stream[0] = True
    grass.grass_profile_begin(cap)
    for i in range(steps):
        one_step()
    launches, recs = grass.grass_profile_end()
    single_stream[0] = False
    clocks = sampler.stop() if rank == 0 else None
    if args.launch_log:
        with open(args.launch_log, "w") as f:
            json.dump([(kname, round(1e3 * ms, 2)) for kname, ms in recs], f)
    per_kernel = {}
    for kname, ms in recs:
        k = per_kernel.setdefault(kname, {"launches": 0, "ms": 0.0})
        k["launches"] += 1
        k["ms"] += ms
    prof_total = sum(k["ms"] for k in per_kernel.values())
    for k in per_kernel.values():
        k["share"] = k["ms"] / prof_total if prof_total > 0 else 0.0
        k["avg_us"] = 1e3 * k["ms"] / k["launches"]

    refresh_steps = [i for i in range(steps) if i % K == 0]
    regular_steps = [i for i in range(steps) if i % K != 0]
    flops_total = wl.flops_regular() * steps + wl.flops_refresh_extra() * len(refresh_steps)
    value = world * flops_total / (total_ms * 1e-3) / 1e12
    n_layers = len(layers)

    # ---- roofline of the dominant kernel (tcgen05 projection GEMM, which now also gathers) ----
    # The measured peak that applies depends on how long the GPU has been under load: a timed
    # region of well under a second runs at burst clocks, a long one settles at the power cap.
    roofline = None
    region_s = (total_ms + prof_total) * 1e-3
    if "project_tc" in per_kernel:
        tc = per_kernel["project_tc"]
        burst, sustained = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
        use_burst = region_s < 1.0
        tpeak = burst if use_burst else sustained
        which = "burst" if use_burst else "sustained"
        path_ms = sum(per_kernel[k]["ms"] for k in ("gather", "project_tc", "splitk_reduce")
                      if k in per_kernel)
        # algorithmic bytes of the projection per layer-step: X once, the r selected columns of
        # dY once, G_C out (2Tn + 2Tr + 4rn); per refresh: X and dY once (2Tn + 2Tm).  What the
        # memory system cannot avoid touching is larger: every 128-byte line of dY that holds a
        # selected column (measured with ncu), i.e. 2Tm (1 - (1 - r/m)^64) instead of 2Tr.
        rs = [(min(wl.r, m), m, n) for _, m, n in wl.shapes]
        alg_reg = sum(2.0 * wl.T * n + 2.0 * wl.T * r_ + 4.0 * r_ * n for r_, m, n in rs) * wl.layers
        touched_reg = sum(2.0 * wl.T * n + 2.0 * wl.T * m * (1.0 - (1.0 - r_ / m) ** 64) + 4.0 * r_ * n
                          for r_, m, n in rs) * wl.layers
        dense = sum(2.0 * wl.T * n + 2.0 * wl.T * m for r_, m, n in rs) * wl.layers
        # the launches of the regular steps only: the dense GEMMs of refresh iterations are the
        # same kernel on all m rows and are accounted separately ("dense" below)
        alg_total = alg_reg * steps
        touched_total = touched_reg * steps
        flops_proj = wl.flops_regular() * steps
        t_tensor = wl.flops_regular() / (tpeak * 1e12)
        t_hbm = alg_reg / (peaks["hbm_gbs"] * 1e9)
        tensor_side = {"achieved": flops_proj / (tc["ms"] * 1e-3) / 1e12, "unit": "TFLOP/s", "peak": tpeak,
                       "peak_source": f"{peaks['source']} cuBLAS bf16, {which} (timed region {region_s:.2f} s)"}
        tensor_side["frac"] = tensor_side["achieved"] / tpeak
        hbm_side = {"achieved": alg_total / (tc["ms"] * 1e-3) / 1e9, "unit": "GB/s", "peak": peaks["hbm_gbs"],
                    "peak_source": f"{peaks['source']} HBM copy bandwidth",
                    "touched_gbs": touched_total / (tc["ms"] * 1e-3) / 1e9}
        hbm_side["frac"] = hbm_side["achieved"] / peaks["hbm_gbs"]
        hbm_side["frac_touched"] = hbm_side["touched_gbs"] / peaks["hbm_gbs"]
        bound = "hbm" if t_hbm > t_tensor else "tensor"
        main_side = hbm_side if bound == "hbm" else tensor_side
        roofline = {"kernel": "project_tc_kernel", "bound": bound,
                    "bound_rule": "regular step: algorithmic bytes / HBM peak vs flops / tensor peak, "
                                  f"{1e6 * t_hbm:.0f} us vs {1e6 * t_tensor:.0f} us",
                    "achieved": main_side["achieved"], "peak": main_side["peak"],
                    "unit": main_side["unit"], "frac": main_side["frac"],
                    "peak_source": main_side["peak_source"],
                    "tensor": tensor_side, "hbm": hbm_side,
                    "frac_of_burst_peak": tensor_side["achieved"] / burst,
                    "frac_of_sustained_peak": tensor_side["achieved"] / sustained,
                    # the projection as the method sees it: selected-column gather (inside the GEMM
                    # kernel unless a pre-pass is used) + GEMM + split-K reduce, same flops
                    "path": {"kernels": [k for k in ("gather", "project_tc", "splitk_reduce")
                                         if k in per_kernel],
                             "ms": path_ms, "achieved": flops_proj / (path_ms * 1e-3) / 1e12,
                             "frac": flops_proj / (path_ms * 1e-3) / 1e12 / tpeak,
                             "hbm_frac_touched": touched_total / (path_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
                    "traffic": NCU_TRAFFIC_BYTES.get(f"{wl.name}_r{wl.r}")}
        if "project_tc_dense" in per_kernel and refresh_steps:
            dn = per_kernel["project_tc_dense"]
            ach = wl.flops_refresh_extra() * len(refresh_steps) / (dn["ms"] * 1e-3) / 1e12
            roofline["dense"] = {"what": "refresh iterations: dY^T X on all m rows with the row-norm "
                                         "epilogue, 2mTn flop per layer", "bound": "tensor",
                                 "achieved": ach, "unit": "TFLOP/s", "peak": tpeak, "frac": ach / tpeak,
                                 "algorithmic_bytes": dense * len(refresh_steps)}
    elif "project_fp32" in per_kernel:
        pk = per_kernel["project_fp32"]
        achieved = flops_total / (pk["ms"] * 1e-3) / 1e12
        peak = 148 * 128 * 2 * 1.965e9 / 1e12      # fp32 FMA lanes x 2 flop x max SM clock
        roofline = {"kernel": "project_simt_kernel", "bound": "alu", "achieved": achieved,
                    "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "peak_source": "148 SMs x 128 fp32 lanes x 2 flop x 1.965 GHz", "traffic": None}
    hbm = {}
    if regular_steps or refresh_steps:
        rn = sum(min(wl.r, m) * n for _, m, n in wl.shapes) * wl.layers
        wbytes = 2 if wl.dtype == torch.bfloat16 else 4
        if "adam" in per_kernel:
            b = 24.0 * rn * steps
            hbm["adam"] = {"gbs": b / (per_kernel["adam"]["ms"] * 1e-3) / 1e9}
        if "scatter" in per_kernel:
            b = (4.0 + 2 * wbytes) * rn * steps
            hbm["scatter"] = {"gbs": b / (per_kernel["scatter"]["ms"] * 1e-3) / 1e9}
        if "adam_scatter" in per_kernel:
            b = (20.0 + 2 * wbytes) * rn * steps      # g, M, V in; M, V out; W in and out
            hbm["adam_scatter"] = {"gbs": b / (per_kernel["adam_scatter"]["ms"] * 1e-3) / 1e9}
        if "gather" in per_kernel:
            # a pre-pass (only when asked for): algorithmic bytes 2Tr in + 2Tr out per layer; what
            # it must touch is every 128-byte line of dY that holds a selected column, and the copy
            alg = sum(4.0 * wl.T * min(wl.r, m) for _, m, n in wl.shapes) * wl.layers * steps
            touched = sum(2.0 * wl.T * m * (1.0 - (1.0 - min(wl.r, m) / m) ** 64) +
                          2.0 * wl.T * min(wl.r, m) for _, m, n in wl.shapes) * wl.layers * steps
            sec = per_kernel["gather"]["ms"] * 1e-3
            hbm["gather"] = {"gbs": alg / sec / 1e9, "touched_gbs": touched / sec / 1e9,
                             "algorithmic_bytes": alg, "touched_bytes": touched}
        for v in hbm.values():
            v["frac_of_hbm_peak"] = v["gbs"] / peaks["hbm_gbs"]

    # ---- e2e: host buffers in, host result out, through the same public calls ----
    e2e = None
    if want_e2e:
        host_in = []
        for dY, X in block_in:
            hd = torch.empty(dY.shape, dtype=dY.dtype, pin_memory=True)
            hx = torch.empty(X.shape, dtype=X.dtype, pin_memory=True)
            hd.copy_(dY)
            hx.copy_(X)
            host_in.append((hd, hx))

        def like(t):      # same shape AND row pitch (empty_like would drop the padding)
            return torch.empty((t.shape[0], t.stride(0)), dtype=t.dtype, device=t.device)[:, : t.shape[1]]

        stage = [(like(d), like(x)) for d, x in block_in]
        max_rn = max(l.Gc.numel() for _, l in layers)
        host_out = [torch.empty(max_rn, dtype=torch.float32, pin_memory=True) for _ in wl.shapes]
        e2e_steps = min(steps, args.e2e_steps)
        h2d = sum(d.numel() * d.element_size() + x.numel() * x.element_size()
                  for d, x in host_in) * wl.layers
        d2h = sum(l.Gc.numel() * 4 for _, l in layers)

        def e2e_step():
            for st in streams[1:]:
                st.wait_stream(main_stream)
            for pi, layer in layers:
                sd, sx = stage[pi]
                with torch.cuda.stream(layer.stream):
                    sd.copy_(host_in[pi][0], non_blocking=True)
                    sx.copy_(host_in[pi][1], non_blocking=True)
                    layer.step(sd, sx)
                    host_out[pi][: layer.Gc.numel()].copy_(layer.Gc.view(-1), non_blocking=True)

        def e2e_join():
            for st in streams[1:]:
                main_stream.wait_stream(st)

        rewind()
        e2e_step()
        e2e_join()
        rewind()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
            e2e_join()
        e1.record()
        barrier()
        e2e_ms = aggregate_max(e0.elapsed_time(e1), dist if world > 1 else None)
        e2e_refresh = len([i for i in range(e2e_steps) if i % K == 0])
        e2e_flops = wl.flops_regular() * e2e_steps + wl.flops_refresh_extra() * e2e_refresh
        e2e = {"value": world * e2e_flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "ms_per_step": e2e_ms / e2e_steps}
        grass.grass_device_status()

    # ---- the oracle on the host cores, rank 0 of a single-GPU run only ----
    cpu_baseline = None
    if rank == 0 and world == 1 and want_cpu:
        T_gen = min(wl.T, 16384)            # about 10 s of oracle work on 16 host threads
        ins = [(syn.to_f32_numpy(d[:T_gen]), syn.to_f32_numpy(x[:T_gen])) for d, x in block_in]
        Ws = [syn.to_f32_numpy(layers[pi][1].W) for pi in range(len(wl.shapes))]
        sub = workloads.get(name, r=r, T=T_gen, layers=args.layers)
        res = time_oracle(sub, ins, Ws, budget_s=args.cpu_budget, steps=1, warmup=0)
        res["sample"] = res["sample"].replace(f"of {T_gen} tokens", f"of {wl.T} tokens")
        cpu_baseline = {"value": res["value"], "unit": "TFLOP/s", "cores": blas_threads(),
                        "kind": "oracle", "sample": res["sample"], "seconds": res["seconds"]}

    line = None
    if rank == 0:
        reg_ms = statistics.mean(step_ms[i] for i in regular_steps) if regular_steps else None
        ref_ms = statistics.mean(step_ms[i] for i in refresh_steps) if refresh_steps else None
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world,
            "steps": steps, "warmup": max(warmup, 3), "ms_per_step": total_ms / steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if wl.dtype == torch.bfloat16 else "f32", "data": "synthetic",
            "config": {"workload": wl.name, "layers": n_layers, "T": wl.T, "r": wl.r,
                       "selection": "top-r" if wl.method == grass.SEL_TOPR else "multinomial-norm",
                       "refresh_every": K, "refreshes_in_timed_region": len(refresh_steps),
                       "inputs": "one block of distinct dY/X reused by every block",
                       "l2": f"inputs {in_bytes / 1e6:.0f} MB per step, larger than the 126 MB L2",
                       "parallelism": "replicas" if world > 1 else "single GPU",
                       "streams": n_streams, "batched": bool(args.batched),
                       "flops": "2rTn per layer-step + 2mTn per refresh"},
            "us_per_layer_step_regular": None if reg_ms is None else 1e3 * reg_ms / n_layers,
            "us_per_layer_step_refresh": None if ref_ms is None else 1e3 * ref_ms / n_layers,
            "tflops_regular_steps": None if reg_ms is None else wl.flops_regular() / (reg_ms * 1e-3) / 1e12,
            "roofline": roofline, "hbm_kernels": hbm, "kernels": per_kernel,
            "profiled_pass_ms_per_step": prof_total / steps,
            "gpu_launches": launches, "e2e": e2e, "cpu_baseline": cpu_baseline, "clocks": clocks,
        }
    # release this workload's device memory before the next one is built
    del block_in, layers, units, wss
    torch.cuda.synchronize()
    torch.cuda.empty_cache()
    return line


def replica_command(args, argv):
    """The command that runs `--gpus N` as N replicas, one process per GPU (argv: this
    process's own arguments)."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
            f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1", "--master-port", str(port),
            os.path.abspath(__file__)] + list(argv)


def check_launch(args):
    """--check-launch: every rank joins a CPU (gloo) process group and rank 0 reports how many
    ranks the launch produced; touches no GPU."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    count = 1
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo")
        t = torch.ones(1, dtype=torch.float64)
        dist.all_reduce(t)
        count = int(t.item())
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"check_launch": True, "n_gpus": args.gpus, "ranks": count}))


def run_gpu(args):
    import torch
    import torch.distributed as dist
    import paper_2406_17660_b200 as grass

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(dev))
    grass.load_library()
    ctx = {"world": world, "rank": rank, "local_rank": local_rank, "dev": dev, "peaks": load_peaks()}

    line = measure_workload(ctx, args.workload, args.rank, args.steps, args.warmup,
                            not args.no_e2e, not args.no_cpu_baseline, args)
    # The other half of the target configuration (LLaMA-13B shapes, and r = 256), as short runs
    # with their own clock records; only beside the default workload.
    also = []
    if not args.no_also and args.workload == "llama7b_block" and args.rank is None and \
            args.tokens is None and args.layers is None:
        for name, r in (("llama13b_block", None), ("llama7b_block", 256), ("llama13b_block", 256)):
            sub = measure_workload(ctx, name, r, min(args.steps, 20), 3, False, False, args)
            if sub is not None:
                also.append({k: sub[k] for k in ("value", "unit", "steps", "ms_per_step", "config",
                                                 "us_per_layer_step_regular", "us_per_layer_step_refresh",
                                                 "tflops_regular_steps", "roofline", "hbm_kernels",
                                                 "kernels", "clocks")})
    if rank == 0:
        line["also"] = also
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="grass", choices=["grass", "reference"])
    ap.add_argument("--workload", default="llama7b_block")
    ap.add_argument("--rank", type=int, default=None, help="override r")
    ap.add_argument("--tokens", type=int, default=None, help="override T")
    ap.add_argument("--layers", type=int, default=None, help="override the number of blocks")
    ap.add_argument("--refresh-every", type=int, default=None, help="override K")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--streams", type=int, default=2, help="streams that layers alternate over")
    ap.add_argument("--unfused", action="store_true", help="separate Adam and apply kernels")
    ap.add_argument("--no-batched", dest="batched", action="store_false",
                    help="one set of launches per layer instead of per run of same-shaped layers")
    ap.add_argument("--cpu-budget", type=float, default=20.0)
    ap.add_argument("--launch-log", default=None,
                    help="write (kernel, microseconds) of every launch of the profiled pass to this file")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true",
                    help="skip the short extra runs (13B shapes, r = 256) beside the default workload")
    ap.add_argument("--check-launch", action="store_true",
                    help="only report how many ranks --gpus N produced (CPU, no GPU work)")
    args = ap.parse_args()
    # --gpus N without a launcher: start N replicas ourselves, one process per GPU
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(subprocess.call(replica_command(args, sys.argv[1:])))
    if args.check_launch:
        check_launch(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
