#!/usr/bin/env python
"""Benchmark of the L4Q linear layer hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole hot path over one batch of synthetic input:
for every L4Q linear of the workload, l4q_linear_fwd, l4q_linear_bwd (dX, dA,
dB, ds, db) and l4q_pack_int.  The default workload is the LLaMA-7B-shaped MLP
(up projection 4096 -> 11008 and down projection 11008 -> 4096, 8192 tokens,
rank 16, 4-bit, group 128), the layer the throughput target is quoted on.

Prints ONE JSON line (rank 0).  `value` is algorithmic TFLOP/s of the whole job
(6*M*o*i + 8*o*i*r flops per linear and step) with inputs resident in HBM;
`e2e` is the same metric with the step's activations (X, dY) copied from pinned
host memory and the parameter gradients copied back inside the timed region;
`sustained` is the device-resident figure again over at least 1.5 s of back-to-back
steps (the GPU at its power cap), against the sustained cuBLAS peak.  The
weight-tile launches (`kernels.dequant`, `kernels.pack`) are given against the
copy bandwidth and against the time of a bare TMA tile copy / read of the same
weights (`l4q_selftest_tile_copy`), the floor the memory system sets at that size.

N > 1 (launched by torch.distributed.run, one rank per GPU): data parallel over
tokens -- every rank runs the same layers on its own token batch (weak scaling)
and the parameter gradients of each layer are all-reduced (sum) over NCCL each step, as one bucket.

`--layer lora|qat_lora` runs the LoRA (Eq. 1-2) or QAT-LoRA (Sec. 3.1) layer instead, through
l4q_lora_linear_fwd / l4q_lora_linear_bwd, for the per-step cost comparison (no export step; the
flop count is that layer's own).  The default, `--layer l4q`, is the benchmark proper.

`--op extras` times the kernels outside the training step -- inference from the packed export (few tokens),
quantizer initialisation, the error sums and the AdamW update -- each against the HBM roofline, and prints its
own JSON line (not the benchmark line).

`--impl reference` times the fp64 CPU oracle (oracle/), as it stands, on the
host cores on a bounded slice of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2402_04902_b200 import synth  # noqa: E402

METRIC = "l4q_linear_fwd_bwd_tflops"
UNIT = "TFLOP/s"


def workloads() -> dict:
    return {
        "llama7b_mlp": [synth.CONFIG3A, synth.CONFIG3B],
        "llama7b_attn_proj": [synth.CONFIG2],
        "llama7b_mlp_3bit_r64": [synth.CONFIG4A, synth.CONFIG4B],
        "mistral7b_block": synth.mistral_block_layers(),
    }


def layer_flops(cfg, tokens=None, d_out=None, layer="l4q") -> float:
    """Algorithmic flops of fwd + bwd of one linear: three M*o*i products, merge twice, dA and dB.
    LoRA: two M*o*i products and six rank-side products; QAT-LoRA adds the full weight gradient."""
    M = cfg.tokens if tokens is None else tokens
    o = cfg.d_out if d_out is None else d_out
    if layer == "l4q":
        return 6.0 * M * o * cfg.d_in + 8.0 * o * cfg.d_in * cfg.rank
    side = 6.0 * M * cfg.rank * (cfg.d_in + o)
    return (4.0 if layer == "lora" else 6.0) * M * o * cfg.d_in + side


def peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", 0)),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


# --------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# --------------------------------------------------------------------------

class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, device_index: int, period_s: float = 0.005):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self) -> dict:
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------
# the oracle as CPU baseline / reference arm (bounded slice of one layer)
# --------------------------------------------------------------------------

def oracle_slice_step(cfg, arrays64, spec, rows: int):
    from oracle import l4q_oracle as orc
    a = arrays64
    sl = slice(0, rows)
    Y = orc.forward(spec, a["X"], a["W0"][sl], a["A"], a["B"][sl], a["s"][sl], a["b"][sl])
    g = orc.backward(spec, a["X"], a["dY"][:, sl], a["W0"][sl], a["A"], a["B"][sl], a["s"][sl], a["b"][sl])
    pk = orc.pack_int(spec, a["W0"][sl], a["A"], a["B"][sl], a["s"][sl], a["b"][sl])
    return Y, g, pk


def oracle_sample(cfg, tokens: int, rows: int, seed: int = 0):
    from oracle import l4q_oracle as orc
    small = cfg.with_(tokens=tokens)
    arrays = synth.make_layer_inputs(small, seed=seed)
    arrays64 = {k: np.asarray(v, dtype=np.float64) for k, v in arrays.items()}
    spec = orc.L4QSpec(rank=cfg.rank, alpha=cfg.alpha, bits=cfg.bits, group_size=cfg.group_size,
                       signed_grid=cfg.signed_grid)
    return arrays64, spec


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 0) for d in threadpool_info() if d.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return int(os.cpu_count() or 1)


def time_oracle(cfg, tokens: int, rows: int, steps: int, warmup: int):
    arrays64, spec = oracle_sample(cfg, tokens, rows)
    for _ in range(warmup):
        oracle_slice_step(cfg, arrays64, spec, rows)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_slice_step(cfg, arrays64, spec, rows)
    dt = (time.perf_counter() - t0) / max(steps, 1)
    flops = layer_flops(cfg, tokens=tokens, d_out=rows)
    return dt, flops


def run_reference(args, layers, wl_name):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = layers[0]
    tokens, rows = 512, max(cfg.d_out // 4 // 8 * 8, 8)
    dt, flops = time_oracle(cfg, tokens, rows, args.steps, args.warmup)
    value = flops / dt / 1e12
    sample = f"{cfg.name}: {tokens} of {cfg.tokens} tokens x first {rows} of {cfg.d_out} output rows, fwd+bwd+pack, fp64"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl_name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------

def run_ours(args, layers, wl_name):
    import torch
    import torch.distributed as dist

    from paper_2402_04902_b200 import binding as l4q
    from paper_2402_04902_b200 import build as l4q_build
    from paper_2402_04902_b200 import dp

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        l4q_build.build()
    if world > 1:
        dist.barrier()
    l4q.lib()

    # ---- synthetic layers: weights shared by all ranks, activations per rank (data parallel) ----
    L = []
    h2d = d2h = 0
    grad_names = ("dA", "dB") if args.layer == "lora" else ("dA", "dB", "ds", "db")
    kind = l4q.LORA_KINDS.get(args.layer)
    for li, cfg in enumerate(layers):
        arrays = synth.make_layer_inputs(cfg, seed=0, layer_id=li, need_acts=False)
        acts = synth.make_layer_acts(cfg, seed=1000 + rank, layer_id=li)
        host = {"X": torch.from_numpy(acts["X"]).to(torch.bfloat16).pin_memory(),
                "dY": torch.from_numpy(acts["dY"]).to(torch.bfloat16).pin_memory()}
        del acts
        d = l4q.to_device(cfg, arrays, device=dev)
        d["X"] = host["X"].to(dev)
        d["dY"] = host["dY"].to(dev)
        desc = l4q.make_desc(cfg)
        outs = l4q.alloc_outputs(cfg, device=dev)
        # the parameter gradients of a layer live in one buffer, so that N > 1 ranks exchange them in one all-reduce
        bucket, views = dp.alloc_grad_bucket({k: outs[k].shape for k in grad_names}, device=dev)
        outs.update(views)
        pk = l4q.alloc_pack_outputs(cfg, device=dev)
        if args.layer == "l4q":
            ws = l4q.alloc_workspace(desc, l4q.L4Q_OP_BWD, device=dev)
        else:
            ws = l4q.alloc_lora_workspace(desc, l4q.LORA_KINDS[args.layer], l4q.L4Q_OP_BWD, device=dev)
        grads_host = {k: torch.empty_like(outs[k], device="cpu").pin_memory() for k in grad_names}
        L.append(dict(cfg=cfg, desc=desc, d=d, outs=outs, pk=pk, ws=ws, host=host, grads_host=grads_host,
                      bucket=bucket))
        h2d += host["X"].numel() * 2 + host["dY"].numel() * 2
        d2h += sum(t.numel() * 4 for t in grads_host.values())

    # End-to-end mode double-buffers the activations: while a layer computes on one pair of device
    # buffers, a copy stream brings the next layer's (or next step's) X and dY from pinned host memory
    # into the other pair.  Every step still copies all of its inputs inside the timed region.
    copy_stream = torch.cuda.Stream(device=dev)
    for l in L:
        l["act"] = [{"X": l["d"]["X"], "dY": l["d"]["dY"]},
                    {"X": torch.empty_like(l["d"]["X"]), "dY": torch.empty_like(l["d"]["dY"])}]
        l["ready"] = [torch.cuda.Event(), torch.cuda.Event()]
        l["free"] = [None, None]                     # recorded when the compute stream is done with the pair

    def prefetch(l, par):
        with torch.cuda.stream(copy_stream):
            if l["free"][par] is not None:
                copy_stream.wait_event(l["free"][par])
            l["act"][par]["X"].copy_(l["host"]["X"], non_blocking=True)
            l["act"][par]["dY"].copy_(l["host"]["dY"], non_blocking=True)
            l["ready"][par].record(copy_stream)

    e2e_units = {"n": 0}                             # steps run in end-to-end mode so far (buffer parity)

    def step(e2e: bool, last: bool = True):
        par = e2e_units["n"] % 2 if e2e else 0
        for li, l in enumerate(L):
            d, o, pk = dict(l["d"]), l["outs"], l["pk"]
            if e2e:
                if li == 0 and not e2e_units.get("primed"):
                    prefetch(l, par)                 # pipeline fill: nothing to overlap the first copy with
                    e2e_units["primed"] = True
                if li + 1 < len(L):
                    prefetch(L[li + 1], par)
                elif not last:
                    prefetch(L[0], par ^ 1)
                torch.cuda.current_stream().wait_event(l["ready"][par])
                d["X"], d["dY"] = l["act"][par]["X"], l["act"][par]["dY"]
            if kind is None:
                l4q.l4q_linear_fwd(l["desc"], d["X"], d["W0"], d["A"], d["B"], d["s"], d["b"], o["Y"], l["ws"])
                l4q.l4q_linear_bwd(l["desc"], d["X"], d["dY"], d["W0"], d["A"], d["B"], d["s"], d["b"],
                                   o["dX"], o["dA"], o["dB"], o["ds"], o["db"], l["ws"])
                l4q.l4q_pack_int(l["desc"], d["W0"], d["A"], d["B"], d["s"], d["b"], pk["codes"], pk["s16"],
                                 pk["b16"], l["ws"])
            else:
                qat = args.layer == "qat_lora"
                sq, bq = (d["s"], d["b"]) if qat else (None, None)
                l4q.l4q_lora_linear_fwd(l["desc"], kind, d["X"], d["W0"], d["A"], d["B"], sq, bq, o["Y"], l["ws"])
                l4q.l4q_lora_linear_bwd(l["desc"], kind, d["X"], d["dY"], d["W0"], d["A"], d["B"], sq, bq, o["dX"],
                                        o["dA"], o["dB"], o["ds"] if qat else None, o["db"] if qat else None,
                                        l["ws"])
            if world > 1:
                dp.allreduce_grad_bucket(l["bucket"])
            if e2e:
                ev = torch.cuda.Event()
                ev.record()
                l["free"][par] = ev
                for k in grad_names:
                    l["grads_host"][k].copy_(o[k], non_blocking=True)
        if e2e:
            e2e_units["n"] += 1
            if last:
                e2e_units["primed"] = False

    def timed(e2e: bool, steps: int, warmup: int):
        for i in range(warmup):
            step(e2e, last=(i == warmup - 1))
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for i in range(steps):
            step(e2e, last=(i == steps - 1))
        ev1.record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        ms = torch.tensor([ev0.elapsed_time(ev1)], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        return float(ms.item())

    flops_step_rank = sum(layer_flops(l["cfg"], layer=args.layer) for l in L)
    tokens_step_rank = L[0]["cfg"].tokens

    # ---- device-resident timing, with per-kernel events and clock samples ----
    launches0 = l4q.l4q_launch_count()
    l4q.l4q_profile_enable(True)
    for _ in range(args.warmup):
        step(False)
    torch.cuda.synchronize()
    l4q.l4q_profile_enable(False)
    l4q.l4q_profile_enable(True)
    launches0 = l4q.l4q_launch_count()
    with ClockSampler(local_rank) as clk:
        ms_total = timed(False, args.steps, 0)
    launches = l4q.l4q_launch_count() - launches0
    prof = l4q.l4q_profile_read()
    l4q.l4q_profile_enable(False)
    l4q.l4q_check()
    ms_step = ms_total / args.steps
    value = world * flops_step_rank / (ms_step * 1e-3) / 1e12

    # ---- the same step for at least 1.5 s: the GPU reaches its power cap and settles at its sustained clock ----
    n_sus = max(args.steps, int(args.sustained_seconds * 1e3 / ms_step) + 1)
    with ClockSampler(local_rank) as clk_sus:
        ms_sus = timed(False, n_sus, 0) / n_sus
    sus_value = world * flops_step_rank / (ms_sus * 1e-3) / 1e12
    l4q.l4q_check()

    # ---- the memory-system floor of the weight-tile launches: a bare TMA tile copy / read of each layer's weight ----
    floor_us = {"read": 0.0, "copy": 0.0}
    if kind is None:
        scratch = [torch.empty_like(l["d"]["W0"]) for l in L]
        for mode in ("read", "copy"):
            def sweep():                                 # layer after layer, as in a step: each weight comes from HBM
                for l, sc in zip(L, scratch):
                    l4q.l4q_selftest_tile_copy(l["d"]["W0"], sc if mode == "copy" else None)
            sweep()
            torch.cuda.synchronize()
            l4q.l4q_profile_enable(False)
            l4q.l4q_profile_enable(True)
            for _ in range(5):
                sweep()
            torch.cuda.synchronize()
            n_, ms_ = l4q.l4q_profile_read()["tile_copy"]
            l4q.l4q_profile_enable(False)
            floor_us[mode] = ms_ / max(n_, 1) * 1e3 * len(L)
        del scratch
        l4q.l4q_check()

    # ---- end to end: host -> device copies of X, dY and device -> host of the gradients, every step ----
    ms_e2e = timed(True, args.steps, max(1, min(args.warmup, 2))) / args.steps
    e2e_value = world * flops_step_rank / (ms_e2e * 1e-3) / 1e12
    l4q.l4q_check()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (live CUDA-event times from the timed region) ----
    pk_ = peaks()
    gemm_flops = {"gemm_fwd": 0.0, "gemm_dgrad": 0.0, "gemm_wgrad": 0.0}
    pack_bytes = deq_bytes = 0.0
    for l in L:
        c = l["cfg"]
        mm = 2.0 * c.tokens * c.d_out * c.d_in
        gemm_flops["gemm_fwd"] += mm
        gemm_flops["gemm_dgrad"] += mm
        gemm_flops["gemm_wgrad"] += mm + 4.0 * c.d_out * c.d_in * c.rank      # G tiles + the dA, dB contractions
        G = c.d_in // c.group_size
        small = 4.0 * c.rank * (c.d_in + c.d_out)
        pack_bytes += c.d_out * c.d_in * (2 + c.bits / 8) + c.d_out * G * 12 + small
        # two launches per step: forward (W0 in, W_q out) and backward (W0 in, W_q and the fp16 STE factors out)
        deq_bytes += (c.d_out * c.d_in * 4 + c.d_out * G * 8 + small) + (c.d_out * c.d_in * 6 + c.d_out * G * 8 + small)
    kernels = {}
    for name, (n, ms) in prof.items():
        if n:
            kernels[name] = {"launches": n, "total_ms": ms, "avg_ms": ms / n}
    total_kernel_ms = sum(k["total_ms"] for k in kernels.values()) or 1.0
    for name, k in kernels.items():
        k["share"] = k["total_ms"] / total_kernel_ms
        steps_timed = args.steps
        if name in gemm_flops:
            k["tflops"] = gemm_flops[name] * steps_timed / (k["total_ms"] * 1e-3) / 1e12
        elif name == "pack":
            k["gbs"] = pack_bytes * steps_timed / (k["total_ms"] * 1e-3) / 1e9
            k["frac_hbm"] = k["gbs"] / pk_["hbm_gbs"]
            # a bare TMA read of the same weights (one launch per layer, nothing else to do) takes floor_us
            k["floor_us_per_step"] = floor_us["read"]
            k["frac_of_floor"] = floor_us["read"] * 1e-3 * steps_timed / k["total_ms"] if floor_us["read"] else None
        elif name == "dequant":
            k["gbs"] = deq_bytes * steps_timed / (k["total_ms"] * 1e-3) / 1e9
            k["frac_hbm"] = k["gbs"] / pk_["hbm_gbs"]
            # forward + backward launch of every layer, each at least a bare TMA copy of the weight
            k["floor_us_per_step"] = 2 * floor_us["copy"]
            k["frac_of_floor"] = 2 * floor_us["copy"] * 1e-3 * steps_timed / k["total_ms"] if floor_us["copy"] else None
    dominant = max(kernels, key=lambda n: kernels[n]["total_ms"]) if kernels else None
    traffic = None
    tpath = os.path.join(ROOT, "profiles", f"dram_traffic_{wl_name}.txt")
    if os.path.exists(tpath):
        for ln in open(tpath):
            f = ln.split()
            if len(f) == 2 and f[0] == dominant:
                traffic = float(f[1])
    roofline = None
    if dominant in gemm_flops:
        ach = kernels[dominant]["tflops"]
        roofline = {"kernel": dominant, "bound": "tensor", "achieved": ach, "peak": pk_["bf16_tflops"],
                    "unit": "TFLOP/s", "frac": ach / pk_["bf16_tflops"], "traffic": traffic,
                    "peak_source": pk_["source"] + " burst cuBLAS bf16",
                    "frac_of_sustained": (ach / pk_["bf16_tflops_sustained"]) if pk_["bf16_tflops_sustained"] else None}
    elif dominant is not None:
        ach = kernels[dominant].get("gbs", 0.0)
        roofline = {"kernel": dominant, "bound": "hbm", "achieved": ach, "peak": pk_["hbm_gbs"], "unit": "GB/s",
                    "frac": ach / pk_["hbm_gbs"], "traffic": traffic, "peak_source": pk_["source"] + " copy"}

    # ---- CPU baseline: the oracle, as it stands, on a bounded slice of the first layer ----
    cfg0 = L[0]["cfg"]
    tokens_s, rows_s = 512, max(cfg0.d_out // 4 // 8 * 8, 8)
    dt, fl = time_oracle(cfg0, tokens_s, rows_s, steps=2, warmup=1)
    cpu = {"value": fl / dt / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
           "sample": f"{cfg0.name}: {tokens_s} of {cfg0.tokens} tokens x first {rows_s} of {cfg0.d_out} output rows, "
                     f"fwd+bwd+pack, fp64, {dt:.2f} s per pass"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": wl_name, "layer": args.layer,
                   "layers": [f"{l['cfg'].d_in}->{l['cfg'].d_out}" for l in L],
                   "tokens_per_gpu": tokens_step_rank, "rank": L[0]["cfg"].rank, "bits": L[0]["cfg"].bits,
                   "group_size": L[0]["cfg"].group_size, "parallelism": f"dp{world}",
                   "l2": "inputs larger than L2 (no flush)"},
        "tokens_per_s": world * tokens_step_rank / (ms_step * 1e-3),
        "frac_of_bf16_peak": value / world / pk_["bf16_tflops"],
        "clocks": clk.summary(),
        "sustained": {"value": sus_value, "unit": UNIT, "ms_per_step": ms_sus, "steps": n_sus,
                      "seconds": ms_sus * n_sus * 1e-3, "clocks": clk_sus.summary(),
                      "frac_of_sustained_peak": (sus_value / world / pk_["bf16_tflops_sustained"])
                      if pk_["bf16_tflops_sustained"] else None},
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h,
                "h2d_what": "X and dY of every layer (bf16, pinned host memory), every step",
                "d2h_what": "the parameter gradients " + ", ".join(grad_names) + " of every layer (fp32); Y, dX and the "
                            "packed export stay on the device (the next layer and the optimizer consume them there)"},
        "gpu_launches": int(launches),
        "kernels": kernels,
        "roofline": roofline,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------
# kernels outside the training step (--op extras)
# --------------------------------------------------------------------------

def run_extras(args):
    """Device times (the library's per-launch CUDA events) of l4q_linear_infer, l4q_init_params, l4q_quant_error
    and l4q_adamw_step on LLaMA-7B-shaped operands, with the bytes each must move.  Weights are rotated over
    enough copies to exceed L2, as the layers of a model would."""
    import torch

    from paper_2402_04902_b200 import binding as l4q
    from paper_2402_04902_b200 import build as l4q_build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    l4q_build.build()
    l4q.lib()
    pk_ = peaks()
    dev = torch.device("cuda", 0)
    reps = max(args.steps, 5)
    out = {}

    def timed(name_key, fn, n_calls):
        for _ in range(args.warmup):
            fn(0)
        torch.cuda.synchronize()
        l4q.l4q_profile_enable(False)
        l4q.l4q_profile_enable(True)
        for k in range(n_calls):
            fn(k)
        torch.cuda.synchronize()
        n, ms = l4q.l4q_profile_read()[name_key]
        l4q.l4q_profile_enable(False)
        l4q.l4q_check()
        return ms / max(n, 1) * 1e3                               # us per launch

    L2_BYTES = 126e6
    # ---- inference from the export (App. F): few tokens, weights streamed from HBM ----
    for d_in, d_out in ((4096, 11008), (11008, 4096), (4096, 4096)):
        cfg = synth.CONFIG3A.with_(name=f"infer_{d_in}x{d_out}", d_in=d_in, d_out=d_out, tokens=64)
        arrays = synth.make_layer_inputs(cfg, seed=0, need_acts=False)
        d = l4q.to_device(cfg, arrays, device=dev)
        desc = l4q.make_desc(cfg)
        pk = l4q.alloc_pack_outputs(cfg, device=dev)
        l4q.l4q_pack_int(desc, d["W0"], d["A"], d["B"], d["s"], d["b"], pk["codes"], pk["s16"], pk["b16"])
        wbytes = pk["codes"].numel() * 4 + pk["s16"].numel() * 4
        copies = int(L2_BYTES * 1.5 // wbytes) + 1
        ring = [{k: v.clone() for k, v in pk.items()} for _ in range(copies)]
        # the unquantized layer for comparison: the same product with a dense bf16 weight through cuBLAS
        # (torch.matmul), weights rotated the same way, CUDA events around every call
        dense_copies = int(L2_BYTES * 1.5 // (d_in * d_out * 2)) + 1
        dense = [d["W0"].clone() for _ in range(dense_copies)]

        def dense_us(X, n_calls):
            for k in range(args.warmup):
                torch.matmul(X, dense[k % dense_copies].t())
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_calls)]
            torch.cuda.synchronize()
            for k, (e0, e1) in enumerate(evs):
                e0.record()
                torch.matmul(X, dense[k % dense_copies].t())
                e1.record()
            torch.cuda.synchronize()
            return sum(e0.elapsed_time(e1) for e0, e1 in evs) / n_calls * 1e3

        for tokens in (1, 2, 16, 64):
            dsc = l4q.make_desc(cfg, tokens=tokens)
            X = torch.randn(tokens, d_in, device=dev).to(torch.bfloat16)
            Y = torch.empty(tokens, d_out, dtype=torch.bfloat16, device=dev)

            def call(k, dsc=dsc, X=X, Y=Y):
                w = ring[k % copies]
                l4q.l4q_linear_infer(dsc, X, w["codes"], w["s16"], w["b16"], Y)

            us = timed("infer", call, reps * copies)
            nbytes = wbytes + tokens * (d_in + d_out) * 2
            out[f"infer_{d_in}x{d_out}_t{tokens}"] = {"us": us, "bytes": nbytes, "gbs": nbytes / us / 1e3,
                                                       "frac_hbm": nbytes / us / 1e3 / pk_["hbm_gbs"],
                                                       "dense_bf16_bytes": d_in * d_out * 2,
                                                       "dense_bf16_cublas_us": dense_us(X, reps * dense_copies)}
        del ring, dense

    # ---- initialisation of s, b (App. B) and the error sums (Table 4): one pass over a bf16 weight ----
    cfg = synth.CONFIG3A
    arrays = synth.make_layer_inputs(cfg, seed=0, need_acts=False)
    d = l4q.to_device(cfg, arrays, device=dev)
    desc = l4q.make_desc(cfg)
    wbytes = cfg.d_out * cfg.d_in * 2
    copies = int(L2_BYTES * 1.5 // wbytes) + 1
    Ws = [d["W0"].clone() for _ in range(copies)]
    G = cfg.d_in // cfg.group_size
    s_out = torch.empty(cfg.d_out, G, device=dev)
    b_out = torch.empty(cfg.d_out, G, device=dev)
    for method in ("lsq+", "symm", "asymm", "l4q"):
        us = timed("init", lambda k, m=method: l4q.l4q_init_params(desc, Ws[k % copies], m, s_out, b_out), reps * copies)
        nbytes = wbytes + 2 * s_out.numel() * 4
        out[f"init_{method}_4096x11008"] = {"us": us, "bytes": nbytes, "gbs": nbytes / us / 1e3,
                                            "frac_hbm": nbytes / us / 1e3 / pk_["hbm_gbs"]}
    err = torch.zeros(2, dtype=torch.float64, device=dev)
    us = timed("error", lambda k: l4q.l4q_quant_error(desc, Ws[k % copies], d["A"], d["B"], d["s"], d["b"], err),
               reps * copies)
    nbytes = wbytes + 2 * s_out.numel() * 4
    out["quant_error_4096x11008"] = {"us": us, "bytes": nbytes, "gbs": nbytes / us / 1e3,
                                     "frac_hbm": nbytes / us / 1e3 / pk_["hbm_gbs"]}
    del Ws

    # ---- AdamW (App. D): 4 reads + 3 writes of fp32 per element ----
    n = 64 * 1024 * 1024
    p_, g_, m_, v_ = (torch.randn(n, device=dev) for _ in range(4))
    v_.abs_()
    us = timed("adamw", lambda k: l4q.l4q_adamw_step(p_, g_, m_, v_, k + 1, 1e-4), reps)
    out["adamw_64Mi"] = {"us": us, "bytes": 28 * n, "gbs": 28 * n / us / 1e3, "frac_hbm": 28 * n / us / 1e3 / pk_["hbm_gbs"]}
    # the size the layer really has: A, B, s, b of the 4096 -> 11008 linear
    n2 = cfg.rank * (cfg.d_in + cfg.d_out) + 2 * cfg.d_out * G
    us = timed("adamw", lambda k: l4q.l4q_adamw_step(p_[:n2], g_[:n2], m_[:n2], v_[:n2], k + 1, 1e-4), reps * 8)
    out["adamw_layer_params"] = {"us": us, "elements": n2, "bytes": 28 * n2}
    # the same parameters as the four tensors they are (A, B, s, b), one launch each against one launch for all
    sizes = [cfg.rank * cfg.d_in, cfg.d_out * cfg.rank, cfg.d_out * G, cfg.d_out * G]
    offs = np.cumsum([0] + sizes)
    views = [(p_[a:b], g_[a:b], m_[a:b], v_[a:b]) for a, b in zip(offs[:-1], offs[1:])]

    def four_launches(k):
        for t in views:
            l4q.l4q_adamw_step(*t, k + 1, 1e-4)

    us4 = timed("adamw", four_launches, reps * 8) * 4            # per-launch average x 4 launches
    us1 = timed("adamw", lambda k: l4q.l4q_adamw_step_multi(views, k + 1, 1e-4), reps * 8)
    out["adamw_layer_A_B_s_b"] = {"us_four_launches": us4, "us_one_launch": us1, "elements": int(offs[-1])}

    print(json.dumps({"op": "extras", "unit": "us per launch (CUDA events around each launch)", "hbm_peak_gbs": pk_["hbm_gbs"],
                      "peak_source": pk_["source"], "l2": "weights rotated over copies totalling 1.5x L2",
                      "kernels": out}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="llama7b_mlp", choices=sorted(workloads()))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layer", default="l4q", choices=["l4q", "lora", "qat_lora"],
                    help="l4q = the benchmark; lora / qat_lora = the comparison layers (ours arm only)")
    ap.add_argument("--sustained-seconds", type=float, default=1.5,
                    help="length of the second, sustained timed region (0: as many steps as --steps; for profiler captures)")
    ap.add_argument("--op", default="train", choices=["train", "extras"],
                    help="train = the benchmark; extras = inference / initialisation / error sums / AdamW kernels")
    args = ap.parse_args()
    if args.op == "extras":
        if int(os.environ.get("RANK", "0")) == 0:
            run_extras(args)
        return
    layers = workloads()[args.workload]
    if args.impl == "reference":
        run_reference(args, layers, args.workload)
    else:
        run_ours(args, layers, args.workload)


if __name__ == "__main__":
    main()
