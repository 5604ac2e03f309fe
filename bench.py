#!/usr/bin/env python
"""Benchmark of the CafeQ optimisation hot path on B200.

One "step" = one forward+backward of the paper's training objective over every matrix of one
Gemma-2-9B-shaped decoder layer (q, k, gate: single block-diagonal transform, Eq. 4 surrogate;
v-o and up-down: paired transform, LogSumExp surrogate with the orthonormality penalty), 3-bit,
group 128, block 256 (198 180 864 weights).  Inputs are seeded synthetic stand-ins for the trained
weights, resident in HBM when the timed region starts; the layer (396 MB) is larger than L2.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 3] [--exact]

Prints one JSON line (rank 0).  With N > 1 (torchrun) every rank optimises its own layer; there is no
data-path collective (layers are independent problems), only a barrier and a max-over-ranks of the time.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import cafeq_synth as syn  # noqa: E402

METRIC = "proxy-loss fwd+bwd steps/s (Gemma2-9B-shaped layer)"
UNIT = "steps/s"


def profiled_traffic():
    """DRAM bytes per launch of the transform pass from the committed ncu summary, or None once the kernel source
    differs from the one that was profiled."""
    import hashlib
    import re
    try:
        txt = open(os.path.join(ROOT, "profiles", "bd_pass_9b_layer.md")).read()
        src = open(os.path.join(ROOT, "paper_2511_19705_b200", "csrc", "kernels_fused.cuh"), "rb").read()
        sha = re.search(r"kernel_source_sha256:\s*([0-9a-f]+)", txt).group(1)
        if hashlib.sha256(src).hexdigest() != sha:
            return None
        return float(re.search(r"traffic_bytes_per_launch:\s*([0-9.e+]+)", txt).group(1))
    except Exception:
        return None


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"], bf16_sus=d.get("bf16_tflops_sustained"),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_sus=1400.0, source="fallback")


# ------------------------------------------------------------------------------------------ inputs
def host_layer(config: int, layer: int):
    """Seeded host copies of one layer: list of (kind, name, arrays...) in bf16 bits / fp32."""
    spec = syn.layer_spec(config)
    k = spec["k"]
    singles, pairs = [], []
    for name, d_out, d_in in spec["singles"]:
        singles.append((name, syn.make_weight(config, name, d_out, d_in, layer),
                        syn.make_transform(name, d_in // k, k, layer)))
    for pname, (n1, h, d1), (n2, d3, rh), kb, r in spec["pairs"]:
        pairs.append((pname, syn.make_weight(config, n1, h, d1, layer), syn.make_weight(config, n2, d3, rh, layer),
                      syn.make_transform(n1, h // kb, kb, layer), r))
    return spec, singles, pairs


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.rows, self.proc = index, [], None

    def run(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            for line in self.proc.stdout:
                self.rows.append([c.strip() for c in line.split(",")])
        except Exception:
            pass

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
        self.join(timeout=2)
        sm, reasons, mx = [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
                for nme, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(nme)
            except Exception:
                continue
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=mx, reasons=sorted(reasons),
                    samples=len(sm))


# ------------------------------------------------------------------------------------------ reference arm / CPU baseline
def oracle_sample_step(spec, singles, pairs, frac: int, ste: bool = False):
    """One oracle fwd+bwd over a 1/frac sample of every matrix of the layer (free-axis slices)."""
    from oracle import cafeq_oracle as orc
    bits, group = spec["bits"], spec["group"]
    for name, Wb, M in singles:
        rows = max(1, Wb.shape[0] // frac)
        W = syn.bf16_bits_to_f64(Wb[:rows])
        f = orc.single_forward(W, M, bits, group, "in")
        if ste:
            orc.single_grad_ste(W, f, bits, group, "in")
        else:
            orc.single_grad_surrogate(W, f, group, "in")
    for pname, W1b, W2b, M, r in pairs:
        c1 = max(group, (W1b.shape[1] // frac) // group * group)
        r2 = max(1, W2b.shape[0] // frac)
        W1 = syn.bf16_bits_to_f64(np.ascontiguousarray(W1b[:, :c1]))
        W2 = syn.bf16_bits_to_f64(W2b[:r2])
        f = orc.pair_forward(W1, W2, M, bits, group, group, r, 5.0, 0.1, ste)
        if ste:
            orc.pair_grad_pqe_ste(W1, W2, f, bits, group, group)
        else:
            orc.pair_grad_lse(W1, W2, f, group, group)


def time_oracle(spec, singles, pairs, frac, steps, warmup, ste=False):
    for _ in range(warmup):
        oracle_sample_step(spec, singles, pairs, frac, ste)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_sample_step(spec, singles, pairs, frac, ste)
    dt = (time.perf_counter() - t0) / steps
    return dt, 1.0 / (dt * frac)


def cpu_threads():
    try:
        import threadpoolctl
        n = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] + [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


# ------------------------------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--exact", action="store_true", help="also evaluate the quantised losses (Eq. 3 / Eq. 5) every step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--serial", action="store_true", help="one stream and one shared workspace for the whole layer")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of a CUDA-graph replay")
    ap.add_argument("--sample-frac", type=int, default=32)
    ap.add_argument("--loss", default="surrogate", choices=["surrogate", "ste"],
                    help="surrogate: Eq. 4 (singles) + LogSumExp (pairs), the paper's objectives; ste: straight-through "
                         "gradients of the quantised losses themselves (Eq. 3 singles, Eq. 5 pairs)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    workload = {3: "gemma2-9b-layer", 1: "config1-256x512", 2: "gemma2-2b-mlp-pair", 5: "gemma2-27b-layer"}.get(
        args.config, f"config{args.config}")
    cfg_json = dict(workload=workload, config=args.config, weights_per_step=None, bits=None, group=None, block=None,
                    loss="surrogate(Eq.4)+LSE" + ("+exact" if args.exact else ""),
                    l2_policy="inputs (one layer) larger than L2", parallelism=f"layers x{world}")
    if args.loss == "ste":
        cfg_json["loss"] = "straight-through: L2 (Eq.3) singles + PQE^2 (Eq.5) pairs"

    if args.impl == "reference":
        if rank != 0:
            return
        spec, singles, pairs = host_layer(args.config, 0)
        dt, sps = time_oracle(spec, singles, pairs, args.sample_frac, max(1, args.steps), min(args.warmup, 1),
                              args.loss == "ste")
        nw = sum(w.size for _, w, _ in singles) + sum(a.size + b.size for _, a, b, _, _ in pairs)
        cfg_json.update(weights_per_step=int(nw), bits=spec["bits"], group=spec["group"], block=spec["k"])
        sample = f"1/{args.sample_frac} of the rows (free axis) of every matrix of the layer per step, extrapolated linearly"
        print(json.dumps(dict(metric=METRIC, value=sps, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                              ms_per_step=1e3 / sps, higher_is_better=True, scaling="weak", vs_baseline=None,
                              dtype="f64", data="synthetic", config=cfg_json, impl="reference",
                              cpu_baseline=dict(value=sps, unit=UNIT, cores=cpu_threads(), kind="oracle", sample=sample),
                              e2e=dict(value=sps, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))))
        return

    import torch
    import paper_2511_19705_b200 as cq
    from paper_2511_19705_b200.layer import LayerStep, PairProblem, SingleProblem

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    from paper_2511_19705_b200 import shard
    my_layer = shard.layers_of_rank(world, world, rank)[0]     # weak scaling: one layer per rank, no data-path collective
    spec, singles, pairs = host_layer(args.config, my_layer)
    bits, group = spec["bits"], spec["group"]

    def up_bf16(b):
        return torch.from_numpy(b.view(np.int16)).to(dev).view(torch.bfloat16)

    ste = args.loss == "ste"
    sp = [SingleProblem(n, up_bf16(W), torch.from_numpy(M).to(dev), bits, group,
                        loss_kind=cq.LOSS_L2_STE if ste else cq.LOSS_SURROGATE) for n, W, M in singles]
    pp = [PairProblem(n, up_bf16(W1), up_bf16(W2), torch.from_numpy(M).to(dev), bits, group, group, r, lr=1e-4,
                      loss_kind=cq.LOSS_PQE_STE if ste else cq.LOSS_LSE) for n, W1, W2, M, r in pairs]

    if args.exact:
        for p in pp:
            p.P = cq.cafeq_pair_product(p.W1, p.W2, k=p.M.shape[-1], replicas=p.d2.replicas)
    layer = LayerStep(sp, pp, parallel=not args.serial)
    cfg_json.update(weights_per_step=int(layer.weights), bits=bits, group=group, block=spec["k"])

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # gradient-descent step size of the single matrices: a small fixed fraction of the first gradient's largest
    # entry, so that the transforms move every step (the block inverse has real work) without leaving the
    # neighbourhood of the initial rotations during the run
    layer.step(0)
    torch.cuda.synchronize()
    for p in sp:
        p.cfg.lr = float(1e-3 / max(float(p.grad.abs().max().item()), 1e-30))

    def one_step():
        layer.opt_step(eval_exact=args.exact)

    for _ in range(max(args.warmup, 3)):
        one_step()
    sync_all()
    assert all(s == 0 for s in layer.statuses()), layer.statuses()

    # ---- pass 1: eager launches on one stream with the library's in-stream event pairs around its main kernels
    par = layer.parallel
    layer.parallel = False
    n_timed = 64 * args.steps
    cq.timer_begin(n_timed)
    l0 = cq.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    e0.record()
    for _ in range(args.steps):
        one_step()
    e1.record()
    sync_all()
    launches = cq.launch_count() - l0
    ms_eager = e0.elapsed_time(e1)
    kms, kinds = cq.timer_read(n_timed)
    layer.parallel = par

    # ---- pass 2 (the reported value): the same step captured once into a CUDA graph and replayed
    graph = None
    if not args.no_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                one_step()
        except Exception as exc:  # capture refused: report the eager number
            print(f"graph capture failed: {exc}", file=sys.stderr)
            graph = None
            torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    if graph is not None:
        for _ in range(3):
            graph.replay()
        sync_all()
        e0.record()
        for _ in range(args.steps):
            graph.replay()
        e1.record()
        sync_all()
        ms = e0.elapsed_time(e1)
    else:
        sync_all()
        e0.record()
        for _ in range(args.steps):
            one_step()
        e1.record()
        sync_all()
        ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    assert all(s == 0 for s in layer.statuses()), layer.statuses()
    ms = shard.max_over_ranks(ms, dev)
    ms_per_step = ms / args.steps
    value = world * args.steps / (ms * 1e-3)
    cfg_json.update(launch="cuda_graph_replay" if graph is not None else "eager",
                    streams=len(layer.streams) if layer.parallel else 1, eager_ms_per_step=ms_eager / args.steps,
                    step="fwd+bwd+update (GD singles, Adam pairs), warm-started block inverse")

    # ---- roofline of the dominant kernel (the block-diagonal transform pass), from the in-stream event pairs
    peaks = load_peaks()
    k = spec["k"]
    by_kind = {}
    for d, kd in zip(kms, kinds):
        by_kind.setdefault(kd, []).append(d)
    names = {1: "transform_pass_generic", 2: "sparse_backward", 3: "block_inverse", 4: "pair_product",
             5: "transform_pass_tcgen05"}
    kernel_ms = {names.get(kd, str(kd)): dict(launches_per_step=len(v) / args.steps, ms_per_step=sum(v) / args.steps)
                 for kd, v in by_kind.items()}
    if "sparse_backward" in kernel_ms and k in (128, 256):
        # the backward is a second tensor-core product over the same weights: 2k flop per weight of algorithmic
        # work, issued twice (the routed coefficients are a two-term bf16 split)
        sb = kernel_ms["sparse_backward"]
        sb["algorithmic_tflops"] = 2.0 * k * layer.weights / (sb["ms_per_step"] * 1e-3) / 1e12
        sb["issued_tflops"] = 2.0 * sb["algorithmic_tflops"]
        sb["kernel"] = "bd_bwd_kernel (tcgen05)"
    roof = None
    tk = max((kd for kd in (1, 5) if kd in by_kind), key=lambda kd: sum(by_kind[kd]), default=None)
    if tk is not None:
        tp = by_kind[tk]
        t_pass = sum(tp) / args.steps * 1e-3                    # seconds of transform passes per step
        passes = len(tp) / args.steps / 7.0                     # passes over the layer per step
        flops = 2.0 * k * layer.weights * passes                # 2k flop per weight per pass
        byts = 2.0 * layer.weights * passes                     # bf16 weights read once per pass
        tc_peak = peaks["bf16_sus"] or peaks["bf16_tflops"]
        t_hbm, t_tc = byts / (peaks["hbm_gbs"] * 1e9), flops / (tc_peak * 1e12)
        if t_tc >= t_hbm:
            ach = flops / t_pass / 1e12
            roof = dict(bound="tensor", achieved=ach, peak=tc_peak, unit="TFLOP/s", frac=ach / tc_peak, traffic=None)
        else:
            ach = byts / t_pass / 1e9
            roof = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"],
                        traffic=None)
        tb = profiled_traffic() if tk == 5 else None  # the committed ncu capture is of the tcgen05 pass
        roof["traffic"] = tb
        roof["traffic_note"] = "ncu dram bytes read+written per launch (mean over the 7 launches of a step)" if tb else None
        roof["algorithmic_bytes_per_launch"] = byts / (len(tp) / args.steps)
        roof.update(kernel=names[tk], peak_source=peaks["source"] + (" sustained" if roof["bound"] == "tensor" else ""),
                    launches_per_step=len(tp) / args.steps, avg_launch_ms=sum(tp) / len(tp),
                    algorithmic_gb_per_step=byts / 1e9, algorithmic_tflop_per_step=flops / 1e12,
                    hbm_gbs_achieved=byts / t_pass / 1e9)
        sbk = kernel_ms.get("sparse_backward")
        if sbk:
            # forward pass + sparse backward taken together against the same algorithmic work (one 2k-flop-per-weight
            # transform and one read of the weights per step): what a single fused kernel would be held to
            t_fb = t_pass + sbk["ms_per_step"] * 1e-3
            roof["fwd_plus_bwd"] = dict(ms_per_step=t_fb * 1e3, achieved=flops / t_fb / 1e12, unit="TFLOP/s",
                                        frac=flops / t_fb / 1e12 / tc_peak)

    # ---- end to end through the C ABI with host buffers (pinned): H2D of every weight and transform, the step,
    #      D2H of the loss histories and the updated transforms, every step
    e2e = None
    if not args.no_e2e and rank == 0:
        hostW = [t.cpu().pin_memory() for p in sp for t in (p.W, p.M)] + \
                [t.cpu().pin_memory() for p in pp for t in (p.W1, p.W2, p.M)]
        devW = [t for p in sp for t in (p.W, p.M)] + [t for p in pp for t in (p.W1, p.W2, p.M)]
        outs = [t for p in sp + pp for t in (p.hist, p.M)]
        hostO = [torch.empty_like(t, device="cpu").pin_memory() for t in outs]
        h2d = sum(t.numel() * t.element_size() for t in hostW)
        d2h = sum(t.numel() * t.element_size() for t in outs)
        n_e2e = max(2, min(args.steps, 5))

        def e2e_step():
            for h, d in zip(hostW, devW):
                d.copy_(h, non_blocking=True)
            one_step()
            for h, d in zip(hostO, outs):
                h.copy_(d, non_blocking=True)

        e2e_step()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(n_e2e):
            e2e_step()
        e1.record()
        torch.cuda.synchronize()
        ems = e0.elapsed_time(e1)
        e2e = dict(value=n_e2e / (ems * 1e-3), unit=UNIT, h2d_bytes_per_step=int(h2d), d2h_bytes_per_step=int(d2h),
                   steps=n_e2e)

    cpu_base = None
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        dt, sps = time_oracle(spec, singles, pairs, args.sample_frac, 1, 0, args.loss == "ste")
        cpu_base = dict(value=sps, unit=UNIT, cores=cpu_threads(), kind="oracle",
                        sample=f"1/{args.sample_frac} of the free-axis rows of every matrix of the layer, one step "
                               f"({dt:.1f} s), extrapolated linearly")

    if rank == 0:
        out = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=max(args.warmup, 3),
                   ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                   data="synthetic", config=cfg_json, clocks=clocks, e2e=e2e, gpu_launches=int(launches),
                   roofline=roof, cpu_baseline=cpu_base, kernels=kernel_ms,
                   gb_per_s_algorithmic=2.0 * layer.weights * world / (ms_per_step * 1e-3) / 1e9,
                   tflops_algorithmic=2.0 * k * layer.weights * world / (ms_per_step * 1e-3) / 1e12)
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
