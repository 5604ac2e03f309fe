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
    """DRAM bytes per launch (mean over the transform-pass and backward launches of a step) from the committed ncu
    summaries, or None once a kernel source differs from the one that was profiled."""
    import hashlib
    import re
    try:
        txt = open(os.path.join(ROOT, "profiles", "bd_bwd_dual_kernel_9b_layer.md")).read()
        src = b"".join(open(os.path.join(ROOT, "paper_2511_19705_b200", "csrc", f), "rb").read()
                       for f in ("kernels_fused.cuh", "kernels_bwd.cuh"))
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


def measure_extras(cq, torch, devS, devP, bits, group, peaks):
    """Round-to-nearest (with and without a transform) and packing on the largest single matrix against the HBM
    roofline, and one iteration of Algorithm 1 / of the learned-offset rounding on the first pair.  Every timed call is
    preceded by a pass over a buffer larger than L2 (read, not written: dirty lines of a written flush buffer would be
    written back during the timed kernel and charged to it)."""
    out = {}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=devS[0][1].device if devS else devP[0][1].device)
    flush.fill_(1)
    flush_sink = torch.zeros((), dtype=torch.int64, device=flush.device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, reps=5):
        best = None
        for _ in range(reps + 1):
            for _ in range(3):  # (three passes keep the device busy while the host prepares the timed call)
                flush_sink.copy_(flush.sum(dtype=torch.int64))
            e0.record()
            r = fn()
            e1.record()
            torch.cuda.synchronize()
            t = e0.elapsed_time(e1)
            best = t if best is None else min(best, t)
        return best * 1e-3, r

    hbm = peaks["hbm_gbs"]
    if devS:
        n, W, M = max(devS, key=lambda x: x[1].numel())
        nw = W.numel()
        g = group or W.shape[1]
        by = nw * (2.0 + 1.0 + 4.0 / g)                     # bf16 in, int8 codes + fp32 scales out
        t, _ = timed(lambda: cq.cafeq_rtn(W, None, bits=bits, group=group))
        out["rtn_plain"] = dict(matrix=n, ms=t * 1e3, gbs=by / t / 1e9, frac_of_hbm=by / t / 1e9 / hbm, bytes_per_weight=by / nw)
        t, (codes, scales) = timed(lambda: cq.cafeq_rtn(W, M, bits=bits, group=group, tblock=int(M.shape[-1])))
        out["rtn_transformed"] = dict(matrix=n, ms=t * 1e3, gbs=by / t / 1e9, frac_of_hbm=by / t / 1e9 / hbm,
                                      tflops=2.0 * M.shape[-1] * nw / t / 1e12)
        byp = nw * (1.0 + bits / 8.0)
        t, _ = timed(lambda: cq.cafeq_pack(codes, bits=bits))
        out["pack"] = dict(matrix=n, ms=t * 1e3, gbs=byp / t / 1e9, frac_of_hbm=byp / t / 1e9 / hbm, bytes_per_weight=byp / nw)
        del codes, scales
    if devP:
        n, W1, W2, M, r = devP[0]
        t0_, _ = timed(lambda: cq.cafeq_adaptive_round(W1, W2, M, iters=0, bits=bits, group1=group, group2=group, replicas=r), reps=1)
        t1_, o = timed(lambda: cq.cafeq_adaptive_round(W1, W2, M, iters=1, bits=bits, group1=group, group2=group, replicas=r), reps=1)
        H = o["pqe"].cpu().numpy()
        out["algorithm1"] = dict(pair=n, ms_per_iteration=(t1_ - t0_) * 1e3, setup_ms=t0_ * 1e3,
                                 pqe_independent=float(H[0]), pqe_after_iteration=float(H[1:].min()))
        t2_, o = timed(lambda: cq.cafeq_adaptive_round(W1, W2, M, iters=2, bits=bits, group1=group, group2=group, replicas=r,
                                                       mode=cq.ROUND_LEARNED_OFFSETS), reps=0)
        H = o["pqe"].cpu().numpy()
        out["learned_offsets"] = dict(pair=n, ms_total_2_iterations=t2_ * 1e3, pqe_independent=float(H[0]), pqe_hardened=float(H[-1]))
    out["inference_apply"] = measure_inference_apply(cq, torch, timed, hbm)
    return out


def measure_inference_apply(cq, torch, timed, hbm, tokens=8192, d_in=9216, d_out=2304):
    """The extra wall-clock time of the block-diagonal multiplication against the product it accompanies, on the shape
    of Section 4.1's table (down projection of the 2B model: 9216 -> 2304; the operator acts on the 2304-wide side,
    which is what the table's extra-FLOPs row, k / 9216, counts).  The product is torch's bf16 matmul (library code,
    used as the yardstick only)."""
    dev = torch.device("cuda", torch.cuda.current_device())
    gen = torch.Generator(device=dev)
    gen.manual_seed(1234)
    X = torch.randn((tokens, d_in), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    W = (torch.randn((d_out, d_in), generator=gen, device=dev, dtype=torch.float32) * 0.02).to(torch.bfloat16)
    t_mm, Y = timed(lambda: X @ W.t())
    res = dict(tokens=tokens, d_in=d_in, d_out=d_out, matmul_ms=t_mm * 1e3, matmul_tflops=2.0 * tokens * d_in * d_out / t_mm / 1e12,
               yardstick="torch bf16 matmul", blocks={})
    for k in (64, 128, 256):
        T = torch.linalg.qr(torch.randn((d_out // k, k, k), generator=gen, device=dev))[0].contiguous()
        t, _ = timed(lambda: cq.cafeq_apply_transform(Y, T))
        by = 2.0 * 2.0 * tokens * d_out                     # bf16 in, bf16 out
        res["blocks"][str(k)] = dict(ms=t * 1e3, extra_time_pct=100.0 * t / t_mm, extra_flops_pct=100.0 * k / d_in,
                                     gbs=by / t / 1e9, frac_of_hbm=by / t / 1e9 / hbm)
    return res


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
    ap.add_argument("--min-seconds", type=float, default=2.0, help="repeat the block of --steps steps until the timed region lasts this long")
    ap.add_argument("--lr-frac", type=float, default=1e-3, help="step of the single matrices = this / max|first gradient|")
    ap.add_argument("--pair-lr", type=float, default=1e-4)
    ap.add_argument("--bits", type=int, default=0, help="override the configuration's bit width")
    ap.add_argument("--group", type=int, default=0, help="override the configuration's group size")
    ap.add_argument("--no-extras", action="store_true", help="skip the one-off kernels (round-to-nearest, pack, Algorithm 1, ...)")
    ap.add_argument("--per-problem", action="store_true", help="time the per-problem calls on one stream each instead of the layer call")
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

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    from paper_2511_19705_b200 import shard
    my_layer = shard.layers_of_rank(world, world, rank)[0]     # weak scaling: one layer per rank, no data-path collective
    spec, singles, pairs = host_layer(args.config, my_layer)
    bits, group, k = spec["bits"], spec["group"], spec["k"]
    if args.group:
        group = args.group
    if args.bits:
        bits = args.bits

    def up_bf16(b):
        return torch.from_numpy(b.view(np.int16)).to(dev).view(torch.bfloat16)

    ste = args.loss == "ste"
    weights = sum(w.size for _, w, _ in singles) + sum(a.size + b.size for _, a, b, _, _ in pairs)
    # transform flops of one pass over the layer: 2 k per weight with each problem's own block size
    pass_flops = sum(2.0 * M.shape[-1] * w.size for _, w, M in singles) + \
        sum(2.0 * M.shape[-1] * (a.size + b.size) for _, a, b, M, _ in pairs)
    cfg_json.update(weights_per_step=int(weights), bits=bits, group=group, block=k)

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # device copies of the layer
    devS = [(n, up_bf16(W), torch.from_numpy(M).to(dev)) for n, W, M in singles]
    devP = [(n, up_bf16(W1), up_bf16(W2), torch.from_numpy(M).to(dev), r) for n, W1, W2, M, r in pairs]

    # gradient-descent step size of the single matrices: a fixed fraction (--lr-frac) of the first gradient's largest
    # entry, so that the transforms move every step and the warm-started block inverse has real work
    lr_single = {}
    for n, W, M in devS:
        out = cq.cafeq_proxy_loss_fwd_bwd(W, M, bits=bits, group=group)
        lr_single[n] = float(args.lr_frac / max(float(out["gradM"].abs().max().item()), 1e-30))
    torch.cuda.synchronize()

    use_layer = (not ste) and (not args.exact) and (not args.per_problem)
    if use_layer:
        # one layer call per block size (the 27B-shaped layer has head blocks of 128 beside blocks of 256)
        by_k = {}
        for n, W, M in devS:
            by_k.setdefault(int(M.shape[-1]), ([], []))[0].append((n, W, M))
        for n, W1, W2, M, r in devP:
            by_k.setdefault(int(M.shape[-1]), ([], []))[1].append((n, W1, W2, M, r))
        opts = []
        for kk_, (ss, pq) in sorted(by_k.items()):
            o = cq.LayerOptimizer(
                [dict(W=W, M=M, bits=bits, group=group,
                      cfg=cq.make_cfg(loss_kind=cq.LOSS_SURROGATE, optimizer=cq.OPT_GD, lr=lr_single[n])) for n, W, M in ss],
                [dict(W1=W1, W2=W2, M=M, bits=bits, group1=group, group2=group, replicas=r,
                      cfg=cq.make_cfg(loss_kind=cq.LOSS_LSE, optimizer=cq.OPT_ADAM, lr=args.pair_lr, beta1=0.1, beta2=0.999, eps=1e-8,
                                      lambda_orth=0.1, lse_t=5.0)) for n, W1, W2, M, r in pq], max_steps=1)
            o.prepare()
            opts.append(o)

        def one_step():
            for o in opts:
                o.step(1)

        def statuses():
            return [int(o.status.item()) for o in opts]

        def set_serial(flag):
            pass

        step_tensors_in = [t for _, W, M in devS for t in (W, M)] + [t for _, W1, W2, M, _ in devP for t in (W1, W2, M)]
        step_tensors_out = [t for o in opts for t in list(o.hist) + list(o.M)]
        n_streams = 1
        step_desc = ("cafeq_optimize_layer: fwd+bwd+update of all %d problems (GD singles, Adam pairs), warm-started block inverse"
                     % (len(devS) + len(devP)))
        cfg_json["workspace_mb"] = round(sum(o.ws_bytes for o in opts) / 1e6, 1)
    else:
        from paper_2511_19705_b200.layer import LayerStep, PairProblem, SingleProblem
        sp = [SingleProblem(n, W, M, bits, group, lr=lr_single[n],
                            loss_kind=cq.LOSS_L2_STE if ste else cq.LOSS_SURROGATE) for n, W, M in devS]
        pp = [PairProblem(n, W1, W2, M, bits, group, group, r, lr=args.pair_lr,
                          loss_kind=cq.LOSS_PQE_STE if ste else cq.LOSS_LSE) for n, W1, W2, M, r in devP]
        if args.exact:
            for p in pp:
                p.P = cq.cafeq_pair_product(p.W1, p.W2, k=p.M.shape[-1], replicas=p.d2.replicas)
        layer = LayerStep(sp, pp, parallel=not args.serial)

        def one_step():
            layer.opt_step(eval_exact=args.exact)

        def statuses():
            return layer.statuses()

        def set_serial(flag):
            layer.parallel = (not flag) and (not args.serial)

        step_tensors_in = [t for p in sp for t in (p.W, p.M)] + [t for p in pp for t in (p.W1, p.W2, p.M)]
        step_tensors_out = [t for p in sp + pp for t in (p.hist, p.M)]
        n_streams = len(layer.streams) if layer.parallel else 1
        step_desc = "per-problem calls: fwd+bwd+update (GD singles, Adam pairs), warm-started block inverse"

    for _ in range(max(args.warmup, 3)):
        one_step()
    sync_all()
    assert all(s == 0 for s in statuses()), statuses()

    # ---- pass 1: eager launches on one stream with the library's in-stream event pairs around its main kernels
    set_serial(True)
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
    launches_per_step = (cq.launch_count() - l0) / args.steps
    ms_eager = e0.elapsed_time(e1)
    kms, kinds = cq.timer_read(n_timed)
    set_serial(False)

    # ---- pass 2 (the reported value): the same step captured once into a CUDA graph and replayed.  `--steps` steps
    #      form one block; blocks are repeated until the timed region lasts --min-seconds, so that the clock sampler
    #      sees the run and the clocks are the sustained ones.
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
    run_step = graph.replay if graph is not None else one_step
    for _ in range(3):
        run_step()
    sync_all()
    e0.record()
    for _ in range(args.steps):
        run_step()
    e1.record()
    sync_all()
    est = max(e0.elapsed_time(e1), 1e-3)
    reps = max(1, int(np.ceil(args.min_seconds * 1e3 / est)))
    if dist is not None:
        t = torch.tensor([reps], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        reps = int(t.item())
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    sync_all()
    e0.record()
    for _ in range(reps * args.steps):
        run_step()
    e1.record()
    sync_all()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    assert all(s == 0 for s in statuses()), statuses()
    ms = shard.max_over_ranks(ms, dev)
    timed_steps = reps * args.steps
    ms_per_step = ms / timed_steps
    value = world * timed_steps / (ms * 1e-3)
    launches = int(round(launches_per_step * timed_steps))
    cfg_json.update(launch="cuda_graph_replay" if graph is not None else "eager", streams=n_streams,
                    eager_ms_per_step=ms_eager / args.steps, step=step_desc, timed_steps=timed_steps,
                    timed_region_s=ms * 1e-3, single_lr="%g / max|grad0|" % args.lr_frac, pair_lr=args.pair_lr)

    # ---- roofline of the weight-touching kernels (transform pass + sparse backward), from the in-stream event pairs.
    #      Bound: what ONE fused forward+backward kernel would need: every weight read once (2 B) and one 2k-flop
    #      transform per weight; the larger of the two times at the measured peaks.
    peaks = load_peaks()
    by_kind = {}
    for d, kd in zip(kms, kinds):
        by_kind.setdefault(kd, []).append(d)
    names = {1: "transform_pass_generic", 2: "sparse_backward", 3: "block_inverse", 4: "pair_product",
             5: "transform_pass_tcgen05"}
    kernel_ms = {names.get(kd, str(kd)): dict(launches_per_step=len(v) / args.steps, ms_per_step=sum(v) / args.steps)
                 for kd, v in by_kind.items()}
    roof = None
    tk = max((kd for kd in (1, 5) if kd in by_kind), key=lambda kd: sum(by_kind[kd]), default=None)
    if tk is not None and not ste:
        t_pass = sum(by_kind[tk]) / args.steps * 1e-3
        t_bwd = sum(by_kind.get(2, [])) / args.steps * 1e-3
        t_fb = t_pass + t_bwd
        flops = pass_flops
        byts = 2.0 * weights
        sus = peaks["bf16_sus"] or peaks["bf16_tflops"]
        # which measured peak the kernels are held to: the sustained one when the clocks sagged during the seconds-long
        # timed region (power cap), the burst one when they stayed at the maximum (this workload draws far less power
        # than a dense GEMM loop); both fractions are reported
        at_max = bool(clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and clocks["sm_mhz"] >= 0.95 * clocks["sm_max_mhz"])
        tc_peak = peaks["bf16_tflops"] if at_max else sus
        bound_is_tensor = flops / (tc_peak * 1e12) >= byts / (peaks["hbm_gbs"] * 1e9)
        n_launch = (len(by_kind[tk]) + len(by_kind.get(2, []))) / args.steps
        if bound_is_tensor:
            ach = flops / t_fb / 1e12
            roof = dict(bound="tensor", achieved=ach, peak=tc_peak, unit="TFLOP/s", frac=ach / tc_peak,
                        frac_of_burst_peak=ach / peaks["bf16_tflops"], frac_of_sustained_peak=ach / sus)
        else:
            ach = byts / t_fb / 1e9
            roof = dict(bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"])
        roof.update(traffic=profiled_traffic() if (use_layer and args.config == 3) else None,
                    algorithmic_bytes_per_launch=byts * 2 / n_launch if n_launch else None,
                    kernel="transform pass + sparse backward (bd_pass_dual_kernel + bd_bwd_dual_kernel: one launch each for both axes; bd_pass_kernel + bd_bwd_kernel per axis on layers with one axis only), the forward+backward of one step",
                    peak_source=peaks["source"] + ((" burst (SM clock stayed at its maximum through the timed region)" if at_max
                                                    else " sustained (SM clock sagged under load)") if bound_is_tensor else ""),
                    launches_per_step=n_launch, ms_per_step=t_fb * 1e3,
                    algorithmic_bytes_per_step=byts, algorithmic_flop_per_step=flops,
                    hbm_gbs_achieved=byts / t_fb / 1e9,
                    forward_only=dict(ms_per_step=t_pass * 1e3, tflops=flops / t_pass / 1e12, frac=flops / t_pass / 1e12 / tc_peak,
                                      hbm_gbs=byts / t_pass / 1e9),
                    backward_only=dict(ms_per_step=t_bwd * 1e3, hbm_gbs=byts / t_bwd / 1e9 if t_bwd > 0 else None,
                                       issued_tflops=(flops if use_layer else 2 * flops) / t_bwd / 1e12 if t_bwd > 0 else None,
                                       form="one fp16 term" if use_layer else "two bf16 terms"),
                    whole_step_frac=(flops / (ms_per_step * 1e-3) / 1e12 / tc_peak) if bound_is_tensor else
                                    (byts / (ms_per_step * 1e-3) / 1e9 / peaks["hbm_gbs"]))

    # ---- end to end through the C ABI with host buffers (pinned): H2D of every weight and transform, the step,
    #      D2H of the loss histories and the updated transforms, every step
    e2e = None
    if not args.no_e2e and rank == 0:
        hostW = [t.cpu().pin_memory() for t in step_tensors_in]
        devW = step_tensors_in
        outs = step_tensors_out
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

    # ---- the one-off kernels of the path, each against the roofline that bounds it (largest matrix of the layer)
    extras = None
    if not args.no_extras and rank == 0 and world == 1 and use_layer:
        extras = measure_extras(cq, torch, devS, devP, bits, group, peaks)

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
                   roofline=roof, cpu_baseline=cpu_base, kernels=kernel_ms, extras=extras,
                   gb_per_s_algorithmic=2.0 * weights * world / (ms_per_step * 1e-3) / 1e9,
                   tflops_algorithmic=pass_flops * world / (ms_per_step * 1e-3) / 1e12)
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
