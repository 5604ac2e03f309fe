"""Whole weight sets streamed through one GPU, one decoder layer resident at a time (Section 6's recipe).

For every layer: the single matrices get a learned block-diagonal transform (gradient descent on Eq. 4) and are
then rounded to nearest and packed; every coupled pair gets a learned paired transform (Adam on the LogSumExp
surrogate with the orthonormality penalty) followed by Algorithm 1 on the transformed pair, and both factors are
packed.  All of it is C-ABI calls (cafeq_layer_prepare / cafeq_optimize_layer, cafeq_rtn, cafeq_adaptive_round,
cafeq_pack, cafeq_proxy_loss_fwd_bwd for the reported errors); this module only generates the seeded stand-in
weights on the host (a background thread works on the next layer while the current one is on the GPU), uploads
them, and collects per-layer results.  Layers are independent problems: with several ranks each takes every
world-th layer and there is no data-path collective (paper_2511_19705_b200.shard).

    python -m paper_2511_19705_b200.stream_layers --config 4 --layers 42 --bits 4 3 --steps 500
"""
from __future__ import annotations

import argparse
import json
import time
import zlib
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

import cafeq_synth as syn

from . import (FLAG_EXACT_LOSS, FLAG_NO_GRAD, LOSS_LSE, LOSS_SURROGATE, OPT_ADAM, OPT_GD, LayerOptimizer, cafeq_adaptive_round,
               cafeq_pack, cafeq_pair_product, cafeq_proxy_loss_fwd_bwd, cafeq_rtn, make_cfg)
from . import shard

N_LAYERS = {3: 1, 4: 42, 5: 46}


def host_layer(config: int, layer: int, pool: ThreadPoolExecutor | None = None):
    """Seeded host arrays of one layer: (spec, {name: bf16 bits}, {problem: fp32 transform}); the matrices are drawn in
    parallel when a pool is given (every matrix has its own generator)."""
    spec = syn.layer_spec(config)
    jobs, transforms = {}, {}

    def submit(name, d_out, d_in):
        if pool is None:
            jobs[name] = syn.make_weight(config, name, d_out, d_in, layer)
        else:
            jobs[name] = pool.submit(syn.make_weight, config, name, d_out, d_in, layer)

    for name, d_out, d_in in spec["singles"]:
        submit(name, d_out, d_in)
        transforms[name] = syn.make_transform(name, d_in // spec["k"], spec["k"], layer)
    for pname, (n1, h, d1), (n2, d3, rh), kb, r in spec["pairs"]:
        submit(n1, h, d1)
        submit(n2, d3, rh)
        transforms[pname] = syn.make_transform(n1, h // kb, kb, layer)
    weights = {n: (j if isinstance(j, np.ndarray) else j.result()) for n, j in jobs.items()}
    return spec, weights, transforms


def _dev_bf16(bits_u16, dev):
    return torch.from_numpy(bits_u16.view(np.int16)).to(dev, non_blocking=True).view(torch.bfloat16)


def process_layer(spec, weights, transforms, dev, *, bits, group, steps, alg1_iters=1, lr_frac=1e-3, pair_lr=1e-3,
                  keep_outputs=False):
    """Everything Section 6 does to one layer; returns a dict of per-matrix results (errors, loss histories' ends,
    packed sizes and checksums; the packed codes and scales themselves with keep_outputs)."""
    W = {n: _dev_bf16(b, dev) for n, b in weights.items()}
    M = {n: torch.from_numpy(t).to(dev) for n, t in transforms.items()}
    res = {}
    # step size of the single matrices: a fraction of the first gradient's largest entry (Eq. 4's scale depends on the shape)
    lr = {}
    for name, d_out, d_in in spec["singles"]:
        g0 = cafeq_proxy_loss_fwd_bwd(W[name], M[name], bits=bits, group=group)["gradM"]
        lr[name] = float(lr_frac / max(float(g0.abs().max().item()), 1e-30))
    # one layer call per block size (a layer call takes one block size)
    by_k = {}
    for name, d_out, d_in in spec["singles"]:
        by_k.setdefault(spec["k"], ([], []))[0].append(name)
    for pname, (n1, h, d1), (n2, d3, rh), kb, r in spec["pairs"]:
        by_k.setdefault(kb, ([], []))[1].append((pname, n1, n2, r))
    t_opt = 0.0
    for k, (sn, pn) in by_k.items():
        opt = LayerOptimizer(
            [dict(W=W[n], M=M[n], bits=bits, group=group, cfg=make_cfg(loss_kind=LOSS_SURROGATE, optimizer=OPT_GD, lr=lr[n]))
             for n in sn],
            [dict(W1=W[n1], W2=W[n2], M=M[p], bits=bits, group1=group, group2=group, replicas=r,
                  cfg=make_cfg(loss_kind=LOSS_LSE, optimizer=OPT_ADAM, lr=pair_lr, beta1=0.1, beta2=0.999, eps=1e-8,
                               lambda_orth=0.1, lse_t=5.0)) for p, n1, n2, r in pn], max_steps=steps)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        opt.prepare()
        opt.step(steps)
        e1.record()
        torch.cuda.synchronize()
        t_opt += e0.elapsed_time(e1) * 1e-3
        st = int(opt.status.item())
        if st != 0:
            raise RuntimeError(f"device status {st} while optimising block size {k}")
        for i, n in enumerate(sn + [p for p, *_ in pn]):
            h = opt.hist[i][:, 0]
            res[n] = dict(loss_first=float(h[0].item()), loss_last=float(h[-1].item()), lr=lr.get(n, pair_lr))
        del opt
    # final quantisation
    for name, d_out, d_in in spec["singles"]:
        codes, scales = cafeq_rtn(W[name], M[name], bits=bits, group=group, tblock=spec["k"])
        packed = cafeq_pack(codes, bits=bits)
        L = cafeq_proxy_loss_fwd_bwd(W[name], M[name], bits=bits, group=group, flags=FLAG_EXACT_LOSS | FLAG_NO_GRAD)["losses"]
        Lc = L.cpu().numpy()
        res[name].update(rel_l2=float(np.sqrt(Lc[1] / Lc[2])), packed_bytes=int(packed.numel()),
                         crc=zlib.crc32(packed.cpu().numpy().tobytes()))
        if keep_outputs:
            res[name].update(packed=packed.cpu(), scales=scales.cpu(), codes=codes.cpu(), M=M[name].cpu())
    for pname, (n1, h, d1), (n2, d3, rh), kb, r in spec["pairs"]:
        out = cafeq_adaptive_round(W[n1], W[n2], M[pname], iters=alg1_iters, bits=bits, group1=group, group2=group, replicas=r)
        st = int(out["status"].item())
        if st != 0:
            raise RuntimeError(f"device status {st} in Algorithm 1 of {pname}")
        p1, p2 = cafeq_pack(out["codes1"], bits=bits), cafeq_pack(out["codes2"], bits=bits)
        normP = float(torch.linalg.norm(cafeq_pair_product(W[n1], W[n2], k=kb, replicas=r)).item())
        H = out["pqe"].cpu().numpy()
        res[pname].update(rel_pqe_independent=float(H[0] / normP), rel_pqe_adaptive=float(H[1:].min() / normP) if len(H) > 1 else None,
                          pqe_history=[float(x) for x in H], packed_bytes=int(p1.numel() + p2.numel()),
                          crc=zlib.crc32(p1.cpu().numpy().tobytes() + p2.cpu().numpy().tobytes()))
        if keep_outputs:
            res[pname].update(packed1=p1.cpu(), packed2=p2.cpu(), scales1=out["scales1"].cpu(), scales2=out["scales2"].cpu(),
                              codes1=out["codes1"].cpu(), codes2=out["codes2"].cpu(), M=M[pname].cpu())
    res["_optimise_seconds"] = t_opt
    return res


def run_weight_set(config: int, variants, layers=None, steps=None, alg1_iters=1, rank=0, world=1, device=None,
                   lr_frac=1e-3, pair_lr=1e-3, keep_outputs=False, log=None):
    """variants: list of (bits, group).  Returns {(layer, bits, group): result dict} for this rank's layers, and a
    summary dict with wall and device times."""
    dev = device or torch.device("cuda", torch.cuda.current_device())
    n_layers = layers if layers is not None else N_LAYERS[config]
    mine = shard.layers_of_rank(n_layers, world, rank)
    spec = syn.layer_spec(config)
    steps = steps or spec["steps"]
    out, t_gpu = {}, 0.0
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=8) as draw_pool, ThreadPoolExecutor(max_workers=1) as ahead:
        nxt = ahead.submit(host_layer, config, mine[0], draw_pool) if mine else None
        for i, layer in enumerate(mine):
            spec, weights, transforms = nxt.result()
            nxt = ahead.submit(host_layer, config, mine[i + 1], draw_pool) if i + 1 < len(mine) else None
            for bits, group in variants:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                # every variant starts from the same initial rotations
                r = process_layer(spec, weights, {k: v.copy() for k, v in transforms.items()}, dev, bits=bits, group=group,
                                  steps=steps, alg1_iters=alg1_iters, lr_frac=lr_frac, pair_lr=pair_lr, keep_outputs=keep_outputs)
                e1.record()
                torch.cuda.synchronize()
                r["_gpu_seconds"] = e0.elapsed_time(e1) * 1e-3
                t_gpu += r["_gpu_seconds"]
                out[(layer, bits, group)] = r
                if log:
                    log(layer, bits, group, r)
    wall = time.perf_counter() - t0
    summary = dict(config=config, layers=len(mine), variants=[list(v) for v in variants], steps=steps, alg1_iters=alg1_iters,
                   wall_seconds=wall, gpu_seconds=t_gpu,
                   optimise_seconds=sum(r["_optimise_seconds"] for r in out.values()),
                   note="wall time includes drawing the synthetic weights on the host (a background thread works one layer ahead)")
    return out, summary


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--layers", type=int, default=None)
    ap.add_argument("--bits", type=int, nargs="+", default=None)
    ap.add_argument("--groups", type=int, nargs="+", default=None)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--alg1-iters", type=int, default=1)
    ap.add_argument("--lr-frac", type=float, default=1e-3)
    ap.add_argument("--pair-lr", type=float, default=1e-3)
    args = ap.parse_args()
    spec = syn.layer_spec(args.config)
    bits = args.bits or ([4, 3] if args.config == 4 else [spec["bits"]])
    groups = args.groups or ([64, 128] if args.config == 5 else [spec["group"]])
    variants = [(b, g) for b in bits for g in groups]

    def log(layer, b, g, r):
        names = [n for n in r if not n.startswith("_")]
        errs = {n: round(r[n].get("rel_l2", r[n].get("rel_pqe_adaptive")) or 0.0, 4) for n in names}
        print(f"layer {layer:3d} bits {b} group {g:3d}: {r['_gpu_seconds']:.2f} s on the device, errors {errs}", flush=True)

    res, summary = run_weight_set(args.config, variants, args.layers, args.steps, args.alg1_iters, lr_frac=args.lr_frac,
                                  pair_lr=args.pair_lr, log=log)
    agg = {}
    for (layer, b, g), r in res.items():
        for n, v in r.items():
            if n.startswith("_"):
                continue
            key = f"{n}/b{b}/g{g}"
            e = v.get("rel_l2", v.get("rel_pqe_adaptive"))
            agg.setdefault(key, []).append(e)
            if "rel_pqe_independent" in v:
                agg.setdefault(key + "/independent", []).append(v["rel_pqe_independent"])
    summary["mean_relative_error"] = {k: float(np.mean(v)) for k, v in agg.items()}
    print(json.dumps(summary))


if __name__ == "__main__":
    main()
