"""One decoder layer's worth of CafeQ problems, prepared once and stepped many times.

Holds descriptors, device buffers and workspaces for every matrix / pair of a layer so that a step is
nothing but C-ABI calls on resident memory (no allocation inside the step).  Marshalling only.

Two kinds of step:
  * ``step(flags)``      forward + backward of the training objective at the current transform
                         (cafeq_proxy_loss_fwd_bwd / cafeq_pair_loss_fwd_bwd);
  * ``opt_step()``       forward + backward + parameter update (cafeq_optimize_single / _pair with
                         steps = 1), resuming from the optimiser state of the previous call, which also
                         carries the previous inverse so the block inverse is refined, not recomputed.
"""
from __future__ import annotations

import ctypes

import torch

from . import (AXIS_IN, LOSS_PQE_STE, OPT_STATE_HEADER, cafeq_pair_product, FLAG_EXACT_LOSS, LOSS_LSE, LOSS_SURROGATE, OFFSETS_NONE, OPT_ADAM, OPT_GD, _check, _p,
               _pair_descs, _stream, lib, make_cfg, make_desc, set_overlap_mode, workspace_size)


class SingleProblem:
    def __init__(self, name, W, M, bits, group, taxis=AXIS_IN, lr=1e-3, loss_kind=LOSS_SURROGATE):
        self.name, self.W, self.M = name, W, M
        self.loss_kind = loss_kind
        d_out, d_in = W.shape
        self.desc = make_desc(d_out, d_in, bits, group, M.shape[-1], taxis, 0, 1, W.stride(0))
        self.losses = torch.zeros(4, dtype=torch.float32, device=W.device)
        self.grad = torch.empty_like(M)
        self.status = torch.zeros(1, dtype=torch.int32, device=W.device)
        self.ws_bytes = workspace_size(self.desc)
        self.weights = W.numel()
        self.opt_state = torch.zeros(OPT_STATE_HEADER + 3 * M.numel(), dtype=torch.float32, device=W.device)
        self.hist = torch.zeros((1, 2), dtype=torch.float32, device=W.device)
        self.cfg = make_cfg(loss_kind=loss_kind, optimizer=OPT_GD, lr=lr, steps=1, eval_every=0, resume=0)

    def step(self, ws, flags=0, loss_kind=None):
        loss_kind = self.loss_kind if loss_kind is None else loss_kind
        rc = lib().cafeq_proxy_loss_fwd_bwd(ctypes.byref(self.desc), _p(self.W), _p(self.M), _p(None), _p(None),
                                            ctypes.c_int(OFFSETS_NONE), ctypes.c_int(loss_kind), ctypes.c_float(0.0),
                                            ctypes.c_int(flags), _p(self.losses), _p(self.grad), _p(None), _p(self.status),
                                            _p(ws), ctypes.c_size_t(ws.numel()), _stream())
        _check(rc, "cafeq_proxy_loss_fwd_bwd")

    def opt_step(self, ws, eval_exact=False):
        self.cfg.eval_every = 1 if eval_exact else 0
        rc = lib().cafeq_optimize_single(ctypes.byref(self.desc), _p(self.W), _p(self.M), _p(self.opt_state),
                                         ctypes.byref(self.cfg), _p(self.hist), _p(self.status), _p(ws),
                                         ctypes.c_size_t(ws.numel()), _stream())
        _check(rc, "cafeq_optimize_single")
        self.cfg.resume = 1


class PairProblem:
    def __init__(self, name, W1, W2, M, bits, group1, group2, replicas, lse_t=5.0, lambda_orth=0.1, lr=1e-4,
                 loss_kind=LOSS_LSE):
        self.name, self.W1, self.W2, self.M = name, W1, W2, M
        self.loss_kind = loss_kind
        self.d1, self.d2 = _pair_descs(W1, W2, M.shape[-1], bits, group1, group2, replicas)
        self.losses = torch.zeros(4, dtype=torch.float32, device=W1.device)
        self.grad = torch.empty_like(M)
        self.status = torch.zeros(1, dtype=torch.int32, device=W1.device)
        self.ws_bytes = workspace_size(self.d1, self.d2)
        self.lse_t, self.lambda_orth = lse_t, lambda_orth
        self.weights = W1.numel() + W2.numel()
        self.P = None
        if loss_kind == LOSS_PQE_STE:  # the product term is the objective itself: W1 W2 is needed every step
            self.P = cafeq_pair_product(W1, W2, k=M.shape[-1], replicas=replicas)
        self.opt_state = torch.zeros(OPT_STATE_HEADER + 3 * M.numel(), dtype=torch.float32, device=W1.device)
        self.hist = torch.zeros((1, 2), dtype=torch.float32, device=W1.device)
        self.cfg = make_cfg(loss_kind=loss_kind, optimizer=OPT_ADAM, lr=lr, beta1=0.1, beta2=0.999, eps=1e-8,
                            lambda_orth=lambda_orth, lse_t=lse_t, steps=1, eval_every=0, resume=0)

    def step(self, ws, flags=0):
        rc = lib().cafeq_pair_loss_fwd_bwd(ctypes.byref(self.d1), _p(self.W1), ctypes.byref(self.d2), _p(self.W2),
                                           _p(self.M),
                                           _p(self.P if ((flags & FLAG_EXACT_LOSS) or self.loss_kind == LOSS_PQE_STE) else None),
                                           ctypes.c_int(self.loss_kind), ctypes.c_float(self.lse_t),
                                           ctypes.c_float(self.lambda_orth), ctypes.c_int(flags), _p(self.losses),
                                           _p(self.grad), _p(self.status), _p(ws), ctypes.c_size_t(ws.numel()),
                                           _stream())
        _check(rc, "cafeq_pair_loss_fwd_bwd")

    def opt_step(self, ws, eval_exact=False):
        self.cfg.eval_every = 1 if (eval_exact and self.P is not None) else 0
        rc = lib().cafeq_optimize_pair(ctypes.byref(self.d1), _p(self.W1), ctypes.byref(self.d2), _p(self.W2),
                                       _p(self.M), _p(self.opt_state),
                                       _p(self.P if (self.cfg.eval_every or self.loss_kind == LOSS_PQE_STE) else None),
                                       ctypes.byref(self.cfg), _p(self.hist), _p(self.status), _p(ws),
                                       ctypes.c_size_t(ws.numel()), _stream())
        _check(rc, "cafeq_optimize_pair")
        self.cfg.resume = 1


class LayerStep:
    """All single matrices and pairs of one layer; step() / opt_step() run over every one of them.

    The problems of a layer are independent, so with ``parallel=True`` every problem gets its own workspace
    and its own stream: opt_step() forks from the current stream, enqueues each problem's calls on that
    problem's stream and joins back, which lets the short, latency-bound kernels of one problem (block
    inverse, k x k products) run beside the bandwidth-bound passes of another.  The fork/join uses events
    only, so it can be captured into a CUDA graph."""

    def __init__(self, singles, pairs, parallel=False):
        self.singles, self.pairs = list(singles), list(pairs)
        probs = self.singles + self.pairs
        dev = probs[0].status.device
        self.parallel = parallel
        if parallel:
            for p in probs:
                p.ws = torch.empty(max(p.ws_bytes, 256), dtype=torch.uint8, device=dev)
            self.streams = [torch.cuda.Stream(device=dev) for _ in probs]
            self.ws = None
        else:
            need = max([p.ws_bytes for p in probs] + [256])
            self.ws = torch.empty(need, dtype=torch.uint8, device=dev)
            for p in probs:
                p.ws = self.ws
        self.weights = sum(p.weights for p in probs)

    def step(self, flags=0):
        for p in self.singles + self.pairs:
            p.step(p.ws, flags)

    def opt_step(self, eval_exact=False):
        probs = self.singles + self.pairs
        # launch shapes for overlapping problems (fewer SM-microseconds per kernel) or for a single chain of kernels
        # running alone (lowest latency)
        set_overlap_mode(self.parallel)
        if not self.parallel:
            for p in probs:
                p.opt_step(p.ws, eval_exact)
            return
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        # largest problems first, so the long chains start early
        order = sorted(range(len(probs)), key=lambda i: -probs[i].weights)
        for i in order:
            st = self.streams[i]
            st.wait_event(fork)
            with torch.cuda.stream(st):
                probs[i].opt_step(probs[i].ws, eval_exact)
                done = torch.cuda.Event()
                done.record(st)
            main.wait_event(done)

    def statuses(self):
        return [int(p.status.item()) for p in self.singles + self.pairs]
