"""One decoder layer's worth of CafeQ problems, prepared once and stepped many times.

Holds descriptors, device buffers and workspaces for every matrix / pair of a layer so that a step is
nothing but C-ABI calls on resident memory (no allocation inside the step).  Marshalling only.
"""
from __future__ import annotations

import ctypes

import torch

from . import (AXIS_IN, FLAG_EXACT_LOSS, LOSS_LSE, LOSS_SURROGATE, OFFSETS_NONE, _check, _p, _pair_descs, _stream,
               lib, make_desc, workspace_size)


class SingleProblem:
    def __init__(self, name, W, M, bits, group, taxis=AXIS_IN):
        self.name, self.W, self.M = name, W, M
        d_out, d_in = W.shape
        self.desc = make_desc(d_out, d_in, bits, group, M.shape[-1], taxis, 0, 1, W.stride(0))
        self.losses = torch.zeros(4, dtype=torch.float32, device=W.device)
        self.grad = torch.empty_like(M)
        self.status = torch.zeros(1, dtype=torch.int32, device=W.device)
        self.ws_bytes = workspace_size(self.desc)
        self.weights = W.numel()

    def step(self, ws, flags=0, loss_kind=LOSS_SURROGATE):
        rc = lib().cafeq_proxy_loss_fwd_bwd(ctypes.byref(self.desc), _p(self.W), _p(self.M), _p(None), _p(None),
                                            ctypes.c_int(OFFSETS_NONE), ctypes.c_int(loss_kind), ctypes.c_float(0.0),
                                            ctypes.c_int(flags), _p(self.losses), _p(self.grad), _p(self.status),
                                            _p(ws), ctypes.c_size_t(ws.numel()), _stream())
        _check(rc, "cafeq_proxy_loss_fwd_bwd")


class PairProblem:
    def __init__(self, name, W1, W2, M, bits, group1, group2, replicas, lse_t=5.0, lambda_orth=0.1):
        self.name, self.W1, self.W2, self.M = name, W1, W2, M
        self.d1, self.d2 = _pair_descs(W1, W2, M.shape[-1], bits, group1, group2, replicas)
        self.losses = torch.zeros(4, dtype=torch.float32, device=W1.device)
        self.grad = torch.empty_like(M)
        self.status = torch.zeros(1, dtype=torch.int32, device=W1.device)
        self.ws_bytes = workspace_size(self.d1, self.d2)
        self.lse_t, self.lambda_orth = lse_t, lambda_orth
        self.weights = W1.numel() + W2.numel()
        self.P = None

    def step(self, ws, flags=0):
        rc = lib().cafeq_pair_loss_fwd_bwd(ctypes.byref(self.d1), _p(self.W1), ctypes.byref(self.d2), _p(self.W2),
                                           _p(self.M), _p(self.P if (flags & FLAG_EXACT_LOSS) else None),
                                           ctypes.c_int(LOSS_LSE), ctypes.c_float(self.lse_t),
                                           ctypes.c_float(self.lambda_orth), ctypes.c_int(flags), _p(self.losses),
                                           _p(self.grad), _p(self.status), _p(ws), ctypes.c_size_t(ws.numel()),
                                           _stream())
        _check(rc, "cafeq_pair_loss_fwd_bwd")


class LayerStep:
    """All single matrices and pairs of one layer; step() = one forward+backward over every one of them."""

    def __init__(self, singles, pairs):
        self.singles, self.pairs = list(singles), list(pairs)
        need = max([p.ws_bytes for p in self.singles + self.pairs] + [256])
        dev = (self.singles + self.pairs)[0].status.device
        self.ws = torch.empty(need, dtype=torch.uint8, device=dev)
        self.weights = sum(p.weights for p in self.singles + self.pairs)

    def step(self, flags=0):
        for p in self.singles:
            p.step(self.ws, flags)
        for p in self.pairs:
            p.step(self.ws, flags)

    def statuses(self):
        return [int(p.status.item()) for p in self.singles + self.pairs]
