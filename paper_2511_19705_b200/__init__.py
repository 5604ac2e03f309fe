"""Thin Python binding of the CafeQ C-ABI library (include/cafeq.h).

Argument marshalling only: every step of the path runs in the CUDA kernels of
``libcafeq.so``.  PyTorch supplies device memory and the current stream.  There is
no CPU fallback: if the library has not been built, every call raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcafeq.so")

AXIS_IN, AXIS_OUT = 0, 1
APPLY_T, APPLY_TT = 0, 1
LOSS_SURROGATE, LOSS_L2_STE, LOSS_LSE, LOSS_PQE_STE, LOSS_SUMSQ, LOSS_SUMSQ_WEIGHTED = 0, 1, 2, 3, 4, 5
OPT_STATE_HEADER = 4   # floats before the moment arrays of an optimiser state (CAFEQ_OPT_STATE_HEADER)
OPT_GD, OPT_ADAM, OPT_CAYLEY = 0, 1, 2
FLAG_EXACT_LOSS, FLAG_NO_GRAD, FLAG_GENERIC, FLAG_WARM_MINV = 1, 2, 4, 8
OFFSETS_NONE, OFFSETS_HARD_U8, OFFSETS_SOFT_F32 = 0, 1, 2
ROUND_ALG1, ROUND_LEARNED_OFFSETS = 0, 1

EXPORTS = [
    "cafeq_workspace_size", "cafeq_rtn", "cafeq_rtn_workspace_size", "cafeq_rtn_noalloc", "cafeq_proxy_loss_fwd_bwd", "cafeq_optimize_single",
    "cafeq_pair_product", "cafeq_pair_loss_fwd_bwd", "cafeq_optimize_pair", "cafeq_adaptive_round",
    "cafeq_pack", "cafeq_apply_workspace_size", "cafeq_apply_transform", "cafeq_dequant", "cafeq_layer_workspace_size", "cafeq_layer_prepare", "cafeq_optimize_layer", "cafeq_layer_debug_fallbacks", "cafeq_debug_set_layer_launch", "cafeq_set_overlap_mode", "cafeq_debug_wait_probe", "cafeq_debug_timer_begin", "cafeq_debug_timer_read",
    "cafeq_debug_launch_count",
    "cafeq_status_string", "cafeq_version",
]


class MatrixDesc(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("d_out", ctypes.c_int32), ("d_in", ctypes.c_int32),
                ("ld", ctypes.c_int64), ("bits", ctypes.c_int32), ("group", ctypes.c_int32),
                ("tblock", ctypes.c_int32), ("taxis", ctypes.c_int32), ("trole", ctypes.c_int32),
                ("replicas", ctypes.c_int32), ("compute_prec", ctypes.c_int32)]


class OptCfg(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("loss_kind", ctypes.c_int32), ("optimizer", ctypes.c_int32),
                ("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float),
                ("eps", ctypes.c_float), ("lambda_orth", ctypes.c_float), ("lse_t", ctypes.c_float),
                ("kappa", ctypes.c_float), ("steps", ctypes.c_int32), ("eval_every", ctypes.c_int32),
                ("resume", ctypes.c_int32)]


class LayerProblem(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("pair", ctypes.c_int32), ("d1", MatrixDesc), ("d2", MatrixDesc),
                ("W1", ctypes.c_void_p), ("W2", ctypes.c_void_p), ("M", ctypes.c_void_p),
                ("opt_state", ctypes.c_void_p), ("loss_history", ctypes.c_void_p), ("cfg", OptCfg)]


class CafeqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2511_19705_b200.build` (nvcc, sm_100a)")
        L = ctypes.CDLL(LIB_PATH)
        L.cafeq_status_string.restype = ctypes.c_char_p
        L.cafeq_status_string.argtypes = [ctypes.c_int]
        L.cafeq_version.restype = ctypes.c_int
        for name in EXPORTS[:-3]:
            getattr(L, name).restype = ctypes.c_int
        L.cafeq_debug_launch_count.restype = ctypes.c_longlong
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().cafeq_status_string(int(code)).decode()


def version() -> int:
    return lib().cafeq_version()


def set_overlap_mode(overlapped: bool) -> None:
    """Process-wide launch-shape rule: True when several problems run concurrently in different streams (kernels
    then take fewer CTAs: fewer SM-microseconds each), False (default) when one problem runs alone (lowest latency)."""
    _check(lib().cafeq_set_overlap_mode(ctypes.c_int(1 if overlapped else 0)), "cafeq_set_overlap_mode")


def set_layer_launch(dual: bool = True, pass_out_pct: int = 0, bwd_out_pct: int = 0) -> None:
    """Process-wide launch rule of the layer step: both axes' matrices in one pass launch and one backward launch
    (dual), and the cost of an output-axis tile in percent of an input-axis tile (0 keeps the current value)."""
    _check(lib().cafeq_debug_set_layer_launch(ctypes.c_int(1 if dual else 0), ctypes.c_int(pass_out_pct), ctypes.c_int(bwd_out_pct)),
           "cafeq_debug_set_layer_launch")


def launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(lib().cafeq_debug_launch_count())


def timer_begin(capacity: int) -> None:
    _check(lib().cafeq_debug_timer_begin(ctypes.c_int(capacity)), "cafeq_debug_timer_begin")


def timer_read(capacity: int):
    """Returns (durations_ms list, kinds list) of the kernels timed since timer_begin."""
    ms = (ctypes.c_float * max(capacity, 1))()
    kinds = (ctypes.c_int * max(capacity, 1))()
    n = ctypes.c_int(0)
    _check(lib().cafeq_debug_timer_read(ms, kinds, ctypes.byref(n)), "cafeq_debug_timer_read")
    return [ms[i] for i in range(n.value)], [kinds[i] for i in range(n.value)]


def _check(rc: int, where: str) -> None:
    if rc != 0:
        raise CafeqError(rc, where)


def _p(t):
    if t is None:
        return ctypes.c_void_p(0)
    if isinstance(t, torch.Tensor):
        return ctypes.c_void_p(t.data_ptr())
    return ctypes.c_void_p(int(t))


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_desc(d_out, d_in, bits, group, tblock=0, taxis=AXIS_IN, trole=APPLY_T, replicas=1, ld=None) -> MatrixDesc:
    return MatrixDesc(ctypes.sizeof(MatrixDesc), d_out, d_in, d_in if ld is None else ld, bits, group, tblock,
                      taxis, trole, replicas, 0)


def make_cfg(loss_kind=LOSS_SURROGATE, optimizer=OPT_GD, lr=0.5, beta1=0.1, beta2=0.999, eps=1e-8,
             lambda_orth=0.1, lse_t=5.0, kappa=0.0, steps=1, eval_every=0, resume=0) -> OptCfg:
    return OptCfg(ctypes.sizeof(OptCfg), loss_kind, optimizer, lr, beta1, beta2, eps, lambda_orth, lse_t, kappa,
                  steps, eval_every, resume)


def workspace_size(d1: MatrixDesc, d2: MatrixDesc | None = None, cfg: OptCfg | None = None) -> int:
    n = ctypes.c_size_t(0)
    rc = lib().cafeq_workspace_size(ctypes.byref(d1), ctypes.byref(d2) if d2 is not None else None,
                                    ctypes.byref(cfg) if cfg is not None else None, ctypes.byref(n))
    _check(rc, "cafeq_workspace_size")
    return int(n.value)


def rtn_workspace_size(d: MatrixDesc, has_transform: bool) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().cafeq_rtn_workspace_size(ctypes.byref(d), ctypes.c_int(1 if has_transform else 0), ctypes.byref(n)),
           "cafeq_rtn_workspace_size")
    return int(n.value)


_ws_cache: dict = {}


def workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A cached uint8 scratch tensor of at least nbytes (torch allocations are 512-byte aligned)."""
    key = str(device)
    t = _ws_cache.get(key)
    if t is None or t.numel() < nbytes:
        _ws_cache[key] = t = torch.empty(int(nbytes), dtype=torch.uint8, device=device)
    return t


def _bits_tensor(W: torch.Tensor) -> torch.Tensor:
    if W.dtype != torch.bfloat16 or not W.is_cuda or W.dim() != 2 or W.stride(1) != 1:
        raise ValueError("W must be a 2-D CUDA bf16 tensor with unit inner stride")
    return W


def _f32(t, name):
    if t is None:
        return None
    if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA float32 tensor")
    return t


# ----------------------------------------------------------------------------- entry points
def cafeq_rtn(W, T=None, *, bits, group, tblock=0, taxis=AXIS_IN, trole=APPLY_T, replicas=1):
    """Round-to-nearest codes (int8 [d_out,d_in]) and scales (fp32 [d_out, d_in/group]) of T o W."""
    W = _bits_tensor(W)
    d_out, d_in = W.shape
    d = make_desc(d_out, d_in, bits, group, tblock if T is not None else 0, taxis, trole, replicas, W.stride(0))
    g = group or d_in
    codes = torch.empty((d_out, d_in), dtype=torch.int8, device=W.device)
    scales = torch.empty((d_out, d_in // g), dtype=torch.float32, device=W.device)
    ws = workspace(max(rtn_workspace_size(d, T is not None), 256), W.device)
    rc = lib().cafeq_rtn(ctypes.byref(d), _p(W), _p(_f32(T, "T")), _p(codes), _p(scales), _p(ws),
                         ctypes.c_size_t(ws.numel()), _stream())
    _check(rc, "cafeq_rtn")
    return codes, scales


NOALLOC_SCRATCH_BYTES = 16 << 20


def cafeq_rtn_noalloc(W, T, codes, scales, *, bits, group, tblock=0, taxis=AXIS_IN, trole=APPLY_T, replicas=1):
    """cafeq_rtn into caller-provided `codes` / `scales`, using the scratch buffer built into the library
    (no workspace, no allocation anywhere on the way).  Raises CafeqError(8) when the matrix needs more than
    NOALLOC_SCRATCH_BYTES of scratch."""
    W = _bits_tensor(W)
    d_out, d_in = W.shape
    g = group or d_in
    if codes.dtype != torch.int8 or tuple(codes.shape) != (d_out, d_in) or not codes.is_contiguous():
        raise ValueError("codes must be a contiguous int8 [d_out, d_in] tensor")
    if scales.dtype != torch.float32 or tuple(scales.shape) != (d_out, d_in // g) or not scales.is_contiguous():
        raise ValueError("scales must be a contiguous float32 [d_out, d_in/group] tensor")
    d = make_desc(d_out, d_in, bits, group, tblock if T is not None else 0, taxis, trole, replicas, W.stride(0))
    rc = lib().cafeq_rtn_noalloc(ctypes.byref(d), _p(W), _p(_f32(T, "T")), _p(codes), _p(scales), _stream())
    _check(rc, "cafeq_rtn_noalloc")
    return codes, scales


def cafeq_proxy_loss_fwd_bwd(W, M, *, bits, group, taxis=AXIS_IN, loss_kind=LOSS_SURROGATE, kappa=0.0, flags=0,
                             offsets=None, want_minv=False, Minv=None, want_grad_offsets=False):
    """Returns dict(losses[4], gradM or None, Minv or None, status int tensor, grad_offsets or None)."""
    W = _bits_tensor(W)
    M = _f32(M, "M")
    d_out, d_in = W.shape
    k = M.shape[-1]
    d = make_desc(d_out, d_in, bits, group, k, taxis, APPLY_T, 1, W.stride(0))
    losses = torch.zeros(4, dtype=torch.float32, device=W.device)
    gradM = None if (flags & FLAG_NO_GRAD) else torch.empty_like(M)
    if Minv is None:
        Minv = torch.empty_like(M) if want_minv else None
    else:
        Minv = _f32(Minv, "Minv")
    status = torch.zeros(1, dtype=torch.int32, device=W.device)
    okind = OFFSETS_NONE
    if offsets is not None:
        okind = OFFSETS_HARD_U8 if offsets.dtype == torch.uint8 else OFFSETS_SOFT_F32
        if not offsets.is_contiguous() or tuple(offsets.shape) != (d_out, d_in):
            raise ValueError("offsets must be contiguous [d_out, d_in]")
    grad_off = torch.empty((d_out, d_in), dtype=torch.float32, device=W.device) if want_grad_offsets else None
    lean = loss_kind == LOSS_SURROGATE and not (flags & (FLAG_EXACT_LOSS | FLAG_GENERIC)) and offsets is None
    ws = workspace(workspace_size(d, None, make_cfg(loss_kind=LOSS_SURROGATE) if lean else None), W.device)
    rc = lib().cafeq_proxy_loss_fwd_bwd(ctypes.byref(d), _p(W), _p(M), _p(Minv), _p(offsets), ctypes.c_int(okind),
                                        ctypes.c_int(loss_kind), ctypes.c_float(kappa), ctypes.c_int(flags),
                                        _p(losses), _p(gradM), _p(grad_off), _p(status), _p(ws),
                                        ctypes.c_size_t(ws.numel()), _stream())
    _check(rc, "cafeq_proxy_loss_fwd_bwd")
    return dict(losses=losses, gradM=gradM, Minv=Minv, status=status, grad_offsets=grad_off)


def cafeq_optimize_single(W, M, cfg: OptCfg, *, bits, group, taxis=AXIS_IN, opt_state=None):
    """Updates M in place; returns (loss_history [steps,2], status, opt_state)."""
    W = _bits_tensor(W)
    M = _f32(M, "M")
    d_out, d_in = W.shape
    d = make_desc(d_out, d_in, bits, group, M.shape[-1], taxis, APPLY_T, 1, W.stride(0))
    hist = torch.zeros((max(cfg.steps, 1), 2), dtype=torch.float32, device=W.device)
    status = torch.zeros(1, dtype=torch.int32, device=W.device)
    if cfg.optimizer == OPT_ADAM and opt_state is None:
        opt_state = torch.zeros(OPT_STATE_HEADER + 3 * M.numel(), dtype=torch.float32, device=W.device)
    ws = workspace(workspace_size(d, None, cfg), W.device)
    rc = lib().cafeq_optimize_single(ctypes.byref(d), _p(W), _p(M), _p(opt_state), ctypes.byref(cfg), _p(hist),
                                     _p(status), _p(ws), ctypes.c_size_t(ws.numel()), _stream())
    _check(rc, "cafeq_optimize_single")
    return hist, status, opt_state


def _pair_descs(W1, W2, k, bits, group1, group2, replicas):
    W1 = _bits_tensor(W1)
    W2 = _bits_tensor(W2)
    d1 = make_desc(W1.shape[0], W1.shape[1], bits, group1, k, AXIS_OUT, APPLY_TT, 1, W1.stride(0))
    d2 = make_desc(W2.shape[0], W2.shape[1], bits, group2, k, AXIS_IN, APPLY_T, replicas, W2.stride(0))
    return d1, d2


def cafeq_pair_product(W1, W2, *, k, bits=4, group1=0, group2=0, replicas=1):
    d1, d2 = _pair_descs(W1, W2, k, bits, group1, group2, replicas)
    P = torch.empty((W1.shape[1], W2.shape[0]), dtype=torch.float32, device=W1.device)
    ws = workspace(workspace_size(d1, d2), W1.device)
    rc = lib().cafeq_pair_product(ctypes.byref(d1), _p(W1), ctypes.byref(d2), _p(W2), _p(P), _p(ws),
                                  ctypes.c_size_t(ws.numel()), _stream())
    _check(rc, "cafeq_pair_product")
    return P


def cafeq_pair_loss_fwd_bwd(W1, W2, M, *, bits, group1, group2, replicas=1, P=None, loss_kind=LOSS_LSE, lse_t=5.0,
                            lambda_orth=0.0, flags=0):
    M = _f32(M, "M")
    d1, d2 = _pair_descs(W1, W2, M.shape[-1], bits, group1, group2, replicas)
    losses = torch.zeros(4, dtype=torch.float32, device=W1.device)
    gradM = None if (flags & FLAG_NO_GRAD) else torch.empty_like(M)
    status = torch.zeros(1, dtype=torch.int32, device=W1.device)
    ws = workspace(workspace_size(d1, d2), W1.device)
    rc = lib().cafeq_pair_loss_fwd_bwd(ctypes.byref(d1), _p(W1), ctypes.byref(d2), _p(W2), _p(M), _p(_f32(P, "P")),
                                       ctypes.c_int(loss_kind), ctypes.c_float(lse_t), ctypes.c_float(lambda_orth),
                                       ctypes.c_int(flags), _p(losses), _p(gradM), _p(status), _p(ws),
                                       ctypes.c_size_t(ws.numel()), _stream())
    _check(rc, "cafeq_pair_loss_fwd_bwd")
    return dict(losses=losses, gradM=gradM, status=status)


def cafeq_optimize_pair(W1, W2, M, cfg: OptCfg, *, bits, group1, group2, replicas=1, P=None, opt_state=None):
    M = _f32(M, "M")
    d1, d2 = _pair_descs(W1, W2, M.shape[-1], bits, group1, group2, replicas)
    hist = torch.zeros((max(cfg.steps, 1), 2), dtype=torch.float32, device=W1.device)
    status = torch.zeros(1, dtype=torch.int32, device=W1.device)
    if cfg.optimizer in (OPT_ADAM, OPT_CAYLEY) and opt_state is None:
        opt_state = torch.zeros(OPT_STATE_HEADER + 3 * M.numel(), dtype=torch.float32, device=W1.device)
    ws = workspace(workspace_size(d1, d2, cfg), W1.device)
    rc = lib().cafeq_optimize_pair(ctypes.byref(d1), _p(W1), ctypes.byref(d2), _p(W2), _p(M), _p(opt_state),
                                   _p(_f32(P, "P")), ctypes.byref(cfg), _p(hist), _p(status), _p(ws),
                                   ctypes.c_size_t(ws.numel()), _stream())
    _check(rc, "cafeq_optimize_pair")
    return hist, status, opt_state


def cafeq_adaptive_round(W1, W2, M, *, iters, bits, group1, group2, replicas=1, k=None, mode=0):
    k = M.shape[-1] if M is not None else k
    d1, d2 = _pair_descs(W1, W2, k, bits, group1, group2, replicas)
    dev = W1.device
    g1 = group1 or W1.shape[1]
    g2 = group2 or W2.shape[1]
    codes1 = torch.empty(tuple(W1.shape), dtype=torch.int8, device=dev)
    codes2 = torch.empty(tuple(W2.shape), dtype=torch.int8, device=dev)
    scales1 = torch.empty((W1.shape[0], W1.shape[1] // g1), dtype=torch.float32, device=dev)
    scales2 = torch.empty((W2.shape[0], W2.shape[1] // g2), dtype=torch.float32, device=dev)
    hist = torch.zeros((iters + 2) if mode == ROUND_LEARNED_OFFSETS else (2 * iters + 1), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = workspace(workspace_size(d1, d2), dev)
    rc = lib().cafeq_adaptive_round(ctypes.byref(d1), _p(W1), ctypes.byref(d2), _p(W2), _p(_f32(M, "M")),
                                    ctypes.c_int(iters), ctypes.c_int(mode), _p(codes1), _p(scales1), _p(codes2),
                                    _p(scales2), _p(hist), _p(status), _p(ws), ctypes.c_size_t(ws.numel()), _stream())
    _check(rc, "cafeq_adaptive_round")
    return dict(codes1=codes1, scales1=scales1, codes2=codes2, scales2=scales2, pqe=hist, status=status)


def cafeq_pack(codes, *, bits):
    if codes.dtype != torch.int8 or not codes.is_cuda or not codes.is_contiguous():
        raise ValueError("codes must be a contiguous CUDA int8 tensor")
    d_out, d_in = codes.shape
    d = make_desc(d_out, d_in, bits, 0)
    packed = torch.empty((d_out, d_in * bits // 8), dtype=torch.uint8, device=codes.device)
    rc = lib().cafeq_pack(ctypes.byref(d), _p(codes), _p(packed), _stream())
    _check(rc, "cafeq_pack")
    return packed


def cafeq_apply_transform(X, T, *, taxis=AXIS_IN, trole=APPLY_T, status=None):
    """Y = P o X on one axis of a bf16 activation matrix X [tokens, d_in] (P = T or T^T, rounded to bf16): the
    inference-side multiplication by the block-diagonal inverse.  Returns bf16 Y [tokens, d_in]."""
    if X.dtype != torch.bfloat16 or not X.is_cuda or X.stride(1) != 1:
        raise ValueError("X must be a CUDA bf16 matrix with unit column stride")
    d_out, d_in = X.shape
    k = T.shape[-1]
    d = make_desc(d_out, d_in, 4, 128 if d_in % 128 == 0 else d_in, k, taxis, trole, 1, X.stride(0))
    n = ctypes.c_size_t(0)
    _check(lib().cafeq_apply_workspace_size(ctypes.byref(d), ctypes.byref(n)), "cafeq_apply_workspace_size")
    ws = torch.empty(max(int(n.value), 256), dtype=torch.uint8, device=X.device)
    Y = torch.empty((d_out, d_in), dtype=torch.bfloat16, device=X.device)
    rc = lib().cafeq_apply_transform(ctypes.byref(d), _p(X), _p(T), _p(Y), _p(status), _p(ws), ctypes.c_size_t(ws.numel()), _stream())
    _check(rc, "cafeq_apply_transform")
    return Y


def cafeq_dequant(packed, scales, *, bits, group, d_in):
    """bf16 [d_out, d_in] = scales * codes from the bit stream of cafeq_pack."""
    d_out = packed.shape[0]
    d = make_desc(d_out, d_in, bits, group)
    out = torch.empty((d_out, d_in), dtype=torch.bfloat16, device=packed.device)
    rc = lib().cafeq_dequant(ctypes.byref(d), _p(packed), _p(scales), _p(out), ctypes.c_longlong(d_in), _stream())
    _check(rc, "cafeq_dequant")
    return out


# ----------------------------------------------------------------------------- one layer at a time
class LayerOptimizer:
    """All single matrices and coupled pairs of one layer behind cafeq_layer_prepare / cafeq_optimize_layer.

    singles: list of dict(W=bf16 [d_out,d_in], M=fp32 [nb,k,k], bits, group, taxis=AXIS_IN, cfg=OptCfg)
    pairs:   list of dict(W1, W2, M, bits, group1, group2, replicas, cfg=OptCfg)
    Marshalling only: builds the descriptor array, owns the workspace, the optimiser states and the loss histories."""

    def __init__(self, singles, pairs, max_steps=1):
        probs = []
        self.keep = []
        dev = (singles[0]["W"] if singles else pairs[0]["W1"]).device
        self.max_steps = max_steps
        self.hist, self.state, self.M = [], [], []
        for s in singles:
            W, M = _bits_tensor(s["W"]), _f32(s["M"], "M")
            d = make_desc(W.shape[0], W.shape[1], s["bits"], s["group"], M.shape[-1], s.get("taxis", AXIS_IN), APPLY_T, 1,
                          W.stride(0))
            probs.append((0, d, d, W, None, M, s["cfg"]))
        for q in pairs:
            M = _f32(q["M"], "M")
            d1, d2 = _pair_descs(q["W1"], q["W2"], M.shape[-1], q["bits"], q["group1"], q["group2"], q.get("replicas", 1))
            probs.append((1, d1, d2, q["W1"], q["W2"], M, q["cfg"]))
        self.n = len(probs)
        self.arr = (LayerProblem * self.n)()
        for i, (pair, d1, d2, W1, W2, M, cfg) in enumerate(probs):
            hist = torch.zeros((max_steps, 2), dtype=torch.float32, device=dev)
            state = torch.zeros(OPT_STATE_HEADER + 3 * M.numel(), dtype=torch.float32, device=dev)
            self.hist.append(hist)
            self.state.append(state)
            self.M.append(M)
            self.keep += [W1, W2]
            a = self.arr[i]
            a.struct_size = ctypes.sizeof(LayerProblem)
            a.pair = pair
            a.d1, a.d2 = d1, d2
            a.W1 = W1.data_ptr()
            a.W2 = W2.data_ptr() if W2 is not None else None
            a.M = M.data_ptr()
            a.opt_state = state.data_ptr()
            a.loss_history = hist.data_ptr()
            a.cfg = cfg
        n = ctypes.c_size_t(0)
        _check(lib().cafeq_layer_workspace_size(self.arr, ctypes.c_int(self.n), ctypes.byref(n)), "cafeq_layer_workspace_size")
        self.ws_bytes = int(n.value)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.prepared = False

    def set_lr(self, i, lr):
        self.arr[i].cfg.lr = lr

    def prepare(self):
        _check(lib().cafeq_layer_prepare(self.arr, ctypes.c_int(self.n), _p(self.status), _p(self.ws),
                                         ctypes.c_size_t(self.ws_bytes), _stream()), "cafeq_layer_prepare")
        self.prepared = True

    def fallbacks(self) -> int:
        """Blocks re-inverted by elimination since prepare() (synchronises)."""
        n = ctypes.c_int(0)
        _check(lib().cafeq_layer_debug_fallbacks(self.arr, ctypes.c_int(self.n), _p(self.ws), ctypes.c_size_t(self.ws_bytes),
                                                 ctypes.byref(n)), "cafeq_layer_debug_fallbacks")
        return int(n.value)

    def step(self, steps=1):
        if not self.prepared:
            self.prepare()
        if steps > self.max_steps:
            raise ValueError("steps exceeds the loss-history rows this object allocated")
        _check(lib().cafeq_optimize_layer(self.arr, ctypes.c_int(self.n), ctypes.c_int(steps), _p(self.status), _p(self.ws),
                                          ctypes.c_size_t(self.ws_bytes), _stream()), "cafeq_optimize_layer")
