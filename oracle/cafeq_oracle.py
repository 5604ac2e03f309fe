"""CPU oracle for the CafeQ per-matrix optimisation path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 numpy restatement of what the paper defines, written to
be checked against the paper by eye.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it; the CUDA product never does, and
this file imports nothing from the CUDA package.

Conventions (the build's, stated once):
  * a linear weight is stored [d_out, d_in]; quantisation groups are `group`
    consecutive entries along d_in, one scale per (row, group); group 0 means
    one group per row (per-channel);
  * a block-diagonal operator is an array T[nb, k, k]; `axis="in"` applies it
    to the d_in index, U[o, B*k+i] = sum_j T[B//r][i, j] W[o, B*k+j];
    `axis="out"` applies it to the d_out index,
    U[B*k+i, c] = sum_j T[B//r][i, j] W[B*k+j, c]; `r` consecutive blocks of the
    matrix may share one operator block (grouped-query attention heads);
  * operands that the device feeds to its tensor cores are bf16: the transform
    that is actually deployed is M_c = bf16(M) (and bf16(inv(M_c)) on the side of
    a pair that receives the inverse).  The oracle rounds the same way and does
    everything else in float64.
  * two places are float32 on purpose because they decide integers: the group
    scale s = fl32(a)/fl32(qmax) and the quotient fl32(U)/s that is rounded to
    the code (both IEEE round-to-nearest divisions, ties of the rounding to even).

Sections cited: Eq. 1-2 (uniform quantiser and its error bound), Section 4
(l2 proxy, Eq. 3), Section 4.1 (block-diagonal transform, Eq. 4 = the
stochastic-rounding surrogate), Section 4.2 (paired transform, Eq. 5 = PQE, the
LogSumExp surrogate), Section 5 (Algorithm 1 and its toy example), Appendix D
(orthonormality regulariser, Adam, alternative pseudo-losses).

Pin status: every function here is pinned by tests/test_oracle_pins.py except
the trend checks on synthetic weights (numeric values of Tables 1-2 need the
trained checkpoints: "parity unpinned" for those values only).
"""
from __future__ import annotations

import itertools

import numpy as np

F32 = np.float32


# ---------------------------------------------------------------------------
# number formats
# ---------------------------------------------------------------------------
def round_bf16(x):
    """Round to the nearest bf16 value (ties to even); returns float64."""
    x32 = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = x32.view(np.uint32).astype(np.uint64)
    keep = (u >> 16) & 1
    u = ((u + 0x7FFF + keep) >> 16) << 16
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


def qmax_of(bits: int) -> int:
    """Largest code of the symmetric restricted-range grid: 2^(b-1) - 1."""
    return (1 << (bits - 1)) - 1


# ---------------------------------------------------------------------------
# Eq. 1: uniform quantiser (asymmetric min/max form, exactly as printed)
# ---------------------------------------------------------------------------
def quant_asym(w, bits: int):
    """Eq. 1 on one block of weights `w` (any shape, one scale for the whole block)."""
    w = np.asarray(w, dtype=np.float64)
    wmin, wmax = w.min(), w.max()
    if wmax == wmin:
        return w.copy(), 0.0
    s = (wmax - wmin) / (2 ** bits - 1)
    return s * np.rint((w - wmin) / s) + wmin, s


# ---------------------------------------------------------------------------
# symmetric absmax group quantiser (the workload's form of Eq. 1)
# ---------------------------------------------------------------------------
def _groups(d_in: int, group: int) -> int:
    g = d_in if group in (0, None) else group
    if d_in % g:
        raise ValueError("group must divide d_in")
    return g


def group_absmax(U, group: int, dtype=F32):
    """a[o, G] = max |fl32(U)| over the group, and the lowest index attaining it."""
    U32 = np.asarray(U, dtype=np.float64).astype(dtype)
    d_out, d_in = U32.shape
    g = _groups(d_in, group)
    A = np.abs(U32).reshape(d_out, d_in // g, g)
    idx = A.argmax(axis=2)                       # first (lowest) index on ties
    a = np.take_along_axis(A, idx[..., None], axis=2)[..., 0]
    return a, idx


def quant_sym(U, bits: int, group: int, offsets=None, dtype=F32):
    """Symmetric group quantiser.

    a = group absmax of fl32(U); s = a/qmax (fp32 division); code
    q = clamp(rne(fl32(U)/s)) (fp32 division), or with `offsets` (same shape as U,
    values in [0,1]) q = clamp(floor(fl32(U)/s) + offsets), except that an entry attaining its group's
    absmax is always coded +-qmax (its exact quotient is +-qmax, a point where floor is discontinuous: the fp32
    quotient lands one ulp above or below depending on the last bits of the maximum).  An all-zero group has
    s = 0 and codes 0.  Returns dict(a, s, idx, q, Uhat) with Uhat = s*q in float64.
    dtype=float64 replaces the normative fp32 steps by float64 ones (finite-difference checks only).
    """
    U = np.asarray(U, dtype=np.float64)
    U32 = U.astype(dtype)
    d_out, d_in = U.shape
    g = _groups(d_in, group)
    qm = qmax_of(bits)
    a, idx = group_absmax(U, group, dtype)
    s = (a / dtype(qm)).astype(dtype)
    s_e = np.repeat(s, g, axis=1)
    with np.errstate(divide="ignore", invalid="ignore"):
        x = (U32 / s_e).astype(dtype)
    x = np.where(s_e > 0, x, dtype(0))
    if offsets is None:
        q = np.rint(x)
    else:
        q = np.floor(x).astype(np.float64) + np.asarray(offsets, dtype=np.float64)
        a_e = np.repeat(a, g, axis=1)
        at_max = (np.abs(U32) >= a_e) & (a_e > 0)
        q = np.where(at_max, np.sign(U32).astype(np.float64) * qm, q)
    q = np.clip(q, -qm, qm)
    Uhat = s_e.astype(np.float64) * q
    if offsets is None:
        q = q.astype(np.int32)
    return dict(a=a, s=s, idx=idx, q=q, Uhat=Uhat)


# ---------------------------------------------------------------------------
# block-diagonal operators (Section 4.1)
# ---------------------------------------------------------------------------
def block_inverse(M):
    """Inverse of every k x k block: Gauss-Jordan elimination with partial pivoting."""
    M = np.asarray(M, dtype=np.float64)
    nb, k, _ = M.shape
    A = np.concatenate([M.copy(), np.broadcast_to(np.eye(k), (nb, k, k)).copy()], axis=2)
    ar = np.arange(nb)
    for p in range(k):
        piv = np.abs(A[:, p:, p]).argmax(axis=1) + p
        rows_p = A[ar, p].copy()
        A[ar, p] = A[ar, piv]
        A[ar, piv] = rows_p
        d = A[:, p, p]
        if np.any(d == 0):
            raise np.linalg.LinAlgError("singular block")
        A[:, p, :] /= d[:, None]
        f = A[:, :, p].copy()
        f[:, p] = 0.0
        A -= f[:, :, None] * A[:, p, None, :]
    return A[:, :, k:]


def apply_blocks(W, T, axis: str, r: int = 1):
    """U = T o W along `axis` ("in" or "out"); r matrix blocks share one operator block."""
    W = np.asarray(W, dtype=np.float64)
    T = np.asarray(T, dtype=np.float64)
    nbT, k, _ = T.shape
    d_out, d_in = W.shape
    if axis == "in":
        nb = d_in // k
        if nb * k != d_in or nb != nbT * r:
            raise ValueError("operator does not tile d_in")
        Wb = W.reshape(d_out, nb, k)
        Te = np.repeat(T, r, axis=0)                       # [nb, k, k]
        Ub = np.matmul(Wb.transpose(1, 0, 2), Te.transpose(0, 2, 1))   # [nb, d_out, k]: rows times T^T
        return np.ascontiguousarray(Ub.transpose(1, 0, 2)).reshape(d_out, d_in)
    if axis == "out":
        nb = d_out // k
        if nb * k != d_out or nb != nbT * r:
            raise ValueError("operator does not tile d_out")
        Wb = W.reshape(nb, k, d_in)
        Te = np.repeat(T, r, axis=0)
        return np.matmul(Te, Wb).reshape(d_out, d_in)
    raise ValueError("axis")


def operator_grad(gU, W, k: int, axis: str, r: int = 1):
    """dL/dT[B][i, j] = sum over the free index of gU[.., i] W[.., j], summed over replicas."""
    gU = np.asarray(gU, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    d_out, d_in = W.shape
    if axis == "in":
        nb = d_in // k
        g = np.matmul(gU.reshape(d_out, nb, k).transpose(1, 2, 0), W.reshape(d_out, nb, k).transpose(1, 0, 2))
    else:
        nb = d_out // k
        g = np.matmul(gU.reshape(nb, k, d_in), W.reshape(nb, k, d_in).transpose(0, 2, 1))
    return g.reshape(nb // r, r, k, k).sum(axis=1)


def _entry_weights(c, shape, k: int, axis: str, r: int = 1):
    """c_{t(e)} for every entry e: t is the entry's index along the transformed axis."""
    d_out, d_in = shape
    ce = np.repeat(np.asarray(c, dtype=np.float64), r, axis=0).reshape(-1)   # per transformed index
    if axis == "in":
        return np.broadcast_to(ce[None, :], (d_out, d_in))
    return np.broadcast_to(ce[:, None], (d_out, d_in))


def _route_to_argmax(dL_da, U, idx, group: int):
    """Sub-gradient of the group absmax: all of dL/da goes to the arg-max entry, times its sign."""
    d_out, d_in = U.shape
    g = _groups(d_in, group)
    gU = np.zeros((d_out, d_in // g, g))
    Ug = np.asarray(U, dtype=np.float64).astype(F32).reshape(d_out, d_in // g, g)
    sel = np.take_along_axis(Ug, idx[..., None], axis=2)
    np.put_along_axis(gU, idx[..., None], dL_da[..., None] * np.sign(sel), axis=2)
    return gU.reshape(d_out, d_in)


# ---------------------------------------------------------------------------
# single matrix: l2 proxy (Eq. 3) and its surrogate (Eq. 4)
# ---------------------------------------------------------------------------
def single_forward(W, M, bits: int, group: int, axis: str = "in", kappa=None, offsets=None,
                   prec: str = "bf16"):
    """One forward evaluation for a single matrix.

    M_c = bf16(M), Minv = inv(M_c), U = M_c o W, (a, s, q, Uhat) = Q(U),
    Delta = Uhat - U, E = Minv o Delta, L2 = ||E||_F^2 = ||M^-1 Q(MW) - W||_F^2 (Eq. 3),
    c_t = sum_i Minv[i, t]^2, surrogate = kappa * sum_entries c_t a_G^2 (Eq. 4 written
    per entry; kappa = 1/(2^N - 1)^2 by default).  prec="exact" skips the bf16 rounding of M
    (used by finite-difference checks, which cannot see through a rounding step).
    """
    W = np.asarray(W, dtype=np.float64)
    Mc = round_bf16(M) if prec == "bf16" else np.asarray(M, dtype=np.float64)
    k = Mc.shape[1]
    Minv = block_inverse(Mc)
    U = apply_blocks(W, Mc, axis)
    Q = quant_sym(U, bits, group, offsets, F32 if prec == "bf16" else np.float64)
    Delta = Q["Uhat"] - U
    E = apply_blocks(Delta, Minv, axis)
    L2 = float(np.sum(E * E))
    c = np.sum(Minv * Minv, axis=1)                              # [nb, k] column square norms
    if kappa is None:
        kappa = 1.0 / (2 ** bits - 1) ** 2
    g = _groups(W.shape[1], group)
    a_e = np.repeat(Q["a"].astype(np.float64), g, axis=1)        # a_G for every entry
    ce = _entry_weights(c, W.shape, k, axis)
    sur = float(kappa * np.sum(ce * a_e * a_e))
    out = dict(Mc=Mc, Minv=Minv, U=U, Delta=Delta, E=E, L2=L2, c=c, surrogate=sur,
               kappa=kappa, normW2=float(np.sum(W * W)))
    out.update(Q)
    out["offsets"] = offsets
    out["rel_l2"] = float(np.sqrt(L2 / out["normW2"])) if out["normW2"] > 0 else 0.0
    return out


def single_grad_surrogate(W, fwd, group: int, axis: str = "in"):
    """Gradient of the surrogate (Eq. 4) with respect to M.

    dL/da_G = 2 kappa a_G sum_{e in G} c_t(e), routed to the arg-max entry;
    dL/dMinv[i, t] = 2 kappa Minv[i, t] A_t with A_t = sum of a_G^2 over entries whose
    transformed index is t; and d(M^-1) = -M^-1 dM M^-1.
    """
    W = np.asarray(W, dtype=np.float64)
    Minv, c, kappa = fwd["Minv"], fwd["c"], fwd["kappa"]
    nb, k, _ = Minv.shape
    d_out, d_in = W.shape
    g = _groups(d_in, group)
    a = fwd["a"].astype(np.float64)
    ce = _entry_weights(c, W.shape, k, axis)
    Csum = ce.reshape(d_out, d_in // g, g).sum(axis=2)           # sum of c over the group's entries
    gU = _route_to_argmax(2.0 * kappa * a * Csum, fwd["U"], fwd["idx"], group)
    gM = operator_grad(gU, W, k, axis)
    a2_e = np.repeat(a * a, g, axis=1)
    if axis == "in":
        A = a2_e.sum(axis=0).reshape(nb, k)
    else:
        A = a2_e.sum(axis=1).reshape(nb, k)
    gMinv = 2.0 * kappa * Minv * A[:, None, :]
    MinvT = np.transpose(Minv, (0, 2, 1))
    return gM - MinvT @ gMinv @ MinvT


def single_grad_ste(W, fwd, bits: int, group: int, axis: str = "in"):
    """Straight-through gradient of L2 = ||Minv (Uhat - U)||^2 with respect to M.

    round'() := 1, so dUhat/dU = 1 (cancels against -U) and dUhat/ds_G = q - U/s_G;
    s_G = |U_e*|/qmax.  What remains: the Minv path 2 E Delta^T and the scale path
    through the arg-max entry.
    """
    W = np.asarray(W, dtype=np.float64)
    Minv, U = fwd["Minv"], fwd["U"]
    nb, k, _ = Minv.shape
    d_out, d_in = W.shape
    g = _groups(d_in, group)
    qm = qmax_of(bits)
    MinvT = np.transpose(Minv, (0, 2, 1))
    gDelta = 2.0 * apply_blocks(fwd["E"], MinvT, axis)
    gMinv = 2.0 * operator_grad(fwd["E"], fwd["Delta"], k, axis)
    s_e = np.repeat(fwd["s"].astype(np.float64), g, axis=1)
    with np.errstate(divide="ignore", invalid="ignore"):
        resid = np.where(s_e > 0, fwd["q"] - U / s_e, 0.0)
    dL_ds = (gDelta * resid).reshape(d_out, d_in // g, g).sum(axis=2)
    gU = _route_to_argmax(dL_ds / qm, U, fwd["idx"], group)
    gM = operator_grad(gU, W, k, axis)
    return gM - MinvT @ gMinv @ MinvT


def single_grad_offsets(fwd, group: int, axis: str = "in"):
    """dL2/d rho for soft rounding offsets rho in [0, 1] (not in the paper: the workload statement's learned rounding
    offsets).  With code q = floor(U/s) + rho and scales kept at their round-to-nearest values,
    Uhat = s (floor(U/s) + rho), so dUhat/drho = s and dL2/drho = s * dL2/dUhat = s * (2 Minv^T E)  (Eq. 3's
    residual E = Minv (Uhat - U)).  The entries attaining their group's absmax are coded +-qmax whatever their offset
    (quant_sym) and have no gradient."""
    Minv = fwd["Minv"]
    MinvT = np.transpose(Minv, (0, 2, 1))
    gUhat = 2.0 * apply_blocks(fwd["E"], MinvT, axis)
    g = _groups(gUhat.shape[1], group)
    s_e = np.repeat(fwd["s"].astype(np.float64), g, axis=1)
    a_e = np.repeat(fwd["a"], g, axis=1)
    at_max = np.abs(np.asarray(fwd["U"], dtype=np.float64).astype(F32)) >= a_e
    return np.where(at_max, 0.0, s_e * gUhat)


def project_offsets(rho):
    """Soft offsets live in [0, 1]: projection after a gradient step."""
    return np.clip(np.asarray(rho, dtype=np.float64), 0.0, 1.0)


def harden_offsets(rho):
    """Soft -> hard: ceil where rho >= 1/2, floor otherwise."""
    return (np.asarray(rho, dtype=np.float64) >= 0.5).astype(np.float64)


# ---------------------------------------------------------------------------
# pair: PQE (Eq. 5), LogSumExp surrogate, orthonormality regulariser (App. D)
# ---------------------------------------------------------------------------
def expand_rows(X, k: int, r: int):
    """Repeat every k-row block r times consecutively (kv head -> its r query heads)."""
    X = np.asarray(X)
    if r == 1:
        return X
    nb = X.shape[0] // k
    return np.repeat(X.reshape(nb, 1, k, -1), r, axis=1).reshape(nb * r * k, -1)


def fold_rows(X, k: int, r: int):
    """Adjoint of expand_rows: sum the r replicas of every block."""
    X = np.asarray(X)
    if r == 1:
        return X
    nb = X.shape[0] // (k * r)
    return X.reshape(nb, r, k, -1).sum(axis=1).reshape(nb * k, -1)


def pair_product(A1s, A2s, k: int, r: int):
    """W1 W2 in the paper's orientation: P[x, y] = sum_h A1exp[h, x] A2s[y, h]."""
    return expand_rows(np.asarray(A1s, dtype=np.float64), k, r).T @ np.asarray(A2s, dtype=np.float64).T


def orth_penalty(M):
    """||M M^T - I||_F / sqrt(d) on the whole block-diagonal M, and its gradient.

    The norm is not squared, so its gradient has no limit at M M^T = I; exactly there (norm 0) the
    sub-gradient 0 is taken.  (A device that forms M M^T in fp32 cannot tell a rotation from its
    rounding noise; that floor belongs to the device and to the inputs a parity test chooses, not here.)"""
    M = np.asarray(M, dtype=np.float64)
    nb, k, _ = M.shape
    R = M @ np.transpose(M, (0, 2, 1)) - np.eye(k)
    nrm = np.sqrt(np.sum(R * R))
    d = nb * k
    if nrm == 0.0:
        return 0.0, np.zeros_like(M)
    return float(nrm / np.sqrt(d)), (2.0 * R @ M) / (nrm * np.sqrt(d))


def pair_forward(W1s, W2s, M, bits: int, group1: int, group2: int, r: int = 1,
                 t: float = 5.0, lam: float = 0.0, want_pqe: bool = True, prec: str = "bf16", Minv_c=None,
                 objective: str = "lse"):
    """Forward for a coupled pair.

    Stored W1s is [h, d1] (the paper's W1 transposed), stored W2s is [d3, r*h].
    U = W1 M  <=> Us = M_c^T o W1s on the d_out axis;  V = M^-1 W2 <=> Vs = Minv_c o W2s on
    the d_in axis with Minv_c = bf16(inv(M_c)).  LSE = (1/t) log(sum_G e^{t a_G}) over the
    group maxima of both (the quantiser's own groups), plus lam * orth_penalty(M).
    PQE = ||Uhat Vhat - W1 W2||_F, relative to ||W1 W2||_F.
    Minv_c: optional, the second factor's operator given from outside (an inverse rounded to bf16 elsewhere:
    which way an entry of an inverse rounds to bf16 depends on its last bits, so two computations of
    bf16(inv(M_c)) can differ in single entries by one bf16 step; a caller that compares integer codes
    passes the operator that was actually applied).  Gradients still differentiate through inv(M_c).
    objective: "lse" (Section 4.2), or the alternatives of Appendix D.1 over the same group maxima:
    "sumsq" = mean of the squared maxima of U + mean of the squared maxima of V; "sumsq_weighted" =
    ||V||_F * mean(squared maxima of U) + ||U||_F * mean(squared maxima of V) (an error in one factor is magnified by
    the norm of the other).  out["surrogate"] holds the chosen objective's value, out["loss"] adds lam * penalty.
    """
    W1s = np.asarray(W1s, dtype=np.float64)
    W2s = np.asarray(W2s, dtype=np.float64)
    Mc = round_bf16(M) if prec == "bf16" else np.asarray(M, dtype=np.float64)
    k = Mc.shape[1]
    Minv = block_inverse(Mc)
    if Minv_c is not None:
        Minv_c = np.asarray(Minv_c, dtype=np.float64)
    else:
        Minv_c = round_bf16(Minv) if prec == "bf16" else Minv
    McT = np.transpose(Mc, (0, 2, 1))
    U = apply_blocks(W1s, McT, "out", 1)
    V = apply_blocks(W2s, Minv_c, "in", r)
    fl = F32 if prec == "bf16" else np.float64
    QU = quant_sym(U, bits, group1, None, fl)
    QV = quant_sym(V, bits, group2, None, fl)
    au = QU["a"].astype(np.float64)
    av = QV["a"].astype(np.float64)
    amax = max(au.max(), av.max())
    Z = np.sum(np.exp(t * (au - amax))) + np.sum(np.exp(t * (av - amax)))
    lse = amax + np.log(Z) / t
    wu = np.exp(t * (au - amax)) / Z                             # softmax weights = dLSE/da
    wv = np.exp(t * (av - amax)) / Z
    pen, gpen = orth_penalty(np.asarray(M, dtype=np.float64))
    if objective == "lse":
        sur = lse
    else:
        su, sv = float(np.mean(au * au)), float(np.mean(av * av))
        nu, nv = float(np.sqrt(np.sum(U * U))), float(np.sqrt(np.sum(V * V)))
        if objective == "sumsq":
            sur, wu, wv = su + sv, 2.0 * au / au.size, 2.0 * av / av.size      # w = d objective / d maximum
        elif objective == "sumsq_weighted":
            sur, wu, wv = nv * su + nu * sv, nv * 2.0 * au / au.size, nu * 2.0 * av / av.size
        else:
            raise ValueError("objective")
    out = dict(Mc=Mc, Minv=Minv, Minv_c=Minv_c, U=U, V=V, QU=QU, QV=QV, lse=float(lse), wu=wu, wv=wv,
               orth=pen, gorth=gpen, loss=float(sur + lam * pen), surrogate=float(sur), objective=objective,
               k=k, r=r, lam=lam, t=t)
    if objective == "sumsq_weighted":
        out.update(su=su, sv=sv, nu=nu, nv=nv)
    if want_pqe:
        P = pair_product(W1s, W2s, k, r)
        R = pair_product(QU["Uhat"], QV["Uhat"], k, r) - P
        out.update(P=P, R=R, pqe=float(np.sqrt(np.sum(R * R))), normP=float(np.sqrt(np.sum(P * P))))
        out["rel_pqe"] = out["pqe"] / out["normP"] if out["normP"] > 0 else 0.0
    return out


def _pair_chain(W1s, W2s, fwd, gU, gV):
    """Chain dL/dU, dL/dV to M: U-side operator is M^T, V-side operator is Minv."""
    k, r, Minv = fwd["k"], fwd["r"], fwd["Minv"]
    gT = operator_grad(gU, W1s, k, "out", 1)                     # gradient w.r.t. M^T blocks
    gM = np.transpose(gT, (0, 2, 1))
    gMinv = operator_grad(gV, W2s, k, "in", r)
    MinvT = np.transpose(Minv, (0, 2, 1))
    return gM - MinvT @ gMinv @ MinvT


def pair_grad_lse(W1s, W2s, fwd, group1: int, group2: int):
    """Gradient of the pair surrogate + lam*orth: d objective / d group maximum (the softmax weights for
    LogSumExp, 2 a / count [times the other factor's norm] for the sums of squares of Appendix D.1) routed to the
    arg-max entries; the weighted form adds the dense terms mean(a_U^2) V / ||V||_F and mean(a_V^2) U / ||U||_F."""
    gU = _route_to_argmax(fwd["wu"], fwd["U"], fwd["QU"]["idx"], group1)
    gV = _route_to_argmax(fwd["wv"], fwd["V"], fwd["QV"]["idx"], group2)
    if fwd.get("objective") == "sumsq_weighted":
        gU = gU + fwd["sv"] * fwd["U"] / fwd["nu"]
        gV = gV + fwd["su"] * fwd["V"] / fwd["nv"]
    return _pair_chain(np.asarray(W1s, np.float64), np.asarray(W2s, np.float64), fwd, gU, gV) \
        + fwd["lam"] * fwd["gorth"]


def pair_grad_pqe_ste(W1s, W2s, fwd, bits: int, group1: int, group2: int):
    """Straight-through gradient of PQE^2 = ||Uhat Vhat - P||_F^2 with respect to M."""
    k, r = fwd["k"], fwd["r"]
    qm = qmax_of(bits)
    R = fwd["R"]
    Uh, Vh = fwd["QU"]["Uhat"], fwd["QV"]["Uhat"]
    gUh = fold_rows(2.0 * (R @ Vh).T, k, r)                      # [h, d1]
    gVh = 2.0 * (expand_rows(Uh, k, r) @ R).T                    # [d3, r*h]

    def through_quantiser(gXh, X, Q, group):
        d_out, d_in = X.shape
        g = _groups(d_in, group)
        s_e = np.repeat(Q["s"].astype(np.float64), g, axis=1)
        with np.errstate(divide="ignore", invalid="ignore"):
            resid = np.where(s_e > 0, Q["q"] - X / s_e, 0.0)
        dL_ds = (gXh * resid).reshape(d_out, d_in // g, g).sum(axis=2)
        return gXh + _route_to_argmax(dL_ds / qm, X, Q["idx"], group)

    gU = through_quantiser(gUh, fwd["U"], fwd["QU"], group1)
    gV = through_quantiser(gVh, fwd["V"], fwd["QV"], group2)
    return _pair_chain(np.asarray(W1s, np.float64), np.asarray(W2s, np.float64), fwd, gU, gV)


# ---------------------------------------------------------------------------
# optimisers (Section 4.1: gradient descent; App. D: Adam)
# ---------------------------------------------------------------------------
def gd_step(M, g, lr: float):
    return np.asarray(M, dtype=np.float64) - lr * g


def adam_step(M, g, state, lr: float, beta1: float = 0.1, beta2: float = 0.999, eps: float = 1e-8):
    """state = (m, v, step) ; returns (M_new, state_new)."""
    m, v, step = state
    step += 1
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    mh = m / (1.0 - beta1 ** step)
    vh = v / (1.0 - beta2 ** step)
    return np.asarray(M, dtype=np.float64) - lr * mh / (np.sqrt(vh) + eps), (m, v, step)


def cayley_step(M, g, momentum, lr: float, beta: float = 0.1):
    """One step of stochastic gradient descent on the rotations by the Cayley transform (Appendix D.2's strictly
    orthonormal baseline), per block: momentum V <- beta V + g; A = V M^T - M V^T (skew-symmetric: the direction in
    the tangent space); M <- (I + lr/2 A)^-1 (I - lr/2 A) M, which is a rotation times M, so an orthonormal M stays
    orthonormal to rounding.  Returns (M_new, V)."""
    M = np.asarray(M, dtype=np.float64)
    V = beta * np.asarray(momentum, dtype=np.float64) + np.asarray(g, dtype=np.float64)
    A = V @ np.transpose(M, (0, 2, 1)) - M @ np.transpose(V, (0, 2, 1))
    eye = np.eye(M.shape[1])
    out = np.empty_like(M)
    for b in range(M.shape[0]):
        out[b] = np.linalg.solve(eye + 0.5 * lr * A[b], (eye - 0.5 * lr * A[b]) @ M[b])
    return out, V


def optimize_single(W, M0, bits: int, group: int, axis: str, steps: int, lr: float, kappa=None):
    """Gradient descent on the surrogate; returns (M, history[steps, 2] = surrogate, L2)."""
    M = np.asarray(M0, dtype=np.float32).astype(np.float64)
    hist = np.zeros((steps, 2))
    for it in range(steps):
        f = single_forward(W, M, bits, group, axis, kappa)
        hist[it] = (f["surrogate"], f["L2"])
        M = gd_step(M, single_grad_surrogate(W, f, group, axis), lr)
        M = M.astype(np.float32).astype(np.float64)              # master parameters are fp32
    return M, hist


def optimize_pair(W1s, W2s, M0, bits: int, group1: int, group2: int, r: int, steps: int, lr: float,
                  t: float = 5.0, lam: float = 0.1, beta1: float = 0.1, beta2: float = 0.999,
                  eps: float = 1e-8, want_pqe: bool = False, objective: str = "lse", optimizer: str = "adam"):
    """Adam (or Cayley SGD with momentum beta1) on the pair surrogate + lam*orth; returns (M, history[steps, 2] =
    loss, PQE or nan)."""
    M = np.asarray(M0, dtype=np.float32).astype(np.float64)
    st = (np.zeros_like(M), np.zeros_like(M), 0)
    mom = np.zeros_like(M)
    hist = np.full((steps, 2), np.nan)
    for it in range(steps):
        f = pair_forward(W1s, W2s, M, bits, group1, group2, r, t, lam, want_pqe, objective=objective)
        hist[it, 0] = f["loss"]
        if want_pqe:
            hist[it, 1] = f["pqe"]
        g = pair_grad_lse(W1s, W2s, f, group1, group2)
        if optimizer == "cayley":
            M, mom = cayley_step(M, g, mom, lr, beta1)
        else:
            M, st = adam_step(M, g, st, lr, beta1, beta2, eps)
        M = M.astype(np.float32).astype(np.float64)
    return M, hist


# ---------------------------------------------------------------------------
# Algorithm 1: adaptive rounding for a matrix product
# ---------------------------------------------------------------------------
def pinv(A, rcond=None):
    """Moore-Penrose inverse from the SVD; singular values below rcond*sigma_max dropped."""
    A = np.asarray(A, dtype=np.float64)
    if rcond is None:
        rcond = max(A.shape) * 2.2e-16
    u, s, vt = np.linalg.svd(A, full_matrices=False)
    keep = s > rcond * (s[0] if s.size else 0.0)
    sinv = np.where(keep, 1.0 / np.where(keep, s, 1.0), 0.0)
    return (vt.T * sinv) @ u.T


def adaptive_round_alg1(W1, W2, Q1, Q2, iters: int):
    """Algorithm 1 verbatim, in the paper's orientation (W1: d1 x h, W2: h x d2).

    Q1, Q2 map a float64 matrix to its quantised (dequantised-value) matrix.
    Returns (W1hat, W2hat, pqe_history) with pqe_history[0] the independent-rounding
    error and one entry after every half-iteration.
    """
    W1 = np.asarray(W1, dtype=np.float64)
    W2 = np.asarray(W2, dtype=np.float64)
    P = W1 @ W2
    W1h = Q1(W1)
    W2h = Q2(W2)
    hist = [float(np.linalg.norm(W1h @ W2h - P))]
    for _ in range(iters):
        W2h = Q2(pinv(W1h) @ P)
        hist.append(float(np.linalg.norm(W1h @ W2h - P)))
        W1h = Q1(P @ pinv(W2h))
        hist.append(float(np.linalg.norm(W1h @ W2h - P)))
    return W1h, W2h, hist


def adaptive_round_stored(U1s, V2s, bits: int, group1: int, group2: int, k: int, r: int, iters: int):
    """Algorithm 1 on a pair in stored layout with r query-head replicas per kv block.

    With E the row-expansion (kv block -> its r replicas) the product is
    P = (E U1s)^T V2s^T.  The second factor's update is Q(pinv((E Uhat)^T) P) as printed; the
    first factor must keep the replica structure, so its least-squares target is
    P pinv(fold(Vhat^T)) (identical to the printed line when r = 1).
    Returns dict(q1, s1, q2, s2, pqe[2*iters+1]).
    """
    U1s = np.asarray(U1s, dtype=np.float64)
    V2s = np.asarray(V2s, dtype=np.float64)
    P = pair_product(U1s, V2s, k, r)                              # [d1, d3]
    Q1 = quant_sym(U1s, bits, group1)
    Q2 = quant_sym(V2s, bits, group2)

    def err(Qa, Qb):
        return float(np.linalg.norm(pair_product(Qa["Uhat"], Qb["Uhat"], k, r) - P))

    hist = [err(Q1, Q2)]
    for _ in range(iters):
        A = expand_rows(Q1["Uhat"], k, r).T                       # [d1, r*h]
        Q2 = quant_sym((pinv(A) @ P).T, bits, group2)             # stored [d3, r*h]
        hist.append(err(Q1, Q2))
        Bf = fold_rows(Q2["Uhat"].T, k, r)                        # [h, d3]
        Q1 = quant_sym((P @ pinv(Bf)).T, bits, group1)            # stored [h, d1]
        hist.append(err(Q1, Q2))
    return dict(q1=Q1["q"], s1=Q1["s"], q2=Q2["q"], s2=Q2["s"], Uhat1=Q1["Uhat"], Uhat2=Q2["Uhat"],
                pqe=np.array(hist))


LEARN_LAMBDA = 0.5  # final weight of the push towards {0, 1}


def adaptive_round_learned(U1s, V2s, bits: int, group1: int, group2: int, k: int, r: int, iters: int):
    """Learned rounding offsets for a coupled product (not in the paper, whose adaptive rounding is Algorithm 1; this
    is the workload statement's gradient-learned alternative, defined here).

    Scales stay at their round-to-nearest values; codes are floor(x) + rho with soft offsets rho in [0, 1], started
    at the fractional parts (Uhat = U exactly, zero error).  Iteration t = 1..iters, on L = || Uhat Vhat - U V ||_F^2
    (Eq. 5 squared): for the first factor, the direction d = (dL/drho) / (per-entry curvature) = gUhat / (s H) with
    H = 2 ||the second factor's matching (replica-folded) row||^2, an exact line search along it (L is quadratic in one
    factor's offsets), projection to [0, 1]; the same for the second factor at the updated first; then both are pushed
    towards the nearer of {0, 1} by lambda_t (2 rho - 1), lambda_t = LEARN_LAMBDA * t / iters, and projected.  At the
    end the offsets are hardened at 1/2.  Entries attaining their group's absmax have no offset (quant_sym).
    Returns dict(Uhat, Vhat, q1, q2, s1, s2, rho1, rho2, history): history[0] the product error of independent
    round-to-nearest, history[t] that of the soft iterate entering iteration t, history[iters + 1] of the hardened result.
    """
    U = np.asarray(U1s, dtype=np.float64)
    V = np.asarray(V2s, dtype=np.float64)
    P = pair_product(U, V, k, r)
    Q1, Q2 = quant_sym(U, bits, group1), quant_sym(V, bits, group2)
    hist = [float(np.linalg.norm(pair_product(Q1["Uhat"], Q2["Uhat"], k, r) - P))]

    def frac(X, Q, group):
        g = _groups(X.shape[1], group)
        s_e = np.repeat(Q["s"], g, axis=1)
        with np.errstate(divide="ignore", invalid="ignore"):
            x = (X.astype(F32) / s_e).astype(F32)
        x = np.where(s_e > 0, x, F32(0)).astype(np.float64)
        a_e = np.repeat(Q["a"], g, axis=1)
        free = (np.abs(X.astype(F32)) < a_e) & (s_e > 0)
        return x - np.floor(x), s_e.astype(np.float64), free

    def line_search(R, D):
        dd = float(np.sum(D * D))
        return float(np.sum(R * D)) / dd if dd > 0 else 0.0

    rho1, s1, free1 = frac(U, Q1, group1)
    rho2, s2, free2 = frac(V, Q2, group2)
    for t in range(1, iters + 1):
        Uh = quant_sym(U, bits, group1, rho1)["Uhat"]
        Vh = quant_sym(V, bits, group2, rho2)["Uhat"]
        R = pair_product(Uh, Vh, k, r) - P
        hist.append(float(np.linalg.norm(R)))
        # first factor
        gUh = fold_rows(2.0 * (R @ Vh).T, k, r)                       # [h, d1]
        Bf = fold_rows(Vh.T, k, r)                                    # [h, d3]: the rows that meet U's rows
        H1 = 2.0 * np.sum(Bf * Bf, axis=1)
        with np.errstate(divide="ignore", invalid="ignore"):
            dr1 = np.where(free1 & (H1[:, None] > 0), gUh / (s1 * H1[:, None]), 0.0)
        alpha = line_search(R, pair_product(s1 * dr1, Vh, k, r))
        rho1 = np.clip(rho1 - alpha * dr1, 0.0, 1.0)
        # second factor, at the updated first
        Uh = quant_sym(U, bits, group1, rho1)["Uhat"]
        R = pair_product(Uh, Vh, k, r) - P
        gVh = 2.0 * (expand_rows(Uh, k, r) @ R).T                     # [d3, r h]
        H2 = expand_rows((2.0 * np.sum(Uh * Uh, axis=1))[:, None], k, r)[:, 0]
        with np.errstate(divide="ignore", invalid="ignore"):
            dr2 = np.where(free2 & (H2[None, :] > 0), gVh / (s2 * H2[None, :]), 0.0)
        alpha = line_search(R, pair_product(Uh, s2 * dr2, k, r))
        rho2 = np.clip(rho2 - alpha * dr2, 0.0, 1.0)
        lam = LEARN_LAMBDA * t / iters
        rho1 = np.clip(rho1 + lam * (2.0 * rho1 - 1.0), 0.0, 1.0)
        rho2 = np.clip(rho2 + lam * (2.0 * rho2 - 1.0), 0.0, 1.0)
    F1 = quant_sym(U, bits, group1, harden_offsets(rho1))
    F2 = quant_sym(V, bits, group2, harden_offsets(rho2))
    hist.append(float(np.linalg.norm(pair_product(F1["Uhat"], F2["Uhat"], k, r) - P)))
    return dict(Uhat=F1["Uhat"], Vhat=F2["Uhat"], q1=F1["q"].astype(np.int32), q2=F2["q"].astype(np.int32),
                s1=Q1["s"], s2=Q2["s"], rho1=rho1, rho2=rho2, history=np.array(hist))


# ---------------------------------------------------------------------------
# exhaustive rounding search (tiny shapes only)
# ---------------------------------------------------------------------------
def brute_force_single(W, M, bits: int, group: int, axis: str = "in"):
    """All 2^n floor/ceil choices at the RTN scales; returns (best L2, best offsets, all L2)."""
    W = np.asarray(W, dtype=np.float64)
    n = W.size
    if n > 16:
        raise ValueError("brute force is for n <= 16")
    best, best_off, allv = np.inf, None, []
    for bitsv in itertools.product((0.0, 1.0), repeat=n):
        off = np.array(bitsv).reshape(W.shape)
        L2 = single_forward(W, M, bits, group, axis, offsets=off)["L2"]
        allv.append(L2)
        if L2 < best:
            best, best_off = L2, off
    return best, best_off, np.array(allv)


def pqe_with_offsets(U1s, V2s, bits, group1, group2, k, r, off1, off2):
    """Eq. 5 for a transformed pair (stored layouts) with both factors rounded by given floor/ceil offsets at
    their round-to-nearest scales: || Q_off1(U) Q_off2(V) - U V ||_F."""
    P = pair_product(U1s, V2s, k, r)
    Q1 = quant_sym(U1s, bits, group1, off1)
    Q2 = quant_sym(V2s, bits, group2, off2)
    return float(np.linalg.norm(pair_product(Q1["Uhat"], Q2["Uhat"], k, r) - P))


def brute_force_pair(U1s, V2s, bits: int, group1: int, group2: int, k: int, r: int):
    """All 2^(n1+n2) floor/ceil choices of both factors at their round-to-nearest scales (n1 + n2 <= 16):
    returns (best PQE, best offsets of the first factor, of the second, all PQE values in enumeration order)."""
    U1s = np.asarray(U1s, dtype=np.float64)
    V2s = np.asarray(V2s, dtype=np.float64)
    n1, n2 = U1s.size, V2s.size
    if n1 + n2 > 16:
        raise ValueError("brute force is for n1 + n2 <= 16")
    best, b1, b2, allv = np.inf, None, None, []
    for bitsv in itertools.product((0.0, 1.0), repeat=n1 + n2):
        o1 = np.array(bitsv[:n1]).reshape(U1s.shape)
        o2 = np.array(bitsv[n1:]).reshape(V2s.shape)
        v = pqe_with_offsets(U1s, V2s, bits, group1, group2, k, r, o1, o2)
        allv.append(v)
        if v < best:
            best, b1, b2 = v, o1, o2
    return best, b1, b2, np.array(allv)


def rtn_offsets(U, bits: int, group: int):
    """The floor/ceil offsets that reproduce round-to-nearest: offset = rne(x) - floor(x) for x = U/s."""
    Q = quant_sym(U, bits, group)
    g = _groups(np.asarray(U).shape[1], group)
    s_e = np.repeat(Q["s"], g, axis=1)
    with np.errstate(divide="ignore", invalid="ignore"):
        x = (np.asarray(U, dtype=np.float64).astype(F32) / s_e).astype(F32)
    x = np.where(s_e > 0, x, F32(0))
    return (np.rint(x) - np.floor(x)).astype(np.float64)


# ---------------------------------------------------------------------------
# packing: unsigned u = q + qmax, little-endian bit stream along d_in per row
# ---------------------------------------------------------------------------
def pack_codes(q, bits: int):
    q = np.asarray(q, dtype=np.int64)
    d_out, d_in = q.shape
    if (d_in * bits) % 8:
        raise ValueError("row does not fill whole bytes")
    u = (q + qmax_of(bits)).astype(np.uint64)
    out = np.zeros((d_out, d_in * bits // 8), dtype=np.uint8)
    for i in range(d_in):
        for b in range(bits):
            pos = i * bits + b
            out[:, pos // 8] |= (((u[:, i] >> np.uint64(b)) & np.uint64(1)) << np.uint64(pos % 8)).astype(np.uint8)
    return out


def unpack_codes(p, bits: int, d_in: int):
    p = np.asarray(p, dtype=np.uint8)
    d_out = p.shape[0]
    u = np.zeros((d_out, d_in), dtype=np.int64)
    for i in range(d_in):
        for b in range(bits):
            pos = i * bits + b
            u[:, i] |= ((p[:, pos // 8].astype(np.int64) >> (pos % 8)) & 1) << b
    return (u - qmax_of(bits)).astype(np.int32)


# ---------------------------------------------------------------------------
# inference side (Section 4.1: the transform is undone on the activations; the table of extra FLOPs / time)
# ---------------------------------------------------------------------------
def inference_apply(X, T, axis: str = "in", transpose: bool = False):
    """The activation-side multiplication that goes with a matrix quantised as Q(W o T) on its input axis:
    y = W x = (W o T)(T^-T x), so the activations X [tokens, d_in] are sent through P = T^-T, i.e. the inverse's
    blocks applied transposed.  This function applies a given block operator P = T (or T^T with transpose=True),
    rounded to bf16 as deployed, on the chosen axis in float64."""
    P = round_bf16(np.asarray(T, dtype=np.float32)).astype(np.float64)
    if transpose:
        P = np.transpose(P, (0, 2, 1))
    return apply_blocks(np.asarray(X, dtype=np.float64), P, axis, 1)


def dequant(packed, scales, bits: int, group: int, d_in: int):
    """What = scale * code from the packed stream (the layout of pack_codes) and the per-group scales [d_out, d_in/group]."""
    q = unpack_codes(packed, bits, d_in).astype(np.float64)
    s = np.repeat(np.asarray(scales, dtype=np.float64), group, axis=1)
    return s * q
