"""Pins for the CPU oracle: values the paper prints, closed forms, invariants, library
special cases, brute force and finite differences.  None of them uses the CUDA path."""
import os

import numpy as np
import pytest
import scipy.linalg

import cafeq_synth as syn
from oracle import cafeq_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = [int(v, 16) if v.startswith("0x") else float(v) for v in vals]
    return out


def _w(d_out, d_in, seed, scale=1.0):
    return syn.bf16_bits_to_f64(syn.weight_small(d_out, d_in, seed, scale))


def _heavy(d_out, d_in, seed):
    return syn.bf16_bits_to_f64(syn.weight_student_t(d_out, d_in, seed, 2, 10.0))


# ------------------------------------------------------------------ number formats
def test_round_bf16_matches_known_values():
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: ties-to-even gives 1; 1 + 3*2^-8 ties up to 1 + 2^-6
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -0.1, 3.0e38])
    r = orc.round_bf16(x)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2 ** -7 and r[3] == 1.0 + 2 ** -6
    assert abs(r[4] + 0.1) <= 0.1 * 2 ** -8
    import torch
    t = torch.tensor(x, dtype=torch.float64).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(r, t)


# ------------------------------------------------------------------ Eq. 1 / Eq. 2 and the toy example (P4, P5)
def test_toy_example_of_section_5():
    g = _read_golden("toy_pair.txt")
    W = np.array(g["W"]).reshape(2, 2)
    bits = int(g["bits"][0])
    Q = lambda X: orc.quant_asym(X, bits)[0]
    W1h, W2h, hist = orc.adaptive_round_alg1(W, W, Q, Q, iters=0)
    assert np.array_equal(W1h, np.array(g["what_independent"]).reshape(2, 2))
    assert hist[0] == pytest.approx(g["pqe_independent"][0], abs=1e-12)
    W1h, W2h, hist = orc.adaptive_round_alg1(W, W, Q, Q, iters=3)
    assert hist[1] == pytest.approx(g["pqe_half_iteration"][0], abs=1e-12)
    assert all(h == pytest.approx(0.36, abs=1e-12) for h in hist[1:])
    # the half-iteration iterate itself
    W2_half = Q(orc.pinv(Q(W)) @ W @ W)
    assert np.array_equal(W2_half, np.array(g["w2hat_half_iteration"]).reshape(2, 2))


def test_quant_asym_error_bound_eq2():
    rng = np.random.default_rng(0)
    for bits in (1, 2, 3, 4, 8):
        w = rng.standard_t(4, size=257)
        wh, s = orc.quant_asym(w, bits)
        bound = (w.max() - w.min()) / (2 * (2 ** bits - 1))
        assert np.max(np.abs(w - wh)) <= bound * (1 + 1e-12)
        assert bound <= np.max(np.abs(w)) / (2 ** bits - 1) * (1 + 1e-12)
        # values land on the grid wmin + s*integer
        lev = (wh - w.min()) / s
        assert np.allclose(lev, np.rint(lev), atol=1e-9)
        assert lev.min() >= -1e-9 and lev.max() <= 2 ** bits - 1 + 1e-9


def test_quant_sym_hand_example():
    g = _read_golden("rtn_hand.txt")
    U = np.array(g["values"]).reshape(1, -1)
    Q = orc.quant_sym(U, int(g["bits"][0]), 0)
    assert Q["s"][0, 0] == g["scale"][0]
    assert Q["q"].reshape(-1).tolist() == [int(c) for c in g["codes"]]
    assert Q["idx"][0, 0] == 0                      # |3| first attained at index 0, not at index 4


def test_quant_sym_error_half_step_and_zero_group():
    U = _heavy(16, 512, 3)
    U[3, 128:256] = 0.0
    for bits, group in ((4, 128), (3, 64), (4, 0)):
        Q = orc.quant_sym(U, bits, group)
        g = U.shape[1] if group == 0 else group
        s_e = np.repeat(Q["s"].astype(np.float64), g, axis=1)
        assert np.all(np.abs(Q["Uhat"] - U) <= 0.5 * s_e * (1 + 1e-5) + 1e-30)
        assert np.abs(Q["q"]).max() <= orc.qmax_of(bits)
        # every group's arg-max entry carries code +-qmax
        qg = Q["q"].reshape(U.shape[0], -1, g)
        top = np.take_along_axis(qg, Q["idx"][..., None], axis=2)[..., 0]
        nz = Q["a"] > 0
        assert np.all(np.abs(top[nz]) == orc.qmax_of(bits))
    Q = orc.quant_sym(U, 4, 128)
    assert Q["s"][3, 1] == 0 and np.all(Q["q"][3, 128:256] == 0) and np.all(Q["Uhat"][3, 128:256] == 0)


def test_offsets_reproduce_rtn():
    # RTN is the floor/ceil choice r = [frac > 1/2, or tie and floor odd]
    U = _w(8, 64, 5)
    Q = orc.quant_sym(U, 4, 32)
    s_e = np.repeat(Q["s"], 32, axis=1)
    x = (U.astype(np.float32) / s_e).astype(np.float32)
    r = (Q["q"] - np.floor(x)).astype(np.float64)
    assert set(np.unique(r)) <= {0.0, 1.0}
    Q2 = orc.quant_sym(U, 4, 32, offsets=r)
    assert np.array_equal(Q2["q"], Q["q"].astype(np.float64))


# ------------------------------------------------------------------ block operators (P2, P14, P16)
def test_block_inverse_matches_library_and_pivots():
    M = syn.perturbed_blocks(3, 16, 11, 0.3).astype(np.float64)
    M[1, 0, 0] = 0.0                                # forces a row exchange at the first pivot
    Minv = orc.block_inverse(M)
    assert np.allclose(Minv, np.linalg.inv(M), rtol=1e-10, atol=1e-10)


@pytest.mark.parametrize("axis", ["in", "out"])
def test_apply_blocks_equals_dense_block_diagonal(axis):
    nb, k = 3, 8
    T = syn.perturbed_blocks(nb, k, 2).astype(np.float64)
    dense = scipy.linalg.block_diag(*T)
    if axis == "in":
        W = _w(10, nb * k, 1)
        ref = W @ dense.T                            # row vector times T^T  <=>  T acts on d_in
        assert np.allclose(orc.apply_blocks(W, T, "in"), ref, atol=1e-12)
        gU = _w(10, nb * k, 9)
        full = gU.T @ W                              # d/dT of sum(gU * (W T^T)) = gU^T W
    else:
        W = _w(nb * k, 10, 1)
        ref = dense @ W
        assert np.allclose(orc.apply_blocks(W, T, "out"), ref, atol=1e-12)
        gU = _w(nb * k, 10, 9)
        full = gU @ W.T
    g = orc.operator_grad(gU, W, k, axis)
    for b in range(nb):
        assert np.allclose(g[b], full[b * k:(b + 1) * k, b * k:(b + 1) * k], atol=1e-12)


def test_pair_identity_preserves_product_to_1e10():
    h, d1, d3, k = 32, 24, 20, 8
    W1s, W2s = _w(h, d1, 1), _w(d3, h, 2)
    for M in (syn.haar_blocks(h // k, k, 3), syn.perturbed_blocks(h // k, k, 4, 0.3)):
        M = M.astype(np.float64)
        U = orc.apply_blocks(W1s, np.transpose(M, (0, 2, 1)), "out")
        V = orc.apply_blocks(W2s, orc.block_inverse(M), "in")
        P = W1s.T @ W2s.T                            # paper's W1 W2 with W1 = W1s^T, W2 = W2s^T
        assert np.linalg.norm(U.T @ V.T - P) / np.linalg.norm(P) <= 1e-10
        assert np.allclose(orc.pair_product(W1s, W2s, k, 1), P, atol=1e-12)
        # U really is W1 M in the paper's orientation
        assert np.allclose(U.T, W1s.T @ scipy.linalg.block_diag(*M), atol=1e-12)
        assert np.allclose(V.T, np.linalg.inv(scipy.linalg.block_diag(*M)) @ W2s.T, atol=1e-10)


def test_gqa_replicas_equal_physical_replication():
    k, nbk, r, d1, d3 = 8, 2, 2, 12, 10
    h = nbk * k
    W1s, W2s = _w(h, d1, 1), _w(d3, r * h, 2)
    M = syn.perturbed_blocks(nbk, k, 5, 0.2)
    f = orc.pair_forward(W1s, W2s, M, 4, 0, 8, r=r, lam=0.1)
    W1rep = orc.expand_rows(W1s, k, r)
    Mrep = np.repeat(M, r, axis=0)
    f1 = orc.pair_forward(W1rep, W2s, Mrep, 4, 0, 8, r=1, lam=0.0)
    assert f["pqe"] == pytest.approx(f1["pqe"], rel=1e-12)
    assert np.allclose(f["P"], f1["P"], atol=1e-12)
    # adjointness of expand/fold
    X, Y = _w(h, 5, 7), _w(r * h, 5, 8)
    assert np.sum(orc.expand_rows(X, k, r) * Y) == pytest.approx(np.sum(X * orc.fold_rows(Y, k, r)), rel=1e-12)


# ------------------------------------------------------------------ single matrix (P1, P3, P6, P9, P15)
@pytest.mark.parametrize("axis", ["in", "out"])
def test_identity_transform_is_plain_rtn(axis):
    W = _heavy(64, 256, 4)
    k = 32
    nb = (W.shape[1] if axis == "in" else W.shape[0]) // k
    f = orc.single_forward(W, syn.identity_blocks(nb, k), 4, 128, axis)
    Q = orc.quant_sym(W, 4, 128)
    assert np.array_equal(f["q"], Q["q"]) and np.array_equal(f["s"], Q["s"])
    assert f["L2"] == pytest.approx(np.sum((Q["Uhat"] - W) ** 2), rel=1e-12)
    # closed form of the surrogate at M = I:  kappa * g * sum a^2
    assert f["surrogate"] == pytest.approx(f["kappa"] * 128 * np.sum(Q["a"].astype(np.float64) ** 2), rel=1e-12)
    assert f["kappa"] == 1.0 / 15 ** 2


def test_weights_on_grid_have_zero_loss():
    rng = np.random.default_rng(1)
    bits, g = 4, 32
    qm = orc.qmax_of(bits)
    codes = rng.integers(-qm, qm + 1, size=(16, 128))
    codes[:, ::g] = qm                                # every group contains +qmax
    e = rng.integers(-6, 3, size=(16, 128 // g))
    W = codes * np.repeat(np.exp2(e), g, axis=1)      # qmax * 2^e is the absmax => scale 2^e exactly
    f = orc.single_forward(W, syn.identity_blocks(4, 32), bits, g, "in")
    assert f["L2"] == 0.0 and np.array_equal(f["q"], codes)


@pytest.mark.parametrize("axis", ["in", "out"])
def test_orthogonal_transform_gives_unit_column_norms(axis):
    W = _heavy(64, 64, 6)
    M = syn.haar_blocks(2, 32, 8).astype(np.float64)
    f = orc.single_forward(W, M, 4, 32, axis, prec="exact")
    assert np.allclose(f["c"], 1.0, rtol=0, atol=1e-6)          # rotation stored in fp32
    assert f["L2"] == pytest.approx(np.sum(f["Delta"] ** 2), rel=1e-6)
    # relative l2 equals the definition written out with a dense matrix
    D = scipy.linalg.block_diag(*M)
    if axis == "in":
        What = f["Uhat"] @ np.linalg.inv(D).T
    else:
        What = np.linalg.inv(D) @ f["Uhat"]
    assert f["rel_l2"] == pytest.approx(np.linalg.norm(What - W) / np.linalg.norm(W), rel=1e-9)


@pytest.mark.parametrize("axis", ["in", "out"])
def test_l2_equals_dense_definition_for_general_M(axis):
    W = _heavy(48, 48, 16)
    M = syn.perturbed_blocks(3, 16, 5, 0.4).astype(np.float64)
    f = orc.single_forward(W, M, 3, 16, axis, prec="exact")
    D = scipy.linalg.block_diag(*M)
    MW = W @ D.T if axis == "in" else D @ W
    Qd = orc.quant_sym(MW, 3, 16, None, np.float64)
    back = Qd["Uhat"] @ np.linalg.inv(D).T if axis == "in" else np.linalg.inv(D) @ Qd["Uhat"]
    assert f["L2"] == pytest.approx(np.linalg.norm(back - W) ** 2, rel=1e-9)


@pytest.mark.parametrize("axis", ["in", "out"])
def test_surrogate_bounds_stochastic_rounding_expectation(axis):
    """Eq. 4: E||Minv (SR(U) - U)||^2 = sum_e c_t(e) s^2 f(1-f) <= (1/4 qmax^2) sum_e c_t a^2."""
    W = _heavy(32, 32, 21)
    k, g, bits = 16, 16, 3
    M = syn.perturbed_blocks(2, k, 13, 0.5).astype(np.float64)
    M = M * np.linspace(0.4, 2.5, k)[None, None, :]              # far from orthogonal: row norms != column norms
    qm = orc.qmax_of(bits)
    f = orc.single_forward(W, M, bits, g, axis, kappa=1.0 / (4 * qm * qm), prec="exact")
    s_e = np.repeat(f["s"].astype(np.float64), g, axis=1)
    x = f["U"] / s_e
    fr = x - np.floor(x)
    # Monte-Carlo estimate of the expectation with real stochastic rounding
    rng = np.random.default_rng(5)
    acc, n = 0.0, 4000
    for _ in range(n):
        up = rng.random(x.shape) < fr
        Delta = s_e * (np.floor(x) + up) - f["U"]
        acc += np.sum(orc.apply_blocks(Delta, f["Minv"], axis) ** 2)
    mc = acc / n
    # closed form with c indexed by the transformed index of the entry
    c_flat = f["c"].reshape(-1)
    ce = np.broadcast_to(c_flat[None, :] if axis == "in" else c_flat[:, None], x.shape)
    closed = np.sum(ce * s_e ** 2 * fr * (1 - fr))
    assert mc == pytest.approx(closed, rel=0.03)
    assert closed <= f["surrogate"] * (1 + 1e-9)
    # a transposed c (row norms instead of column norms of Minv) would not match the expectation
    c_wrong = np.sum(f["Minv"] ** 2, axis=2).reshape(-1)
    cw = np.broadcast_to(c_wrong[None, :] if axis == "in" else c_wrong[:, None], x.shape)
    assert abs(np.sum(cw * s_e ** 2 * fr * (1 - fr)) - mc) > 0.05 * mc


def test_eq4_verbatim_for_per_channel_output_axis():
    """Axis OUT with one group per row is Eq. 4 as printed: d2/(2^N-1)^2 sum_ij Minv_ij^2 ||(MW)_j||_inf^2."""
    W = _heavy(16, 40, 2)
    M = syn.perturbed_blocks(1, 16, 3, 0.3).astype(np.float64)
    f = orc.single_forward(W, M, 4, 0, "out", prec="exact")
    MW = M[0] @ W
    Minv = np.linalg.inv(M[0])
    printed = W.shape[1] / (2 ** 4 - 1) ** 2 * sum(
        Minv[i, j] ** 2 * np.max(np.abs(MW[j])) ** 2
        for i in range(16) for j in range(16))
    assert f["surrogate"] == pytest.approx(printed, rel=1e-10)


def test_invariances_permutation_and_scaling():
    W = _heavy(32, 128, 9)
    bits, g, k = 4, 32, 64
    f0 = orc.single_forward(W, syn.identity_blocks(2, k), bits, g, "in")
    P = syn.signed_perm_blocks(2, k, 3, within=g)
    fp = orc.single_forward(W, P, bits, g, "in")
    assert fp["L2"] == pytest.approx(f0["L2"], rel=1e-12)
    assert np.array_equal(np.sort(np.abs(fp["q"]), axis=1), np.sort(np.abs(f0["q"]), axis=1))
    assert np.array_equal(fp["s"], f0["s"])
    f2 = orc.single_forward(W * 8.0, syn.identity_blocks(2, k), bits, g, "in")
    assert np.array_equal(f2["q"], f0["q"]) and np.array_equal(f2["s"], f0["s"] * 8)
    assert f2["L2"] == pytest.approx(64 * f0["L2"], rel=1e-12)
    assert f2["surrogate"] == pytest.approx(64 * f0["surrogate"], rel=1e-12)
    D = syn.pow2_diag_blocks(2, k, 4)
    fd = orc.single_forward(W, D, bits, g, "in")
    assert fd["Mc"].tolist() == D.astype(np.float64).tolist()   # +-2^e survives bf16 rounding


# ------------------------------------------------------------------ gradients against finite differences (P7)
def _fd(fun, M, eps=1e-6):
    g = np.zeros_like(M)
    it = np.nditer(M, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        Mp, Mm = M.copy(), M.copy()
        Mp[i] += eps
        Mm[i] -= eps
        g[i] = (fun(Mp) - fun(Mm)) / (2 * eps)
    return g


@pytest.mark.parametrize("axis,group", [("in", 4), ("in", 8), ("out", 4), ("out", 0)])
def test_surrogate_gradient_matches_finite_differences(axis, group):
    k = 4
    W = _w(8, 8, 31 + len(axis))
    M = syn.perturbed_blocks(2, k, 17, 0.4).astype(np.float64)
    f = orc.single_forward(W, M, 4, group, axis, prec="exact")
    g = orc.single_grad_surrogate(W, f, group, axis)
    fd = _fd(lambda X: orc.single_forward(W, X, 4, group, axis, prec="exact")["surrogate"], M)
    assert np.allclose(g, fd, rtol=2e-5, atol=1e-8)


@pytest.mark.parametrize("axis", ["in", "out"])
def test_ste_gradient_matches_fd_of_frozen_code_loss(axis):
    k, bits, group = 4, 3, 4
    W = _w(8, 8, 41)
    M = syn.perturbed_blocks(2, k, 19, 0.4).astype(np.float64)
    f = orc.single_forward(W, M, bits, group, axis, prec="exact")
    g = orc.single_grad_ste(W, f, bits, group, axis)
    q, idx, qm = f["q"].astype(np.float64), f["idx"], orc.qmax_of(bits)
    x0 = f["U"] / np.repeat(f["s"], group, axis=1)               # U/s at the evaluation point, held fixed

    def frozen(X):
        # straight-through: round(x) := q + (x - stop(x)), so Uhat - U = s(X) * (q - x0)
        U = orc.apply_blocks(W, X, axis)
        Ug = U.reshape(8, -1, group)
        a = np.abs(np.take_along_axis(Ug, idx[..., None], axis=2))[..., 0]
        Delta = np.repeat(a / qm, group, axis=1) * (q - x0)
        E = orc.apply_blocks(Delta, orc.block_inverse(X), axis)
        return np.sum(E * E)

    assert frozen(M) == pytest.approx(f["L2"], rel=1e-12)
    assert np.allclose(g, _fd(frozen, M), rtol=2e-5, atol=1e-8)


@pytest.mark.parametrize("r", [1, 2])
def test_lse_gradient_matches_finite_differences(r):
    k, nbk, d1, d3 = 4, 2, 6, 5
    h = nbk * k
    W1s, W2s = _w(h, d1, 51), _w(d3, r * h, 52)
    M = syn.perturbed_blocks(nbk, k, 23, 0.4).astype(np.float64)
    kw = dict(bits=4, group1=0, group2=4, r=r, t=5.0, lam=0.3, want_pqe=False, prec="exact")
    f = orc.pair_forward(W1s, W2s, M, **kw)
    g = orc.pair_grad_lse(W1s, W2s, f, 0, 4)
    fd = _fd(lambda X: orc.pair_forward(W1s, W2s, X, **kw)["loss"], M)
    assert np.allclose(g, fd, rtol=2e-5, atol=1e-8)


@pytest.mark.parametrize("r", [1, 2])
def test_pqe_ste_gradient_matches_fd_of_frozen_code_loss(r):
    k, nbk, d1, d3, bits = 4, 2, 6, 5, 3
    h = nbk * k
    g1, g2 = 0, 4
    W1s, W2s = _w(h, d1, 61), _w(d3, r * h, 62)
    M = syn.perturbed_blocks(nbk, k, 29, 0.4).astype(np.float64)
    f = orc.pair_forward(W1s, W2s, M, bits, g1, g2, r=r, prec="exact")
    g = orc.pair_grad_pqe_ste(W1s, W2s, f, bits, g1, g2)
    qm = orc.qmax_of(bits)
    P = f["P"]

    def soft(X, Q, U0, group):
        # straight-through value: s(X) * (q + X/s(X) - stop(U0/s0)) = X + s(X) * (q - x0)
        d_out, d_in = X.shape
        gg = d_in if group == 0 else group
        a = np.abs(np.take_along_axis(X.reshape(d_out, -1, gg), Q["idx"][..., None], axis=2))[..., 0]
        x0 = U0 / np.repeat(Q["s"], gg, axis=1)
        return X + np.repeat(a / qm, gg, axis=1) * (Q["q"] - x0)

    def frozen(Mx):
        U = orc.apply_blocks(W1s, np.transpose(Mx, (0, 2, 1)), "out")
        V = orc.apply_blocks(W2s, orc.block_inverse(Mx), "in", r)
        Uh = soft(U, f["QU"], f["U"], g1)
        Vh = soft(V, f["QV"], f["V"], g2)
        R = orc.pair_product(Uh, Vh, k, r) - P
        return np.sum(R * R)

    assert frozen(M) == pytest.approx(f["pqe"] ** 2, rel=1e-12)
    assert np.allclose(g, _fd(frozen, M), rtol=5e-5, atol=1e-8)


def test_orth_penalty_value_and_gradient():
    M = syn.perturbed_blocks(2, 4, 3, 0.5).astype(np.float64)
    val, g = orc.orth_penalty(M)
    D = scipy.linalg.block_diag(*M)
    assert val == pytest.approx(np.linalg.norm(D @ D.T - np.eye(8)) / np.sqrt(8), rel=1e-12)
    assert np.allclose(g, _fd(lambda X: orc.orth_penalty(X)[0], M), rtol=1e-5, atol=1e-9)
    assert orc.orth_penalty(syn.identity_blocks(2, 4))[0] == 0.0
    v, g0 = orc.orth_penalty(syn.haar_blocks(2, 4, 1))          # a rotation stored in fp32: value ~1e-8
    assert 0 < v < 1e-6


# ------------------------------------------------------------------ LogSumExp (P8)
def test_lse_bounds_weights_and_lipschitz():
    h, d1, d3, k = 16, 12, 10, 8
    W1s, W2s = _heavy(h, d1, 1), _heavy(d3, h, 2)
    M = syn.haar_blocks(2, k, 3)
    for t in (1.0, 5.0, 10.0):
        f = orc.pair_forward(W1s, W2s, M, 4, 0, 8, t=t, want_pqe=False)
        amax = max(f["QU"]["a"].max(), f["QV"]["a"].max())
        n = f["QU"]["a"].size + f["QV"]["a"].size
        assert amax <= f["lse"] <= amax + np.log(n) / t + 1e-12
        assert f["wu"].sum() + f["wv"].sum() == pytest.approx(1.0, rel=1e-12)
    # 1-Lipschitz in the sup norm of the maxima: perturbing W2s by delta moves LSE by <= max|dV|
    f0 = orc.pair_forward(W1s, W2s, M, 4, 0, 8, want_pqe=False, prec="exact")
    d = 1e-3 * np.random.default_rng(0).standard_normal(W2s.shape)
    f1 = orc.pair_forward(W1s, W2s + d, M, 4, 0, 8, want_pqe=False, prec="exact")
    assert abs(f1["lse"] - f0["lse"]) <= np.max(np.abs(f1["V"] - f0["V"])) * (1 + 1e-6) + 1e-7


# ------------------------------------------------------------------ optimisers
def test_adam_first_step_is_sign_step():
    M = np.array([[[1.0, -2.0], [0.5, 3.0]]])
    g = np.array([[[0.3, -4.0], [1e-3, 2.0]]])
    M1, st = orc.adam_step(M, g, (np.zeros_like(M), np.zeros_like(M), 0), lr=0.01, beta1=0.1, beta2=0.999, eps=1e-8)
    # after bias correction m_hat = g and v_hat = g^2, so the step is lr * g/(|g| + eps)
    assert np.allclose(M1, M - 0.01 * g / (np.abs(g) + 1e-8), rtol=1e-12)
    assert st[2] == 1
    M2, st = orc.adam_step(M1, g, st, lr=0.01)
    assert np.allclose(M2, M1 - 0.01 * np.sign(g), rtol=1e-6)   # constant gradient keeps the ratio at 1


def test_learned_transform_beats_rotation_beats_identity():
    """Qualitative ordering of Table 1 on synthetic heavy-tailed weights (values unpinned)."""
    W = syn.bf16_bits_to_f64(syn.weight_gauss_outliers(64, 128, 77))
    k, bits, g = 32, 4, 32
    ident = orc.single_forward(W, syn.identity_blocks(4, k), bits, g, "in")["rel_l2"]
    M0 = syn.haar_blocks(4, k, 5)
    rot = orc.single_forward(W, M0, bits, g, "in")
    M, hist = orc.optimize_single(W, M0, bits, g, "in", steps=60, lr=0.5 / rot["surrogate"] * 0.05)
    learned = orc.single_forward(W, M, bits, g, "in")["rel_l2"]
    assert hist[-1, 0] < hist[0, 0]
    assert learned < rot["rel_l2"] < ident


# ------------------------------------------------------------------ Algorithm 1 (P13) and brute force (P11)
def test_alg1_zero_iterations_and_on_grid_first_factor():
    h, d1, d3, k = 8, 6, 5, 8
    U1s, V2s = _w(h, d1, 3), _w(d3, h, 4)
    out = orc.adaptive_round_stored(U1s, V2s, 4, 0, 0, k, 1, iters=0)
    assert np.array_equal(out["q1"], orc.quant_sym(U1s, 4, 0)["q"])
    assert np.array_equal(out["q2"], orc.quant_sym(V2s, 4, 0)["q"])
    # first factor already on the grid => W2' = W2 (pinv(W1) W1 = I for full column rank), nothing to compensate
    W1 = np.rint(_w(6, 4, 5) * 3)
    W1[0, :] = 7
    W2 = _w(4, 5, 6)
    Q1 = lambda X: orc.quant_sym(X.T, 4, 0)["Uhat"].T          # per-column groups of the paper-orientation matrix
    assert np.array_equal(Q1(W1), W1)
    W2p = orc.pinv(Q1(W1)) @ W1 @ W2
    assert np.allclose(W2p, W2, atol=1e-12)


def test_stored_alg1_matches_paper_orientation_and_improves():
    h, d1, d3, k, bits = 16, 24, 20, 8, 3
    U1s, V2s = _heavy(h, d1, 7), _heavy(d3, h, 8)
    out = orc.adaptive_round_stored(U1s, V2s, bits, 0, 8, k, 1, iters=3)
    Q1 = lambda X: orc.quant_sym(X.T, bits, 0)["Uhat"].T
    Q2 = lambda X: orc.quant_sym(X.T, bits, 8)["Uhat"].T
    W1h, W2h, hist = orc.adaptive_round_alg1(U1s.T, V2s.T, Q1, Q2, iters=3)
    assert np.allclose(out["pqe"], hist, rtol=1e-9)
    assert np.allclose(out["Uhat1"].T, W1h, atol=1e-12)
    assert min(hist[1:]) < hist[0]                   # Table 2's direction: adaptive < independent
    out2 = orc.adaptive_round_stored(_heavy(8, d1, 9), _heavy(d3, 16, 10), bits, 0, 8, 8, 2, iters=2)
    assert min(out2["pqe"][1:]) < out2["pqe"][0]


def test_pinv_matches_library():
    A = _w(9, 5, 12)
    A[:, 4] = A[:, 0] + A[:, 1]                      # rank deficient
    assert np.allclose(orc.pinv(A), np.linalg.pinv(A), atol=1e-9)


def test_brute_force_rtn_is_optimal_for_identity():
    W = _w(2, 8, 71)
    best, off, allv = orc.brute_force_single(W, syn.identity_blocks(2, 4), 3, 4, "in")
    rtn = orc.single_forward(W, syn.identity_blocks(2, 4), 3, 4, "in")
    assert best == pytest.approx(rtn["L2"], rel=1e-12)
    assert len(allv) == 2 ** 16
    # with a non-orthogonal transform RTN need not be optimal but can never beat the enumeration
    M = syn.perturbed_blocks(1, 4, 7, 0.8)
    W = _w(3, 4, 72)
    best, off, allv = orc.brute_force_single(W, M, 3, 4, "in")
    rtn = orc.single_forward(W, M, 3, 4, "in")
    assert best <= rtn["L2"] * (1 + 1e-12)
    assert any(abs(v - rtn["L2"]) <= 1e-12 * max(1.0, rtn["L2"]) for v in allv)


# ------------------------------------------------------------------ packing (P12)
def test_pack_hand_values_and_round_trip():
    g = _read_golden("pack_hand.txt")
    q4 = np.array(g["bits4_codes"], dtype=np.int64).reshape(1, -1)
    assert orc.pack_codes(q4, 4).reshape(-1).tolist() == [int(b) for b in g["bits4_bytes"]]
    q3 = np.array(g["bits3_codes"], dtype=np.int64).reshape(1, -1)
    assert orc.pack_codes(q3, 3).reshape(-1).tolist() == [int(b) for b in g["bits3_bytes"]]
    rng = np.random.default_rng(0)
    for bits in (2, 3, 4, 8):
        qm = orc.qmax_of(bits)
        q = rng.integers(-qm, qm + 1, size=(5, 64))
        p = orc.pack_codes(q, bits)
        assert p.shape == (5, 64 * bits // 8)
        assert np.array_equal(orc.unpack_codes(p, bits, 64), q)
        # the stream read as one little-endian integer is sum u_i 2^(bits*i)
        for row in range(5):
            big = sum(int(q[row, i] + qm) << (bits * i) for i in range(64))
            assert int.from_bytes(bytes(p[row].tolist()), "little") == big


def test_pinv_moore_penrose_identities_rank_deficient():
    """The four Moore-Penrose conditions fix the pseudo-inverse uniquely; checked on a matrix of rank 3 < min(6, 5)
    (where dropping the small singular values matters) and on a quantised factor with a zero row."""
    rng = np.random.default_rng(12)
    A = rng.standard_normal((6, 3)) @ rng.standard_normal((3, 5))
    B = np.round(rng.standard_normal((5, 4)) * 2.0)
    B[2] = 0.0
    for X in (A, B, A.T):
        Xp = orc.pinv(X)
        assert np.allclose(X @ Xp @ X, X, atol=1e-9)
        assert np.allclose(Xp @ X @ Xp, Xp, atol=1e-9)
        assert np.allclose((X @ Xp).T, X @ Xp, atol=1e-9)
        assert np.allclose((Xp @ X).T, Xp @ X, atol=1e-9)


def test_orth_penalty_zero_only_at_exact_orthonormality():
    """||M M^T - I||_F / sqrt(d): zero value and zero sub-gradient at a signed permutation (exactly orthonormal in
    floating point), the analytic gradient everywhere else - also a hair away from a rotation."""
    P = syn.signed_perm_blocks(2, 8, 3).astype(np.float64)
    v, g = orc.orth_penalty(P)
    assert v == 0.0 and not g.any()
    M = P + 1e-7 * np.random.default_rng(0).standard_normal(P.shape)
    v, g = orc.orth_penalty(M)
    assert v > 0 and np.linalg.norm(g) > 0.1            # a unit-scale direction, however small the distance
    eps = 1e-10
    d = np.random.default_rng(1).standard_normal(M.shape)
    fd = (orc.orth_penalty(M + eps * d)[0] - orc.orth_penalty(M - eps * d)[0]) / (2 * eps)
    assert abs(fd - np.sum(g * d)) <= 1e-4 * abs(fd)


def test_pqe_with_offsets_and_brute_force_pair():
    """Offsets equal to round-to-nearest reproduce the pair forward's product error; no offset vector beats the
    enumerated minimum; and the enumeration's entry for the round-to-nearest vector is that same error."""
    rng = np.random.default_rng(5)
    k, r = 2, 1
    U = rng.standard_normal((2, 3)) * 0.7            # stored [h, d1]
    V = rng.standard_normal((3, 2)) * 0.7            # stored [d3, r h]
    bits = 3
    o1, o2 = orc.rtn_offsets(U, bits, 0), orc.rtn_offsets(V, bits, 0)
    rtn = orc.pqe_with_offsets(U, V, bits, 0, 0, k, r, o1, o2)
    Q1, Q2 = orc.quant_sym(U, bits, 0), orc.quant_sym(V, bits, 0)
    direct = np.linalg.norm(orc.pair_product(Q1["Uhat"], Q2["Uhat"], k, r) - orc.pair_product(U, V, k, r))
    assert abs(rtn - direct) <= 1e-12
    best, b1, b2, allv = orc.brute_force_pair(U, V, bits, 0, 0, k, r)
    assert allv.size == 2 ** 12 and best == allv.min() and best <= rtn
    idx = int("".join(str(int(b)) for b in np.concatenate([o1.ravel(), o2.ravel()])), 2)
    assert abs(allv[idx] - rtn) <= 1e-12
    assert abs(orc.pqe_with_offsets(U, V, bits, 0, 0, k, r, b1, b2) - best) <= 1e-12


def test_optimize_pair_composes_the_pinned_pieces():
    """optimize_pair = pair_forward + pair_grad_lse + adam_step in a loop: the recorded losses are the forward's at
    the iterates, the first step is Adam's closed form lr * sign(g) (up to eps), and with lr = 0 nothing moves."""
    k, r, h, d1, d3 = 4, 2, 8, 6, 5
    W1, W2 = np.random.default_rng(1).standard_normal((h, d1)), np.random.default_rng(2).standard_normal((d3, r * h))
    M0 = syn.perturbed_blocks(h // k, k, 3, 0.1)
    M2, hist = orc.optimize_pair(W1, W2, M0, 4, 0, 4, r, 2, 1e-3, 5.0, 0.1)
    f0 = orc.pair_forward(W1, W2, M0, 4, 0, 4, r, 5.0, 0.1, False)
    assert abs(hist[0, 0] - f0["loss"]) <= 1e-12
    g0 = orc.pair_grad_lse(W1, W2, f0, 0, 4)
    M1, _ = orc.optimize_pair(W1, W2, M0, 4, 0, 4, r, 1, 1e-3, 5.0, 0.1)
    big = np.abs(g0) > 1e-6
    assert np.allclose((M1 - M0.astype(np.float32).astype(np.float64))[big], -1e-3 * np.sign(g0[big]), atol=2e-7)
    f1 = orc.pair_forward(W1, W2, M1, 4, 0, 4, r, 5.0, 0.1, False)
    assert abs(hist[1, 0] - f1["loss"]) <= 1e-12
    Mz, hz = orc.optimize_pair(W1, W2, M0, 4, 0, 4, r, 3, 0.0, 5.0, 0.1)
    assert np.array_equal(Mz, M0.astype(np.float32).astype(np.float64)) and np.ptp(hz[:, 0]) == 0.0


def test_single_grad_offsets_finite_differences():
    """dL2/drho against central differences of the forward evaluated with perturbed soft offsets (the loss is an
    exact quadratic in rho as long as no code is clamped), and the projection / hardening conventions."""
    rng = np.random.default_rng(3)
    W = rng.standard_normal((6, 8)) * 0.3
    M = syn.perturbed_blocks(2, 4, 2, 0.2)
    for axis, shape_nb in (("in", 2),):
        rho = rng.uniform(0.2, 0.8, size=W.shape)
        f = orc.single_forward(W, M, 4, 4, axis, offsets=rho)
        g = orc.single_grad_offsets(f, 4, axis)
        fd = np.zeros_like(g)
        eps = 1e-4
        for i in range(W.shape[0]):
            for j in range(W.shape[1]):
                d = np.zeros_like(rho)
                d[i, j] = eps
                fd[i, j] = (orc.single_forward(W, M, 4, 4, axis, offsets=rho + d)["L2"] -
                            orc.single_forward(W, M, 4, 4, axis, offsets=rho - d)["L2"]) / (2 * eps)
        assert np.allclose(g, fd, rtol=1e-4, atol=1e-7)     # fp32 scales inside the forward limit the agreement
    assert np.array_equal(orc.project_offsets([-0.2, 0.3, 1.7]), [0.0, 0.3, 1.0])
    assert np.array_equal(orc.harden_offsets([0.49, 0.5, 0.51]), [0.0, 1.0, 1.0])
    # soft offsets equal to the fractional part reproduce U exactly: zero loss
    f0 = orc.single_forward(W, M, 4, 4, "in")
    s_e = np.repeat(f0["s"].astype(np.float64), 4, axis=1)
    x = f0["U"] / s_e
    fz = orc.single_forward(W, M, 4, 4, "in", offsets=x - np.floor(x))
    assert fz["L2"] <= 1e-10 * f0["L2"]


def test_adaptive_round_learned_pins():
    """The learned-offset iteration: starts at zero error (offsets = fractional parts reproduce U, V), ends on the
    grid (hardened offsets are floor/ceil choices: its result is one of the enumerated vectors, so never below the
    enumerated minimum), its reported errors are Eq. 5 of what it returns, and on a pair where independent rounding
    leaves room it lowers the error."""
    rng = np.random.default_rng(0)
    U, V = rng.standard_normal((2, 3)) * 0.7, rng.standard_normal((3, 2)) * 0.7
    o = orc.adaptive_round_learned(U, V, 3, 0, 0, 2, 1, 12)
    best, _, _, allv = orc.brute_force_pair(U, V, 3, 0, 0, 2, 1)
    P = orc.pair_product(U, V, 2, 1)
    assert o["history"][1] <= 1e-6 * o["history"][0]
    assert abs(o["history"][-1] - np.linalg.norm(orc.pair_product(o["Uhat"], o["Vhat"], 2, 1) - P)) <= 1e-12
    assert best <= o["history"][-1] * (1 + 1e-12)
    assert np.min(np.abs(allv - o["history"][-1])) <= 1e-9        # the result is one of the enumerated choices
    Q1, Q2 = orc.quant_sym(U, 3, 0), orc.quant_sym(V, 3, 0)
    assert abs(o["history"][0] - np.linalg.norm(orc.pair_product(Q1["Uhat"], Q2["Uhat"], 2, 1) - P)) <= 1e-12
    assert np.all(np.abs(o["q1"] - Q1["q"]) <= 1) and np.all(np.abs(o["q2"] - Q2["q"]) <= 1)   # floor or ceil of the same quotient
    U, V = rng.standard_normal((32, 48)) * 0.1, rng.standard_normal((40, 64)) * 0.1
    o = orc.adaptive_round_learned(U, V, 3, 16, 16, 16, 2, 10)
    assert o["history"][-1] < 0.9 * o["history"][0]


@pytest.mark.parametrize("objective", ["sumsq", "sumsq_weighted"])
def test_pair_sum_of_squares_objectives(objective):
    """Appendix D.1's alternatives to LogSumExp: the value from its definition written out with plain loops over the
    group maxima, and the gradient against central finite differences (no rounding of the operators, jittered inputs:
    no arg-max ties)."""
    rng = np.random.default_rng(11)
    k, r, h, d1, d3 = 4, 2, 8, 6, 5
    W1, W2 = rng.standard_normal((h, d1)), rng.standard_normal((d3, r * h))
    M = syn.perturbed_blocks(h // k, k, 5, 0.2).astype(np.float64)

    def value(Mx):
        return orc.pair_forward(W1, W2, Mx, 4, 3, 4, r, 5.0, 0.0, False, prec="exact", objective=objective)

    f = value(M)
    U, V = f["U"], f["V"]
    mu = [max(abs(U[i, 3 * G:3 * G + 3])) for i in range(h) for G in range(d1 // 3)]
    mv = [max(abs(V[j, 4 * G:4 * G + 4])) for j in range(d3) for G in range(r * h // 4)]
    su, sv = sum(x * x for x in mu) / len(mu), sum(x * x for x in mv) / len(mv)
    want = su + sv if objective == "sumsq" else np.linalg.norm(V) * su + np.linalg.norm(U) * sv
    assert f["surrogate"] == pytest.approx(want, rel=1e-12)
    g = orc.pair_grad_lse(W1, W2, f, 3, 4)
    fd = _fd(lambda Mx: value(Mx)["surrogate"], M)
    assert np.allclose(g, fd, rtol=2e-5, atol=1e-8)


def test_cayley_step_pins():
    """The Cayley update keeps rotations rotations, moves along minus the skew part of the gradient to first order,
    and carries momentum."""
    rng = np.random.default_rng(2)
    M = np.stack([np.linalg.qr(rng.standard_normal((6, 6)))[0] for _ in range(2)])   # rotations to float64 accuracy
    g = rng.standard_normal(M.shape)
    M1, V = orc.cayley_step(M, g, np.zeros_like(M), 1e-2, 0.1)
    I = np.eye(6)
    assert np.allclose(M1 @ np.transpose(M1, (0, 2, 1)), I, atol=1e-12)
    assert np.array_equal(V, g)
    A = g @ np.transpose(M, (0, 2, 1)) - M @ np.transpose(g, (0, 2, 1))
    M_small, _ = orc.cayley_step(M, g, np.zeros_like(M), 1e-6, 0.1)
    assert np.allclose((M_small - M) / 1e-6, -A @ M, atol=1e-4)
    _, V2 = orc.cayley_step(M1, g, V, 1e-2, 0.1)
    assert np.allclose(V2, 1.1 * g)
    # descent: a linear loss <C, M> decreases along the step
    C = rng.standard_normal(M.shape)
    M2, _ = orc.cayley_step(M, C, np.zeros_like(M), 1e-2, 0.0)
    assert np.sum(C * M2) < np.sum(C * M)


# ---------------------------------------------------------------------------
# inference side (Section 4.1): function preservation, special operators, dequantisation against its definition
# ---------------------------------------------------------------------------
def test_inference_apply_preserves_the_product_and_special_cases():
    rng = np.random.default_rng(11)
    k, nb = 4, 3
    W, X = rng.standard_normal((5, nb * k)), rng.standard_normal((7, nb * k))
    M = orc.round_bf16(rng.standard_normal((nb, k, k)).astype(np.float32)).astype(np.float64)
    # y = W x = (W o M)(M^-T x): the activations go through the inverse's blocks applied transposed
    Minv = orc.round_bf16(np.linalg.inv(M).astype(np.float32)).astype(np.float64)     # deployed in bf16
    U = orc.apply_blocks(W, M, "in", 1)
    Xp = orc.inference_apply(X, Minv, "in", transpose=True)
    exact = W @ X.T
    assert np.abs(U @ Xp.T - exact).max() <= 2.0 ** -7 * np.abs(exact).max() * k      # only the bf16 rounding of M^-1
    # with an operator that bf16 holds exactly (a signed permutation) the identity is exact
    P = np.zeros((nb, k, k))
    for b in range(nb):
        perm = rng.permutation(k)
        P[b, np.arange(k), perm] = rng.choice([-1.0, 1.0], k)
    Up = orc.apply_blocks(W, P, "in", 1)
    Xq = orc.inference_apply(X, np.linalg.inv(P), "in", transpose=True)
    assert np.array_equal(Up @ Xq.T, W @ X.T) or np.abs(Up @ Xq.T - W @ X.T).max() < 1e-13
    # the identity operator returns the input; transpose=True with a symmetric operator changes nothing
    eye = np.broadcast_to(np.eye(k), (nb, k, k))
    assert np.array_equal(orc.inference_apply(X, eye), X)
    S = M + np.transpose(M, (0, 2, 1))
    assert np.array_equal(orc.inference_apply(X, S, "in", True), orc.inference_apply(X, S, "in", False))
    # one entry by hand: Y[o, B k + i] = sum_j P[B][i][j] X[o, B k + j]
    Y = orc.inference_apply(X, M)
    o, B, i = 3, 1, 2
    assert abs(Y[o, B * k + i] - sum(M[B, i, j] * X[o, B * k + j] for j in range(k))) < 1e-14


def test_dequant_inverts_pack_and_matches_the_quantiser_output():
    rng = np.random.default_rng(12)
    U = rng.standard_normal((6, 32)) * np.array([1, 10, 0.1, 1, 3, 1])[:, None]
    for bits in (3, 4):
        out = orc.quant_sym(U, bits, 16)
        q, s, Uhat = out["q"], out["s"], out["Uhat"]
        packed = orc.pack_codes(q, bits)
        What = orc.dequant(packed, s, bits, 16, 32)
        assert np.allclose(What, np.asarray(Uhat, dtype=np.float64), rtol=1e-6, atol=0)   # the quantiser's own s * q
        # one entry by hand from the bit stream: code i of a row sits at bits [bits * i, bits * i + bits)
        r, i = 2, 5
        pos = bits * i
        word = int(packed[r, pos // 8]) | (int(packed[r, pos // 8 + 1]) << 8)
        u = (word >> (pos % 8)) & ((1 << bits) - 1)
        assert abs(What[r, i] - float(s[r, i // 16]) * (u - (2 ** (bits - 1) - 1))) < 1e-12
