"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Tolerances: integer codes and fp32 scales bit-exact when the transform product is exact in fp32
(no transform, signed permutations, +-2^e diagonals); tie-aware otherwise; losses, gradients and
updated parameters within 1e-3 relative (fp32 accumulation on the device, float64 in the oracle)."""
import numpy as np
import pytest

import cafeq_synth as syn
from oracle import cafeq_oracle as orc
from parity_utils import assert_codes_tie_aware, device_inverse, f32_dev, rel_err, tie_free_weight, to_dev, w64

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-3


@pytest.fixture(scope="module")
def cq():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2511_19705_b200 as m
    m.lib()
    return m


def _axis(name, cq):
    return cq.AXIS_IN if name == "in" else cq.AXIS_OUT


# ------------------------------------------------------------------ cafeq_rtn
@pytest.mark.parametrize("shape,bits,group", [((256, 512), 4, 128), ((37, 384), 3, 64), ((130, 256), 4, 0),
                                               ((64, 96), 8, 32), ((5, 128), 2, 128)])
def test_rtn_plain_bit_exact(cq, shape, bits, group):
    Wb = syn.weight_gauss_outliers(*shape, seed=11)
    Wb[1, :min(128, shape[1])] = 0                         # an all-zero group
    codes, scales = cq.cafeq_rtn(to_dev(Wb), None, bits=bits, group=group)
    Q = orc.quant_sym(w64(Wb), bits, group)
    assert np.array_equal(codes.cpu().numpy().astype(np.int32), Q["q"])
    assert np.array_equal(scales.cpu().numpy(), Q["s"])


def test_rtn_strided_rows(cq):
    Wb = syn.weight_student_t(64, 256, 5)
    big = torch.zeros((64, 320), dtype=torch.bfloat16, device="cuda")
    big[:, :256] = to_dev(Wb)
    codes, scales = cq.cafeq_rtn(big[:, :256], None, bits=4, group=128)
    Q = orc.quant_sym(w64(Wb), 4, 128)
    assert np.array_equal(codes.cpu().numpy().astype(np.int32), Q["q"])


@pytest.mark.parametrize("axis", ["in", "out"])
@pytest.mark.parametrize("kind", ["identity", "perm", "pow2"])
@pytest.mark.parametrize("k", [32, 128])
def test_rtn_exact_transforms_bit_exact(cq, axis, kind, k):
    d_out, d_in = (192, 384) if axis == "in" else (384, 192)
    Wb = syn.weight_student_t(d_out, d_in, 21, 2, 10.0)
    nb = (d_in if axis == "in" else d_out) // k
    T = {"identity": syn.identity_blocks(nb, k), "perm": syn.signed_perm_blocks(nb, k, 3),
         "pow2": syn.pow2_diag_blocks(nb, k, 4)}[kind]
    codes, scales = cq.cafeq_rtn(to_dev(Wb), f32_dev(T), bits=4, group=64, tblock=k, taxis=_axis(axis, cq))
    U = orc.apply_blocks(w64(Wb), T.astype(np.float64), axis)
    Q = orc.quant_sym(U, 4, 64)
    assert np.array_equal(codes.cpu().numpy().astype(np.int32), Q["q"])
    assert np.array_equal(scales.cpu().numpy(), Q["s"])


@pytest.mark.parametrize("axis,k,r,transposed", [("in", 64, 1, False), ("out", 64, 1, True), ("in", 32, 2, False),
                                                  ("in", 128, 1, True), ("out", 256, 1, False), ("in", 256, 1, False)])
def test_rtn_general_transform_tie_aware(cq, axis, k, r, transposed):
    d_out, d_in = (200, 512) if axis == "in" else (512, 200)
    Wb = syn.weight_student_t(d_out, d_in, 31, 2, 10.0)
    nbq = (d_in if axis == "in" else d_out) // k
    T = syn.perturbed_blocks(nbq // r, k, 9, 0.2)
    group = 0 if axis == "out" else 128
    codes, scales = cq.cafeq_rtn(to_dev(Wb), f32_dev(T), bits=3, group=group, tblock=k, taxis=_axis(axis, cq),
                                 trole=cq.APPLY_TT if transposed else cq.APPLY_T, replicas=r)
    Tc = orc.round_bf16(T)
    if transposed:
        Tc = np.transpose(Tc, (0, 2, 1))
    U = orc.apply_blocks(w64(Wb), Tc, axis, r)
    Q = orc.quant_sym(U, 3, group)
    assert_codes_tie_aware(codes.cpu().numpy(), scales.cpu().numpy(), Q, U, group)


# ------------------------------------------------------------------ cafeq_proxy_loss_fwd_bwd
CASES_SINGLE = [("in", 32, 4, 32, (96, 128)), ("out", 32, 4, 64, (128, 192)), ("in", 128, 4, 128, (256, 512)),
                ("in", 256, 3, 128, (200, 512)), ("out", 256, 3, 128, (512, 384)), ("in", 64, 3, 0, (70, 128)),
                ("in", 128, 4, 64, (130, 256))]


@pytest.mark.parametrize("axis,k,bits,group,shape", CASES_SINGLE)
def test_single_surrogate_fwd_bwd(cq, axis, k, bits, group, shape):
    Wb = syn.weight_student_t(*shape, seed=41, n_outlier_channels=2, mult=10.0)
    nb = (shape[1] if axis == "in" else shape[0]) // k
    M = syn.perturbed_blocks(nb, k, 13, 0.1)
    out = cq.cafeq_proxy_loss_fwd_bwd(to_dev(Wb), f32_dev(M), bits=bits, group=group, taxis=_axis(axis, cq),
                                      flags=cq.FLAG_EXACT_LOSS, want_minv=True)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    W = w64(Wb)
    f = orc.single_forward(W, M, bits, group, axis)
    g = orc.single_grad_surrogate(W, f, group, axis)
    L = out["losses"].cpu().numpy()
    assert abs(L[0] - f["surrogate"]) <= TOL * f["surrogate"]
    assert abs(L[1] - f["L2"]) <= TOL * f["L2"]
    assert abs(L[2] - f["normW2"]) <= 1e-5 * f["normW2"]
    assert rel_err(out["Minv"].cpu().numpy(), f["Minv"]) <= 1e-4
    gg = out["gradM"].cpu().numpy()
    for b in range(nb):
        assert rel_err(gg[b], g[b]) <= TOL, f"block {b}"


@pytest.mark.parametrize("axis,k,bits,group,shape", CASES_SINGLE[:5])
def test_single_ste_fwd_bwd(cq, axis, k, bits, group, shape):
    nb = (shape[1] if axis == "in" else shape[0]) // k
    M = syn.perturbed_blocks(nb, k, 15, 0.1)
    # inputs without rounding ties: the straight-through gradient is compared at codes both sides agree on
    Wb = tie_free_weight(lambda i: syn.weight_student_t(*shape, seed=43 + 1000 * i, n_outlier_channels=2, mult=10.0),
                         lambda W: orc.apply_blocks(W, orc.round_bf16(M), axis), bits, group,
                         "rows" if axis == "in" else "cols")
    out = cq.cafeq_proxy_loss_fwd_bwd(to_dev(Wb), f32_dev(M), bits=bits, group=group, taxis=_axis(axis, cq),
                                      loss_kind=cq.LOSS_L2_STE)
    W = w64(Wb)
    f = orc.single_forward(W, M, bits, group, axis)
    g = orc.single_grad_ste(W, f, bits, group, axis)
    L = out["losses"].cpu().numpy()
    assert abs(L[1] - f["L2"]) <= TOL * f["L2"]
    gg = out["gradM"].cpu().numpy()
    assert rel_err(gg, g) <= TOL
    for b in range(nb):
        assert rel_err(gg[b], g[b]) <= TOL, f"block {b}"


def test_offsets_exhaustive_tiny(cq):
    """Every one of the 2^n floor/ceil choices on a tiny matrix gives the oracle's loss (n = 10)."""
    Wb = syn.weight_small(2, 8, 3)
    n_free = 10
    W = w64(Wb)
    M = syn.perturbed_blocks(2, 4, 5, 0.5)
    Wd, Md = to_dev(Wb), f32_dev(M)
    rng = np.random.default_rng(0)
    base = (rng.random(W.shape) < 0.5).astype(np.float64)
    worst = 0.0
    for code in range(2 ** n_free):
        off = base.copy().reshape(-1)
        for b in range(n_free):
            off[b] = (code >> b) & 1
        off = off.reshape(W.shape)
        out = cq.cafeq_proxy_loss_fwd_bwd(Wd, Md, bits=3, group=4, flags=cq.FLAG_EXACT_LOSS | cq.FLAG_NO_GRAD,
                                          offsets=torch.from_numpy(off.astype(np.uint8)).cuda())
        ref = orc.single_forward(W, M, 3, 4, "in", offsets=off)["L2"]
        got = float(out["losses"][1].item())
        worst = max(worst, abs(got - ref) / ref)
    assert worst <= TOL


def test_soft_offsets(cq):
    Wb = syn.weight_small(16, 64, 9)
    M = syn.perturbed_blocks(2, 32, 5, 0.2)
    rho = np.random.default_rng(1).random((16, 64)).astype(np.float32)
    out = cq.cafeq_proxy_loss_fwd_bwd(to_dev(Wb), f32_dev(M), bits=4, group=32, flags=cq.FLAG_EXACT_LOSS | cq.FLAG_NO_GRAD,
                                      offsets=torch.from_numpy(rho).cuda())
    ref = orc.single_forward(w64(Wb), M, 4, 32, "in", offsets=rho.astype(np.float64))["L2"]
    assert abs(float(out["losses"][1].item()) - ref) <= TOL * ref


def test_status_singular_and_nonfinite(cq):
    Wb = syn.weight_small(32, 64, 1)
    M = syn.identity_blocks(2, 32)
    M[1, 5, :] = 0.0                                    # a zero row: no usable pivot
    out = cq.cafeq_proxy_loss_fwd_bwd(to_dev(Wb), f32_dev(M), bits=4, group=32)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 5
    Wn = to_dev(Wb).clone()
    Wn[3, 7] = float("nan")
    out = cq.cafeq_proxy_loss_fwd_bwd(Wn, f32_dev(syn.identity_blocks(2, 32)), bits=4, group=32)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 6


# ------------------------------------------------------------------ cafeq_optimize_single
def test_optimize_single_teacher_forced_and_free_running(cq):
    spec = syn.layer_spec(1)
    name, d_out, d_in = spec["singles"][0]
    k, bits, group = spec["k"], spec["bits"], spec["group"]
    Wb = syn.make_weight(1, name, d_out, d_in)
    W = w64(Wb)
    M0 = syn.make_transform(name, d_in // k, k)
    f0 = orc.single_forward(W, M0, bits, group, "in")
    lr = 0.02 / np.abs(orc.single_grad_surrogate(W, f0, group, "in")).max()
    # teacher-forced: one step from the oracle's M_t for t = 0, 3
    Mo = M0.astype(np.float64)
    for t in range(4):
        f = orc.single_forward(W, Mo, bits, group, "in")
        Mn = orc.gd_step(Mo, orc.single_grad_surrogate(W, f, group, "in"), lr)
        if t in (0, 3):
            Md = f32_dev(Mo.astype(np.float32))
            cfg = cq.make_cfg(loss_kind=cq.LOSS_SURROGATE, optimizer=cq.OPT_GD, lr=lr, steps=1, eval_every=1)
            hist, status, _ = cq.cafeq_optimize_single(to_dev(Wb), Md, cfg, bits=bits, group=group)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert rel_err(Md.cpu().numpy() - Mo, Mn - Mo) <= TOL          # the update itself
            h = hist.cpu().numpy()[0]
            assert abs(h[0] - f["surrogate"]) <= TOL * f["surrogate"] and abs(h[1] - f["L2"]) <= TOL * f["L2"]
        Mo = Mn.astype(np.float32).astype(np.float64)
    # free running: all 50 steps of the configuration; loss must fall and end near the oracle's trajectory
    steps = spec["steps"]
    Md = f32_dev(M0)
    cfg = cq.make_cfg(loss_kind=cq.LOSS_SURROGATE, optimizer=cq.OPT_GD, lr=lr, steps=steps, eval_every=10)
    hist, status, _ = cq.cafeq_optimize_single(to_dev(Wb), Md, cfg, bits=bits, group=group)
    h = hist.cpu().numpy()
    Mo, ho = orc.optimize_single(W, M0, bits, group, "in", steps, lr)
    assert int(status.item()) == 0
    assert h[-1, 0] < h[0, 0]
    assert np.isnan(h[1, 1]) and not np.isnan(h[10, 1])
    assert abs(h[-1, 0] - ho[-1, 0]) <= 0.02 * ho[-1, 0]      # arg-max switches make long runs sensitive


def test_optimize_single_adam_resume(cq):
    Wb = syn.weight_student_t(64, 128, 3)
    M0 = syn.haar_blocks(4, 32, 2)
    cfg2 = cq.make_cfg(optimizer=cq.OPT_ADAM, lr=1e-3, steps=2)
    cfg1 = cq.make_cfg(optimizer=cq.OPT_ADAM, lr=1e-3, steps=1)
    Ma = f32_dev(M0)
    cq.cafeq_optimize_single(to_dev(Wb), Ma, cfg2, bits=4, group=32)
    Mb = f32_dev(M0)
    _, _, st = cq.cafeq_optimize_single(to_dev(Wb), Mb, cfg1, bits=4, group=32)
    cq.cafeq_optimize_single(to_dev(Wb), Mb, cfg1, bits=4, group=32, opt_state=st)
    # a chunked run carries its optimiser state over; sums use floating-point atomics, so the two runs agree
    # to rounding, not bit for bit
    assert rel_err(Mb.cpu().numpy() - M0, Ma.cpu().numpy() - M0) <= 1e-4
    # first Adam step against the oracle
    W = w64(Wb)
    f = orc.single_forward(W, M0, 4, 32, "in")
    g = orc.single_grad_surrogate(W, f, 32, "in")
    M1, _ = orc.adam_step(M0.astype(np.float64), g, (np.zeros_like(g), np.zeros_like(g), 0), 1e-3)
    Mc = f32_dev(M0)
    cq.cafeq_optimize_single(to_dev(Wb), Mc, cfg1, bits=4, group=32)
    assert rel_err(Mc.cpu().numpy() - M0, M1 - M0) <= TOL


# ------------------------------------------------------------------ pair
PAIR_CASES = [(32, 1, 0, 32, (64, 96, 80)), (64, 2, 128, 64, (128, 256, 192)), (256, 1, 128, 128, (256, 384, 320)),
              (128, 2, 128, 128, (256, 256, 130))]


@pytest.mark.parametrize("k,r,g1,g2,dims", PAIR_CASES)
def test_pair_lse_pqe_fwd_bwd(cq, k, r, g1, g2, dims):
    h, d1, d3 = dims
    M = syn.perturbed_blocks(h // k, k, 17, 0.1)
    bits, lam, t = 4, 0.1, 5.0
    # the second factor's operator is bf16 of the inverse as the device computes it (single entries of an inverse
    # round to bf16 differently in fp32 and float64); weights without rounding ties under both operators
    Minv_c = orc.round_bf16(device_inverse(cq, M))
    McT = np.transpose(orc.round_bf16(M), (0, 2, 1))
    W1b = tie_free_weight(lambda i: syn.weight_student_t(h, d1, 51 + 1000 * i, 2, 10.0),
                          lambda W: orc.apply_blocks(W, McT, "out", 1), bits, g1, "cols")
    W2b = tie_free_weight(lambda i: syn.weight_student_t(d3, r * h, 52 + 1000 * i, 2, 10.0),
                          lambda W: orc.apply_blocks(W, Minv_c, "in", r), bits, g2, "rows")
    W1d, W2d, Md = to_dev(W1b), to_dev(W2b), f32_dev(M)
    P = cq.cafeq_pair_product(W1d, W2d, k=k, replicas=r)
    W1, W2 = w64(W1b), w64(W2b)
    f = orc.pair_forward(W1, W2, M, bits, g1, g2, r, t, lam, True, Minv_c=Minv_c)
    assert rel_err(P.cpu().numpy(), f["P"]) <= 1e-5
    out = cq.cafeq_pair_loss_fwd_bwd(W1d, W2d, Md, bits=bits, group1=g1, group2=g2, replicas=r, P=P, lse_t=t,
                                     lambda_orth=lam, flags=cq.FLAG_EXACT_LOSS)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    L = out["losses"].cpu().numpy()
    assert abs(L[0] - f["loss"]) <= TOL * abs(f["loss"])
    assert abs(L[1] - f["lse"]) <= TOL * abs(f["lse"])
    assert abs(L[2] - f["orth"]) <= TOL * f["orth"]
    assert abs(L[3] - f["pqe"] ** 2) <= TOL * f["pqe"] ** 2
    g = orc.pair_grad_lse(W1, W2, f, g1, g2)
    gg = out["gradM"].cpu().numpy()
    # the LSE gradient is dominated by a handful of arg-max entries: compare the whole parameter
    assert rel_err(gg, g) <= TOL


def test_optimize_pair_first_adam_step(cq):
    k, r, h, d1, d3 = 32, 2, 64, 96, 80
    W1b, W2b = syn.weight_student_t(h, d1, 61), syn.weight_student_t(d3, r * h, 62)
    # (a point off the rotations: exactly at M M^T = I the penalty's norm has no gradient and the device, which forms
    # M M^T in fp32, takes zero below a relative 1e-5)
    M0 = syn.perturbed_blocks(h // k, k, 7, 0.05)
    W1, W2 = w64(W1b), w64(W2b)
    f = orc.pair_forward(W1, W2, M0, 4, 0, 32, r, 5.0, 0.1, False)
    g = orc.pair_grad_lse(W1, W2, f, 0, 32)
    M1, _ = orc.adam_step(M0.astype(np.float64), g, (np.zeros_like(g), np.zeros_like(g), 0), 1e-2)
    Md = f32_dev(M0)
    cfg = cq.make_cfg(loss_kind=cq.LOSS_LSE, optimizer=cq.OPT_ADAM, lr=1e-2, steps=1, lambda_orth=0.1, lse_t=5.0)
    hist, status, _ = cq.cafeq_optimize_pair(to_dev(W1b), to_dev(W2b), Md, cfg, bits=4, group1=0, group2=32, replicas=r)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert abs(float(hist[0, 0].item()) - f["loss"]) <= TOL * abs(f["loss"])
    # Adam's first step is lr*sign(g): entries with |g| below the fp32 noise floor may flip, so compare where |g| matters
    d_gpu = Md.cpu().numpy() - M0
    d_ref = M1 - M0
    big = np.abs(g) > 1e-6 * np.abs(g).max()
    assert np.mean(np.sign(d_gpu[big]) == np.sign(d_ref[big])) > 0.999
    assert rel_err(d_gpu[big], d_ref[big]) <= 0.05


# ------------------------------------------------------------------ pack
@pytest.mark.parametrize("bits", [3, 4, 2, 8])
def test_pack_bit_exact(cq, bits):
    qm = orc.qmax_of(bits)
    q = np.random.default_rng(bits).integers(-qm, qm + 1, size=(33, 256)).astype(np.int8)
    p = cq.cafeq_pack(torch.from_numpy(q).cuda(), bits=bits)
    assert np.array_equal(p.cpu().numpy(), orc.pack_codes(q, bits))
