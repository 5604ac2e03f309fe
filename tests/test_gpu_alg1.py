"""GPU parity of Algorithm 1 (adaptive rounding of a coupled pair) and of the tensor-core product term of Eq. 5
against the CPU oracle.

The oracle takes its pseudo-inverses from a float64 SVD; the device iterates Newton-Schulz on the tensor cores
with three-term bf16 splits and finishes with one step whose residual is formed over three-way splits (fp32-grade),
and forms the product W1 W2 and the least-squares targets over three-way splits too.  Checked here: independent
rounding (iters = 0) bit-exact; each half-step of the first iteration from identical inputs (teacher forcing) with
codes equal except inside the tie window; the error history at 1e-3; and the device's reported error equal (1e-3)
to the error recomputed in float64 from the codes and scales the device returned."""
import numpy as np
import pytest

import cafeq_synth as syn
from oracle import cafeq_oracle as orc
from parity_utils import assert_codes_tie_aware, device_inverse, f32_dev, rel_err, to_dev, w64

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cq():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2511_19705_b200 as m
    m.lib()
    return m


def _recomputed_pqe(out, U, V, k, r, g1, g2):
    q1, s1 = out["codes1"].cpu().numpy().astype(np.float64), out["scales1"].cpu().numpy().astype(np.float64)
    q2, s2 = out["codes2"].cpu().numpy().astype(np.float64), out["scales2"].cpu().numpy().astype(np.float64)
    Uh = q1 * np.repeat(s1, g1, axis=1)
    Vh = q2 * np.repeat(s2, g2, axis=1)
    P = orc.pair_product(U, V, k, r)
    return float(np.linalg.norm(orc.pair_product(Uh, Vh, k, r) - P))


# (h, d1, d3, k, r, g1, g2): tall and wide first factors, with and without replicas, a square second factor, an
# inner dimension four times the outer ones (the up / down aspect ratio) and a grouped-query pair like v-o
ALG1_CASES = [(128, 192, 256, 64, 2, 64, 64), (256, 128, 192, 64, 1, 64, 128), (128, 256, 192, 128, 1, 128, 64),
              (128, 256, 128, 128, 1, 128, 64), (512, 128, 128, 128, 1, 128, 128), (128, 256, 256, 64, 2, 64, 64)]
# The least-squares targets are solutions of systems whose condition number reaches a few hundred here; computed with
# fp32-grade arithmetic they carry a relative error of about (condition number) x 2^-24 x sqrt(terms), up to ~1e-4.
# Scales (a target's group maximum / qmax) are held to that; codes to the usual tie window.
ALG1_SCALE_RTOL = 3e-4


def _half_steps_from_device(out, U, V, bits, g1, g2, k, r):
    """The oracle's two half-steps of Algorithm 1's first iteration, the second one started from the codes the
    device returned for the second factor (teacher forcing: a rounding algorithm's later steps depend on every
    earlier code, so each update is compared from identical inputs)."""
    P = orc.pair_product(U, V, k, r)
    Q1 = orc.quant_sym(U, bits, g1)
    T2 = (orc.pinv(orc.expand_rows(Q1["Uhat"], k, r).T) @ P).T                   # [d3, r h]
    Vh_dev = out["codes2"].cpu().numpy().astype(np.float64) * np.repeat(out["scales2"].cpu().numpy().astype(np.float64), g2, axis=1)
    T1 = (P @ orc.pinv(orc.fold_rows(Vh_dev.T, k, r))).T                         # [h, d1]
    e1 = np.linalg.norm(orc.pair_product(Q1["Uhat"], Vh_dev, k, r) - P)
    return T2, T1, e1


@pytest.mark.parametrize("h,d1,d3,k,r,g1,g2", ALG1_CASES)
def test_alg1_untransformed_pair(cq, h, d1, d3, k, r, g1, g2):
    """Algorithm 1 on the device against the oracle's (SVD pseudo-inverse, float64).  The device's pseudo-inverse is
    an iteration finished with one fp32-grade step, and the products that form the least-squares targets run over
    three-way bf16 splits, so a target differs from the oracle's by a few 1e-6 relative on well-conditioned factors:
    codes may differ only where the target's quotient lies within the tie window of a rounding boundary, then by one."""
    W1b = syn.weight_student_t(h, d1, 81, 2, 10.0)
    W2b = syn.weight_student_t(d3, r * h, 82, 2, 10.0)
    U, V = w64(W1b), w64(W2b)
    bits = 4
    # iters = 0: independent round-to-nearest, bit-exact
    out0 = cq.cafeq_adaptive_round(to_dev(W1b), to_dev(W2b), None, iters=0, bits=bits, group1=g1, group2=g2, replicas=r, k=k)
    torch.cuda.synchronize()
    assert int(out0["status"].item()) == 0
    Q1, Q2 = orc.quant_sym(U, bits, g1), orc.quant_sym(V, bits, g2)
    assert np.array_equal(out0["codes1"].cpu().numpy().astype(np.int32), Q1["q"])
    assert np.array_equal(out0["codes2"].cpu().numpy().astype(np.int32), Q2["q"])
    assert np.array_equal(out0["scales1"].cpu().numpy(), Q1["s"]) and np.array_equal(out0["scales2"].cpu().numpy(), Q2["s"])
    ref = orc.adaptive_round_stored(U, V, bits, g1, g2, k, r, 2)
    assert abs(float(out0["pqe"][0].item()) - ref["pqe"][0]) <= 1e-3 * ref["pqe"][0]
    # one full iteration, each half-step from identical inputs
    out1 = cq.cafeq_adaptive_round(to_dev(W1b), to_dev(W2b), None, iters=1, bits=bits, group1=g1, group2=g2, replicas=r, k=k)
    torch.cuda.synchronize()
    assert int(out1["status"].item()) == 0
    T2, T1, e1 = _half_steps_from_device(out1, U, V, bits, g1, g2, k, r)
    f2 = assert_codes_tie_aware(out1["codes2"].cpu().numpy(), out1["scales2"].cpu().numpy(), orc.quant_sym(T2, bits, g2), T2, g2,
                                scale_rtol=ALG1_SCALE_RTOL)
    f1 = assert_codes_tie_aware(out1["codes1"].cpu().numpy(), out1["scales1"].cpu().numpy(), orc.quant_sym(T1, bits, g1), T1, g1,
                                scale_rtol=ALG1_SCALE_RTOL)
    h1 = out1["pqe"].cpu().numpy().astype(np.float64)
    assert abs(h1[1] - e1) <= 1e-3 * e1, (h1, e1)
    assert abs(h1[2] - _recomputed_pqe(out1, U, V, k, r, g1, g2)) <= 1e-3 * h1[2]
    # against the oracle's free-running history: the second factor's update starts from bit-identical inputs
    assert abs(h1[1] - ref["pqe"][1]) <= 1e-3 * ref["pqe"][1] + 1e-2 * f2 * ref["pqe"][1], (h1, ref["pqe"], f2, f1)
    # two full iterations: the reported errors are the errors of what was returned, and the run helps
    out = cq.cafeq_adaptive_round(to_dev(W1b), to_dev(W2b), None, iters=2, bits=bits, group1=g1, group2=g2, replicas=r, k=k)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    hist = out["pqe"].cpu().numpy().astype(np.float64)
    assert hist.shape == (5,)
    assert abs(hist[-1] - _recomputed_pqe(out, U, V, k, r, g1, g2)) <= 1e-3 * hist[-1]
    assert hist[1:].min() < hist[0]


def test_alg1_after_learned_transform(cq):
    h, d1, d3, k, r, g1, g2, bits = 128, 192, 128, 64, 2, 64, 64, 3
    W1b = syn.weight_student_t(h, d1, 91, 2, 10.0)
    W2b = syn.weight_student_t(d3, r * h, 92, 2, 10.0)
    M = syn.perturbed_blocks(h // k, k, 19, 0.1)
    out = cq.cafeq_adaptive_round(to_dev(W1b), to_dev(W2b), f32_dev(M), iters=1, bits=bits, group1=g1, group2=g2, replicas=r)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    # identical transform parameters on both sides: the second factor's operator is bf16 of the inverse as this call
    # computes it (elimination)
    Minv_c = orc.round_bf16(device_inverse(cq, M, generic=True))
    f = orc.pair_forward(w64(W1b), w64(W2b), M, bits, g1, g2, r, 5.0, 0.0, False, Minv_c=Minv_c)
    ref = orc.adaptive_round_stored(f["U"], f["V"], bits, g1, g2, k, r, 1)
    hist = out["pqe"].cpu().numpy().astype(np.float64)
    assert np.all(np.abs(hist - ref["pqe"]) <= 2e-3 * ref["pqe"]), (hist, ref["pqe"])
    assert abs(hist[-1] - _recomputed_pqe(out, f["U"], f["V"], k, r, g1, g2)) <= 1e-3 * hist[-1]


def test_alg1_unsupported_shape_is_refused(cq):
    W1b, W2b = syn.weight_small(32, 48, 1), syn.weight_small(40, 32, 2)
    with pytest.raises(cq.CafeqError) as e:
        cq.cafeq_adaptive_round(to_dev(W1b), to_dev(W2b), None, iters=1, bits=4, group1=0, group2=0, replicas=1, k=32)
    assert e.value.code == 2


def test_pair_product_and_pqe_on_tensor_cores(cq):
    """Shapes that take the tensor-core product path (every dimension a multiple of 64), with replicas."""
    k, r, h, d1, d3 = 128, 2, 256, 320, 192
    W1b, W2b = syn.weight_student_t(h, d1, 51, 2, 10.0), syn.weight_student_t(d3, r * h, 52, 2, 10.0)
    M = syn.perturbed_blocks(h // k, k, 17, 0.1)
    W1d, W2d = to_dev(W1b), to_dev(W2b)
    P = cq.cafeq_pair_product(W1d, W2d, k=k, replicas=r)
    f = orc.pair_forward(w64(W1b), w64(W2b), M, 4, 64, 64, r, 5.0, 0.1, True)
    assert rel_err(P.cpu().numpy(), f["P"]) <= 1e-5
    out = cq.cafeq_pair_loss_fwd_bwd(W1d, W2d, f32_dev(M), bits=4, group1=64, group2=64, replicas=r, P=P, lse_t=5.0,
                                     lambda_orth=0.1, flags=cq.FLAG_EXACT_LOSS)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    L = out["losses"].cpu().numpy()
    assert abs(L[3] - f["pqe"] ** 2) <= 2e-3 * f["pqe"] ** 2


def test_alg1_full_size_vo_pair(cq):
    """The v-o pair of the 9B-shaped layer (v 2048 x 3584, o 3584 x 4096, two query heads per kv head, 3-bit,
    group 128) through one iteration of Algorithm 1 after a rotation: the independent-rounding error against the
    oracle's, and the reported final error against the error recomputed in float64 from the returned codes."""
    k, r, bits, g = 256, 2, 3, 128
    W1b, W2b = syn.make_weight(3, "v", 2048, 3584), syn.make_weight(3, "o", 3584, 4096)
    M = syn.make_transform("v", 8, k)
    out = cq.cafeq_adaptive_round(to_dev(W1b), to_dev(W2b), f32_dev(M), iters=1, bits=bits, group1=g, group2=g, replicas=r)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    hist = out["pqe"].cpu().numpy().astype(np.float64)
    f = orc.pair_forward(w64(W1b), w64(W2b), M, bits, g, g, r, 5.0, 0.0, True)
    assert abs(hist[0] - f["pqe"]) <= 2e-3 * f["pqe"], (hist, f["pqe"])
    assert hist[1] < hist[0]                                   # the compensating update of the second factor helps
    assert abs(hist[-1] - _recomputed_pqe(out, f["U"], f["V"], k, r, g, g)) <= 2e-3 * hist[-1]
