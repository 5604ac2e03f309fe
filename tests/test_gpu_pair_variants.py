"""Appendix D.1's alternative pair objectives (mean and norm-weighted mean of the squared group maxima) and Appendix
D.2's Cayley optimiser on the device against the oracle."""
import numpy as np
import pytest

import cafeq_synth as syn
from oracle import cafeq_oracle as orc
from parity_utils import f32_dev, rel_err, to_dev, w64

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


CASES = [(32, 1, 0, 32, (64, 96, 80)), (64, 2, 128, 64, (128, 256, 192)), (256, 1, 128, 128, (256, 384, 320)),
         (128, 2, 128, 128, (256, 384, 256))]


@pytest.mark.parametrize("k,r,g1,g2,dims", CASES)
@pytest.mark.parametrize("objective", ["sumsq", "sumsq_weighted"])
def test_sum_of_squares_objectives_match_oracle(cq, k, r, g1, g2, dims, objective):
    h, d1, d3 = dims
    W1b = syn.weight_student_t(h, d1, 51, 2, 10.0)
    W2b = syn.weight_student_t(d3, r * h, 52, 2, 10.0)
    M = syn.perturbed_blocks(h // k, k, 17, 0.1)
    kind = cq.LOSS_SUMSQ if objective == "sumsq" else cq.LOSS_SUMSQ_WEIGHTED
    out = cq.cafeq_pair_loss_fwd_bwd(to_dev(W1b), to_dev(W2b), f32_dev(M), bits=4, group1=g1, group2=g2, replicas=r,
                                     loss_kind=kind, lambda_orth=0.1)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    W1, W2 = w64(W1b), w64(W2b)
    f = orc.pair_forward(W1, W2, M, 4, g1, g2, r, 5.0, 0.1, False, objective=objective)
    L = out["losses"].cpu().numpy()
    assert abs(L[1] - f["surrogate"]) <= TOL * f["surrogate"]
    assert abs(L[0] - f["loss"]) <= TOL * f["loss"]
    g = orc.pair_grad_lse(W1, W2, f, g1, g2)
    gg = out["gradM"].cpu().numpy()
    assert rel_err(gg, g) <= TOL
    for b in range(g.shape[0]):
        assert rel_err(gg[b], g[b]) <= TOL, f"block {b}"


def test_cayley_optimiser_keeps_rotations_and_matches_oracle(cq):
    k, r, h, d1, d3 = 64, 2, 128, 192, 128
    W1b, W2b = syn.weight_student_t(h, d1, 61, 2, 10.0), syn.weight_student_t(d3, r * h, 62, 2, 10.0)
    M0 = syn.haar_blocks(h // k, k, 7)
    W1, W2 = w64(W1b), w64(W2b)
    f = orc.pair_forward(W1, W2, M0, 4, 64, 64, r, 5.0, 0.0, False)
    g = orc.pair_grad_lse(W1, W2, f, 64, 64)
    A = g @ np.transpose(M0.astype(np.float64), (0, 2, 1))
    lr = float(0.05 / np.abs(A - np.transpose(A, (0, 2, 1))).sum(axis=2).max())     # lr ||A||_inf = 0.05
    steps = 3
    Mr, hist = orc.optimize_pair(W1, W2, M0, 4, 64, 64, r, steps, lr, 5.0, 0.0, beta1=0.1, optimizer="cayley")
    Md = f32_dev(M0)
    cfg = cq.make_cfg(loss_kind=cq.LOSS_LSE, optimizer=cq.OPT_CAYLEY, lr=lr, beta1=0.1, steps=steps, lambda_orth=0.0, lse_t=5.0)
    hd, status, _ = cq.cafeq_optimize_pair(to_dev(W1b), to_dev(W2b), Md, cfg, bits=4, group1=64, group2=64, replicas=r)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.allclose(hd[:, 0].cpu().numpy(), hist[:, 0], rtol=TOL)
    Mg = Md.cpu().numpy().astype(np.float64)
    assert rel_err(Mg - M0, Mr - M0) <= 5e-3
    I = np.eye(k)
    assert np.abs(Mg @ np.transpose(Mg, (0, 2, 1)) - I).max() <= 5e-6            # still a rotation (fp32)
