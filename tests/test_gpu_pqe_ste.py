"""GPU parity of the pair's straight-through gradient of the squared product error (Eq. 5 squared; the pairwise
loss itself of Section 4.2, differentiated with the quantiser passed through except for its scale) against the
float64 oracle, and a short optimisation run on it."""
import numpy as np
import pytest

import cafeq_synth as syn
from oracle import cafeq_oracle as orc
from parity_utils import device_inverse, tie_free_weight, f32_dev, rel_err, to_dev, w64

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cq():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2511_19705_b200 as m
    m.lib()
    return m


def _pair(h, d1, d3, r, seed):
    W1b = syn.weight_student_t(h, d1, seed, 2, 10.0)
    W2b = syn.weight_student_t(d3, r * h, seed + 1, 2, 10.0)
    return W1b, W2b


# (k, r, h, d1, d3, group1, group2, bits): every dimension a multiple of 64; several product tiles, r > 1,
# groups narrower and wider than a transform block
CASES = [(64, 1, 128, 192, 128, 64, 64, 4), (128, 2, 256, 384, 192, 128, 128, 3), (256, 2, 512, 384, 320, 128, 128, 3),
         (64, 4, 128, 256, 192, 128, 64, 3), (128, 1, 384, 256, 448, 64, 128, 4)]


@pytest.mark.parametrize("k,r,h,d1,d3,g1,g2,bits", CASES)
@pytest.mark.parametrize("generic", [False, True])
def test_pqe_ste_gradient_matches_oracle(cq, k, r, h, d1, d3, g1, g2, bits, generic):
    M = syn.perturbed_blocks(h // k, k, 23, 0.1)
    # identical transform parameters on both sides: the second factor's operator is bf16 of the inverse as the
    # device computes it; weights without rounding ties under either operator, so both sides decide the same codes
    Minv_c = orc.round_bf16(device_inverse(cq, M, generic))
    McT = np.transpose(orc.round_bf16(M), (0, 2, 1))
    seed = 300 + k + r
    W1b = tie_free_weight(lambda i: syn.weight_student_t(h, d1, seed + 1000 * i, 2, 10.0),
                          lambda W: orc.apply_blocks(W, McT, "out", 1), bits, g1, "cols")
    W2b = tie_free_weight(lambda i: syn.weight_student_t(d3, r * h, seed + 1 + 1000 * i, 2, 10.0),
                          lambda W: orc.apply_blocks(W, Minv_c, "in", r), bits, g2, "rows")
    W1d, W2d = to_dev(W1b), to_dev(W2b)
    P = cq.cafeq_pair_product(W1d, W2d, k=k, replicas=r)
    out = cq.cafeq_pair_loss_fwd_bwd(W1d, W2d, f32_dev(M), bits=bits, group1=g1, group2=g2, replicas=r, P=P,
                                     loss_kind=cq.LOSS_PQE_STE, flags=cq.FLAG_GENERIC if generic else 0)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    W1, W2 = w64(W1b), w64(W2b)
    f = orc.pair_forward(W1, W2, M, bits, g1, g2, r, 5.0, 0.0, True, Minv_c=Minv_c)
    L = out["losses"].cpu().numpy()
    pqe2 = f["pqe"] ** 2
    assert abs(L[0] - pqe2) <= 1e-3 * pqe2 and abs(L[3] - pqe2) <= 1e-3 * pqe2
    assert abs(L[1] - f["lse"]) <= 1e-3 * abs(f["lse"])
    g = orc.pair_grad_pqe_ste(W1, W2, f, bits, g1, g2)
    gg = out["gradM"].cpu().numpy()
    assert np.isfinite(gg).all()
    assert rel_err(gg, g) <= 1e-3
    for b in range(g.shape[0]):
        assert rel_err(gg[b], g[b]) <= 1e-3, f"block {b}"


def test_pqe_ste_refuses_shapes_off_the_tensor_core_grid(cq):
    W1b, W2b = _pair(128, 100, 96, 1, 7)
    M = syn.perturbed_blocks(2, 64, 3, 0.05)
    W1d, W2d = to_dev(W1b), to_dev(W2b)
    P = cq.cafeq_pair_product(W1d, W2d, k=64, replicas=1)
    with pytest.raises(RuntimeError, match="unsupported"):
        cq.cafeq_pair_loss_fwd_bwd(W1d, W2d, f32_dev(M), bits=4, group1=0, group2=64, replicas=1, P=P,
                                   loss_kind=cq.LOSS_PQE_STE)


def test_pqe_ste_optimisation_lowers_the_product_error(cq):
    """Adam on the straight-through gradient from the identity: the history's two columns are both PQE^2 and the
    best value seen is below the starting one (the starting value equals round-to-nearest without transform)."""
    k, r, h, d1, d3 = 128, 2, 256, 384, 192
    W1b, W2b = _pair(h, d1, d3, r, 911)
    W1d, W2d = to_dev(W1b), to_dev(W2b)
    P = cq.cafeq_pair_product(W1d, W2d, k=k, replicas=r)
    M = f32_dev(syn.identity_blocks(h // k, k))
    cfg = cq.make_cfg(loss_kind=cq.LOSS_PQE_STE, optimizer=cq.OPT_ADAM, lr=1e-3, steps=30, eval_every=1)
    hist, status, _ = cq.cafeq_optimize_pair(W1d, W2d, M, cfg, bits=3, group1=128, group2=128, replicas=r, P=P)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    H = hist.cpu().numpy()
    assert np.isfinite(H).all() and np.array_equal(H[:, 0], H[:, 1])
    f0 = orc.pair_forward(w64(W1b), w64(W2b), syn.identity_blocks(h // k, k), 3, 128, 128, r, 5.0, 0.0, True)
    assert abs(H[0, 0] - f0["pqe"] ** 2) <= 1e-3 * f0["pqe"] ** 2
    assert H[1:, 0].min() < H[0, 0]
