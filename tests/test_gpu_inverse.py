"""The block inverse on the device (Newton-Schulz on the tensor cores, checked per block, with an elimination
fall-back) against the oracle's float64 Gauss-Jordan, and the warm-start / resume plumbing around it."""
import numpy as np
import pytest

import cafeq_synth as syn
from oracle import cafeq_oracle as orc
from parity_utils import f32_dev, rel_err, to_dev, w64

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cq():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2511_19705_b200 as m
    m.lib()
    return m


@pytest.mark.parametrize("k", [64, 128, 256])
@pytest.mark.parametrize("eps", [0.0, 0.1, 1.5])
def test_inverse_matches_float64_from_near_rotation_to_far(cq, k, eps):
    """eps = 0: a rotation (converges at once); 0.1: the regime of the method; 1.5: far from orthogonal, where the
    iteration from M^T does not converge and the per-block check hands the block to the elimination kernel."""
    d_out, d_in = 64, 2 * k
    Wb = syn.weight_student_t(d_out, d_in, 5)
    M = syn.perturbed_blocks(2, k, 23, eps) if eps > 0 else syn.haar_blocks(2, k, 23)
    out = cq.cafeq_proxy_loss_fwd_bwd(to_dev(Wb), f32_dev(M), bits=4, group=64, flags=cq.FLAG_NO_GRAD, want_minv=True)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    ref = orc.block_inverse(orc.round_bf16(M))
    assert rel_err(out["Minv"].cpu().numpy(), ref) <= 1e-4
    f = orc.single_forward(w64(Wb), M, 4, 64, "in")
    assert abs(float(out["losses"][0].item()) - f["surrogate"]) <= 1e-3 * f["surrogate"]


def test_warm_start_refines_a_nearby_inverse(cq):
    k = 128
    Wb = syn.weight_student_t(96, 2 * k, 6)
    M0 = syn.perturbed_blocks(2, k, 29, 0.1)
    rng = np.random.default_rng(3)
    M1 = (M0 + 2e-3 * rng.standard_normal(M0.shape) / np.sqrt(k)).astype(np.float32)   # one small optimiser step away
    Wd = to_dev(Wb)
    first = cq.cafeq_proxy_loss_fwd_bwd(Wd, f32_dev(M0), bits=4, group=64, flags=cq.FLAG_NO_GRAD, want_minv=True)
    Minv = first["Minv"].clone()
    warm = cq.cafeq_proxy_loss_fwd_bwd(Wd, f32_dev(M1), bits=4, group=64, flags=cq.FLAG_NO_GRAD | cq.FLAG_WARM_MINV, Minv=Minv)
    torch.cuda.synchronize()
    assert int(warm["status"].item()) == 0
    assert rel_err(Minv.cpu().numpy(), orc.block_inverse(orc.round_bf16(M1))) <= 1e-4
    # a useless warm start (zeros) must not leak into the result: the check falls back to elimination
    junk = torch.zeros_like(Minv)
    out = cq.cafeq_proxy_loss_fwd_bwd(Wd, f32_dev(M1), bits=4, group=64, flags=cq.FLAG_NO_GRAD | cq.FLAG_WARM_MINV, Minv=junk)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    assert rel_err(junk.cpu().numpy(), orc.block_inverse(orc.round_bf16(M1))) <= 1e-4


def test_chunked_pair_run_with_resume_matches_one_call(cq):
    k, r, h, d1, d3 = 64, 2, 128, 192, 128
    W1b, W2b = syn.weight_student_t(h, d1, 61), syn.weight_student_t(d3, r * h, 62)
    M0 = syn.haar_blocks(h // k, k, 7)
    kw = dict(bits=4, group1=64, group2=64, replicas=r)
    cfg3 = cq.make_cfg(loss_kind=cq.LOSS_LSE, optimizer=cq.OPT_ADAM, lr=1e-3, steps=3)
    Ma = f32_dev(M0)
    ha, sa, _ = cq.cafeq_optimize_pair(to_dev(W1b), to_dev(W2b), Ma, cfg3, **kw)
    Mb = f32_dev(M0)
    cfg1 = cq.make_cfg(loss_kind=cq.LOSS_LSE, optimizer=cq.OPT_ADAM, lr=1e-3, steps=1)
    _, _, st = cq.cafeq_optimize_pair(to_dev(W1b), to_dev(W2b), Mb, cfg1, **kw)
    cfg1r = cq.make_cfg(loss_kind=cq.LOSS_LSE, optimizer=cq.OPT_ADAM, lr=1e-3, steps=1, resume=1)
    for _ in range(2):
        hb, sb, st = cq.cafeq_optimize_pair(to_dev(W1b), to_dev(W2b), Mb, cfg1r, opt_state=st, **kw)
    torch.cuda.synchronize()
    assert int(sa.item()) == 0 and int(sb.item()) == 0
    assert float(st[0].item()) == 3.0                                  # three optimiser steps counted
    # Same arithmetic in the same order up to the floating-point atomics of the reductions.  Adam's first steps are
    # lr * g / (|g| + eps): an entry whose gradient is a structural zero plus summation noise steps anywhere in
    # [-lr, lr] depending on the order of the atomic adds, in either run (the LogSumExp gradient reaches most entries
    # only through such noise).  The comparison is therefore on the entries whose first moment is well above that
    # noise; they agree to 1e-3 of a step, and the loss history agrees.
    da, db = Ma.cpu().numpy() - M0, Mb.cpu().numpy() - M0
    m1 = st[cq.OPT_STATE_HEADER:cq.OPT_STATE_HEADER + M0.size].cpu().numpy().reshape(M0.shape)
    # (an entry at 1e-3 of the largest first moment sits where the summation noise is about 1e-3 of the entry itself,
    # i.e. exactly at the tolerance: the mask starts a decade above that)
    big = np.abs(m1) > 1e-2 * np.abs(m1).max()
    assert big.sum() >= 50
    off = np.abs(da - db)[big] > 1e-3 * 1e-3
    assert off.mean() <= 2e-2, int(off.sum())
    assert abs(float(hb[0, 0].item()) - float(ha[2, 0].item())) <= 1e-3 * abs(float(ha[2, 0].item()))


def test_overlap_mode_does_not_change_results(cq):
    """The process-wide launch-shape knob is a tuning parameter only: forward + backward of a
    single matrix give the same losses and (to accumulation order) the same gradient in both modes."""
    k, d_out, d_in = 256, 192, 768
    Wb = syn.weight_student_t(d_out, d_in, seed=5, n_outlier_channels=2, mult=10.0)
    M = f32_dev(syn.perturbed_blocks(d_in // k, k, 9, 0.1))
    outs = []
    try:
        for n in (False, True):
            cq.set_overlap_mode(n)
            o = cq.cafeq_proxy_loss_fwd_bwd(to_dev(Wb), M, bits=3, group=128, flags=cq.FLAG_EXACT_LOSS)
            torch.cuda.synchronize()
            assert int(o["status"].item()) == 0
            outs.append((o["losses"].cpu().numpy().copy(), o["gradM"].cpu().numpy().copy()))
        with pytest.raises(RuntimeError):
            cq._check(cq.lib().cafeq_set_overlap_mode(7), "cafeq_set_overlap_mode")
    finally:
        cq.set_overlap_mode(False)
    assert np.allclose(outs[0][0], outs[1][0], rtol=1e-6)
    assert rel_err(outs[0][1], outs[1][1]) <= 1e-5
