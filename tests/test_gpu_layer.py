"""GPU parity of the layer-level calls (cafeq_layer_prepare / cafeq_optimize_layer) against the CPU oracle.

A miniature layer (two single matrices, one grouped-query pair with two replicas, one plain pair) is advanced by the
layer call; with plain gradient descent the parameter change divided by the step size is the gradient the device
used, which is compared problem by problem with the oracle's gradient of Eq. 4 (singles) and of the LogSumExp
surrogate plus orthonormality penalty (pairs).  A second test free-runs two steps (Adam on the pairs, warm-started
inverse on the second step) against the oracle's own loops."""
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


def _mini_layer(k, group, seed):
    """Shapes with several tiles, ragged row tiles and both pair kinds; weights heavy-tailed like the benchmark's."""
    sing = [("q", 3 * k + 40, 2 * 256), ("gate", 5 * k, 256)]
    pairs = [("vo", (2 * k, 384), (384, 4 * k), 2), ("updown", (4 * k, 256), (256, 4 * k), 1)]
    S, P = [], []
    for i, (name, d_out, d_in) in enumerate(sing):
        S.append((name, syn.weight_student_t(d_out, d_in, seed + i, 2, 10.0), syn.perturbed_blocks(d_in // k, k, seed + 10 + i, 0.05)))
    for i, (name, (h, d1), (d3, rh), r) in enumerate(pairs):
        P.append((name, syn.weight_student_t(h, d1, seed + 20 + i, 2, 10.0), syn.weight_student_t(d3, rh, seed + 30 + i, 2, 10.0),
                  syn.perturbed_blocks(h // k, k, seed + 40 + i, 0.05), r))
    return S, P


def _build(cq, S, P, bits, group, lrs, pair_opt, max_steps):
    singles = [dict(W=to_dev(Wb), M=f32_dev(M), bits=bits, group=group,
                    cfg=cq.make_cfg(loss_kind=cq.LOSS_SURROGATE, optimizer=cq.OPT_GD, lr=lrs[n])) for n, Wb, M in S]
    pairs = [dict(W1=to_dev(W1b), W2=to_dev(W2b), M=f32_dev(M), bits=bits, group1=group, group2=group, replicas=r,
                  cfg=cq.make_cfg(loss_kind=cq.LOSS_LSE, optimizer=pair_opt, lr=lrs[n], beta1=0.1, beta2=0.999, eps=1e-8,
                                  lambda_orth=0.1, lse_t=5.0)) for n, W1b, W2b, M, r in P]
    return cq.LayerOptimizer(singles, pairs, max_steps=max_steps)


@pytest.mark.parametrize("k,group", [(128, 128), (256, 128), (256, 64), (128, 64)])
def test_layer_step_gradients_match_oracle(cq, k, group):
    bits = 3
    S, P = _mini_layer(k, group, 100 + k + group)
    ref, lrs = {}, {}
    for name, Wb, M in S:
        f = orc.single_forward(w64(Wb), M, bits, group, "in")
        g = orc.single_grad_surrogate(w64(Wb), f, group, "in")
        ref[name] = (f["surrogate"], g)
        lrs[name] = float(0.02 / np.abs(g).max())
    for name, W1b, W2b, M, r in P:
        f = orc.pair_forward(w64(W1b), w64(W2b), M, bits, group, group, r, 5.0, 0.1, False)
        g = orc.pair_grad_lse(w64(W1b), w64(W2b), f, group, group)
        ref[name] = (f["loss"], g)
        lrs[name] = float(0.02 / np.abs(g).max())
    opt = _build(cq, S, P, bits, group, lrs, cq.OPT_GD, 1)
    opt.step(1)
    torch.cuda.synchronize()
    assert int(opt.status.item()) == 0
    names = [n for n, *_ in S] + [n for n, *_ in P]
    M0s = [M for _, _, M in S] + [M for _, _, _, M, _ in P]
    for i, name in enumerate(names):
        loss_ref, g_ref = ref[name]
        loss = float(opt.hist[i][0, 0].item())
        assert abs(loss - loss_ref) <= TOL * abs(loss_ref), (name, loss, loss_ref)
        g_dev = (M0s[i].astype(np.float64) - opt.M[i].cpu().numpy().astype(np.float64)) / lrs[name]
        assert rel_err(g_dev, g_ref) <= TOL, (name, rel_err(g_dev, g_ref))
        for b in range(g_ref.shape[0]):
            # the parameters are fp32: a change read back from them carries their rounding (half an ulp per entry)
            floor = np.linalg.norm(M0s[i][b]) * 2.0 ** -24 / lrs[name]
            err = np.linalg.norm(g_dev[b] - g_ref[b])
            assert err <= 2 * TOL * np.linalg.norm(g_ref[b]) + floor, (name, b, err, np.linalg.norm(g_ref[b]), floor)


def test_layer_two_steps_free_running_adam(cq):
    k, group, bits = 128, 128, 4
    S, P = _mini_layer(k, group, 7)
    lrs = {}
    for name, Wb, M in S:
        f = orc.single_forward(w64(Wb), M, bits, group, "in")
        lrs[name] = float(0.01 / np.abs(orc.single_grad_surrogate(w64(Wb), f, group, "in")).max())
    for name, *_ in P:
        lrs[name] = 1e-3
    opt = _build(cq, S, P, bits, group, lrs, cq.OPT_ADAM, 2)
    opt.step(2)
    torch.cuda.synchronize()
    assert int(opt.status.item()) == 0
    i = 0
    for name, Wb, M in S:
        Mr, hist = orc.optimize_single(w64(Wb), M, bits, group, "in", 2, lrs[name])
        assert np.allclose(opt.hist[i][:, 0].cpu().numpy(), hist[:, 0], rtol=TOL)
        assert rel_err(opt.M[i].cpu().numpy() - M, Mr - M) <= 5e-3, name
        i += 1
    for name, W1b, W2b, M, r in P:
        Mr, hist = orc.optimize_pair(w64(W1b), w64(W2b), M, bits, group, group, r, 2, lrs[name], 5.0, 0.1)
        assert np.allclose(opt.hist[i][:, 0].cpu().numpy(), hist[:, 0], rtol=TOL)
        # Adam's first steps move every entry by about lr whatever the gradient's size: compare where the gradient
        # is not noise
        d_dev, d_ref = opt.M[i].cpu().numpy() - M, Mr - M
        big = np.abs(d_ref) > 0.5 * lrs[name]
        assert np.mean(np.sign(d_dev[big]) == np.sign(d_ref[big])) > 0.999, name
        assert rel_err(d_dev[big], d_ref[big]) <= 2e-2, name
        i += 1


def test_layer_call_rejects_what_it_does_not_cover(cq):
    Wb = syn.weight_student_t(256, 512, 3, 0, 1.0)
    M = syn.haar_blocks(8, 64, 1)  # block 64: the per-problem calls cover it, the layer call does not
    single = dict(W=to_dev(Wb), M=f32_dev(M), bits=4, group=64, cfg=cq.make_cfg(loss_kind=cq.LOSS_SURROGATE, optimizer=cq.OPT_GD, lr=0.1))
    with pytest.raises(cq.CafeqError) as e:
        cq.LayerOptimizer([single], [])
    assert e.value.code == 2
