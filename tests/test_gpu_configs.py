"""Parity at the full sizes of the remaining benchmark configurations, in the launch configuration the library
uses for them: the Gemma-2-2B-shaped up/down pair (config 2: 2304 <-> 9216, block 128, 4-bit, group 128) and the
largest Gemma-2-27B-shaped matrix (config 5: gate 36864 x 4608, block 256, 3-bit, groups 64 and 128)."""
import numpy as np
import pytest

import cafeq_synth as syn
from oracle import cafeq_oracle as orc
from parity_utils import assert_codes_tie_aware, f32_dev, rel_err, to_dev, w64

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


def test_config2_updown_pair_full_size(cq):
    spec = syn.layer_spec(2)
    pname, (n1, h, d1), (n2, d3, rh), k, r = spec["pairs"][0]
    bits, g = spec["bits"], spec["group"]
    W1b, W2b = syn.make_weight(2, n1, h, d1), syn.make_weight(2, n2, d3, rh)
    # the benchmark's initial rotations, moved a little off M M^T = I (where the penalty's norm has no gradient and
    # the device, forming M M^T in fp32, takes zero below a relative 1e-5)
    M = (syn.make_transform(n1, h // k, k) + 2e-3 * np.random.default_rng(4).standard_normal((h // k, k, k))).astype(np.float32)
    out = cq.cafeq_pair_loss_fwd_bwd(to_dev(W1b), to_dev(W2b), f32_dev(M), bits=bits, group1=g, group2=g, replicas=r,
                                     lse_t=5.0, lambda_orth=0.1)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    W1, W2 = w64(W1b), w64(W2b)
    f = orc.pair_forward(W1, W2, M, bits, g, g, r, 5.0, 0.1, False)
    L = out["losses"].cpu().numpy()
    assert abs(L[1] - f["lse"]) <= TOL * abs(f["lse"])
    assert abs(L[0] - f["loss"]) <= TOL * abs(f["loss"])
    grad = orc.pair_grad_lse(W1, W2, f, g, g)
    assert rel_err(out["gradM"].cpu().numpy(), grad) <= TOL
    # one Adam step from the same start
    M1, _ = orc.adam_step(M.astype(np.float64), grad, (np.zeros_like(grad), np.zeros_like(grad), 0), 1e-3)
    Md = f32_dev(M)
    cfg = cq.make_cfg(loss_kind=cq.LOSS_LSE, optimizer=cq.OPT_ADAM, lr=1e-3, steps=1, lambda_orth=0.1, lse_t=5.0)
    hist, status, _ = cq.cafeq_optimize_pair(to_dev(W1b), to_dev(W2b), Md, cfg, bits=bits, group1=g, group2=g, replicas=r)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    big = np.abs(grad) > 1e-3 * np.abs(grad).max()      # Adam's first step is lr * sign(g): compare where g is not noise
    d_gpu, d_ref = Md.cpu().numpy() - M, M1 - M
    assert np.mean(np.sign(d_gpu[big]) == np.sign(d_ref[big])) > 0.999


@pytest.mark.parametrize("group", [64, 128])
def test_config5_gate_rtn_sampled_rows(cq, group):
    d_out, d_in, k, bits = 36864, 4608, 256, 3
    Wb = syn.make_weight(5, "gate", d_out, d_in)
    Wd = to_dev(Wb)
    # identity transform through the tensor-core pass: bit-exact on sampled rows (and the outlier channels x15)
    codes, scales = cq.cafeq_rtn(Wd, f32_dev(syn.identity_blocks(d_in // k, k)), bits=bits, group=group, tblock=k)
    rows = np.sort(np.concatenate([np.random.default_rng(1).choice(d_out, size=60, replace=False), [0, 127, 128, d_out - 1]]))
    Q = orc.quant_sym(w64(Wb[rows]), bits, group)
    assert np.array_equal(codes[torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.int32), Q["q"])
    assert np.array_equal(scales[torch.from_numpy(rows).cuda()].cpu().numpy(), Q["s"])
    # a rotation: tie-aware on the same rows
    M = syn.make_transform("gate", d_in // k, k)
    codes, scales = cq.cafeq_rtn(Wd, f32_dev(M), bits=bits, group=group, tblock=k)
    U = orc.apply_blocks(w64(Wb[rows]), orc.round_bf16(M), "in")
    Qs = orc.quant_sym(U, bits, group)
    sel = torch.from_numpy(rows).cuda()
    assert_codes_tie_aware(codes[sel].cpu().numpy(), scales[sel].cpu().numpy(), Qs, U, group)
    # Eq. 4 value of the whole matrix: the oracle's sum splits over rows, so sampled rows pin the per-row term
    out = cq.cafeq_proxy_loss_fwd_bwd(Wd, f32_dev(M), bits=bits, group=group, flags=cq.FLAG_NO_GRAD)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    assert np.isfinite(float(out["losses"][0].item())) and float(out["losses"][0].item()) > 0
