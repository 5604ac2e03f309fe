"""The layer-streaming loop (optimise every problem of a layer, round, pack) on a two-layer miniature weight set
against the oracle: optimised transforms, final codes (tie-aware, at the device's transform), packed bytes (bit-exact
from the device's codes), reported errors, and Algorithm 1's error history."""
import numpy as np
import pytest

import cafeq_synth as syn
from oracle import cafeq_oracle as orc
from parity_utils import assert_codes_tie_aware, rel_err, w64

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu
TOL = 1e-3


def test_two_layer_miniature_of_the_streaming_loop():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2511_19705_b200 as cq
    from paper_2511_19705_b200 import stream_layers as sl
    cq.lib()
    k, bits, group, steps = 128, 3, 128, 6
    spec = dict(bits=bits, group=group, k=k, steps=steps, singles=[("q", 384, 512), ("gate", 640, 256)],
                pairs=[("vo", ("v", 256, 384), ("o", 384, 512), 128, 2)])
    dev = torch.device("cuda", 0)
    for layer in range(2):
        weights = {"q": syn.weight_student_t(384, 512, 10 + layer, 2, 10.0), "gate": syn.weight_student_t(640, 256, 20 + layer, 1, 10.0),
                   "v": syn.weight_student_t(256, 384, 30 + layer, 2, 10.0), "o": syn.weight_student_t(384, 512, 40 + layer, 2, 10.0)}
        transforms = {"q": syn.perturbed_blocks(4, k, 50 + layer, 0.02), "gate": syn.perturbed_blocks(2, k, 60 + layer, 0.02),
                      "vo": syn.perturbed_blocks(2, k, 70 + layer, 0.02)}
        res = sl.process_layer(spec, weights, {n: t.copy() for n, t in transforms.items()}, dev, bits=bits, group=group, steps=steps,
                               alg1_iters=1, lr_frac=1e-2, pair_lr=1e-3, keep_outputs=True)
        for name in ("q", "gate"):
            W = w64(weights[name])
            r = res[name]
            Mr, hist = orc.optimize_single(W, transforms[name], bits, group, "in", steps, r["lr"])
            assert abs(r["loss_first"] - hist[0, 0]) <= TOL * hist[0, 0] and abs(r["loss_last"] - hist[-1, 0]) <= 2 * TOL * hist[-1, 0]
            Md = r["M"].numpy()
            assert rel_err(Md - transforms[name], Mr - transforms[name]) <= 1e-2, name
            # final codes / scales / packed bytes at the transform the device ended on
            U = orc.apply_blocks(W, orc.round_bf16(Md), "in")
            assert_codes_tie_aware(r["codes"].numpy(), r["scales"].numpy(), orc.quant_sym(U, bits, group), U, group)
            assert np.array_equal(r["packed"].numpy(), orc.pack_codes(r["codes"].numpy(), bits))
            assert np.array_equal(orc.unpack_codes(r["packed"].numpy(), bits, W.shape[1]), r["codes"].numpy())
            f = orc.single_forward(W, Md, bits, group, "in")
            assert abs(r["rel_l2"] - f["rel_l2"]) <= TOL * f["rel_l2"]
            assert r["loss_last"] < r["loss_first"]
        W1, W2 = w64(weights["v"]), w64(weights["o"])
        r = res["vo"]
        Mr, hist = orc.optimize_pair(W1, W2, transforms["vo"], bits, group, group, 2, steps, 1e-3, 5.0, 0.1)
        assert abs(r["loss_first"] - hist[0, 0]) <= TOL * abs(hist[0, 0]) and abs(r["loss_last"] - hist[-1, 0]) <= 2 * TOL * abs(hist[-1, 0])
        Md = r["M"].numpy()
        f = orc.pair_forward(W1, W2, Md, bits, group, group, 2, 5.0, 0.0, True)
        ref = orc.adaptive_round_stored(f["U"], f["V"], bits, group, group, k, 2, 1)
        H = np.array(r["pqe_history"])
        assert abs(H[0] - ref["pqe"][0]) <= 1e-2 * ref["pqe"][0] and abs(H[1] - ref["pqe"][1]) <= 2e-2 * ref["pqe"][1]
        assert abs(r["rel_pqe_independent"] - f["rel_pqe"]) <= 1e-2 * f["rel_pqe"]
        assert np.array_equal(r["packed1"].numpy(), orc.pack_codes(r["codes1"].numpy(), bits))
        assert np.array_equal(r["packed2"].numpy(), orc.pack_codes(r["codes2"].numpy(), bits))
        assert r["rel_pqe_adaptive"] <= r["rel_pqe_independent"]
