"""Inference side (Section 4.1 and its table of extra FLOPs / wall-clock time): the block-diagonal multiplication of
the activations (cafeq_apply_transform) and the dequantisation of packed weights (cafeq_dequant) against the oracle.

The device writes bf16; both sides therefore round to bf16 at the end.  The fp32 accumulation order differs from the
oracle's float64 sum, so an output whose exact value lies next to a bf16 rounding boundary may land on the other
side: such entries must be rare, and every entry must lie within half a bf16 step of the exact value plus a bound on
the fp32 sum's error (which, where the terms cancel, can exceed a bf16 step of the small result)."""
import numpy as np
import pytest

import cafeq_synth as syn
from oracle import cafeq_oracle as orc
from parity_utils import f32_dev, to_dev, w64

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cq():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2511_19705_b200 as m
    m.lib()
    return m


def _bf16_check(Y_dev, Y64, A64, max_frac=2e-3):
    """Y_dev: float64 view of the device's bf16 output; Y64: exact result; A64: the same product over absolute values
    (what the fp32 accumulation error of an entry scales with)."""
    ref = orc.round_bf16(Y64.astype(np.float32)).astype(np.float64)
    frac = float((Y_dev != ref).mean())
    assert frac <= max_frac, f"{frac:.2e} of the outputs differ from the bf16 rounding of the exact result"
    # every entry: half a bf16 step of the exact value plus the fp32 sum's error (k terms, 2^-24 each, far from worst case)
    assert (np.abs(Y_dev - Y64) <= 2.0 ** -8 * np.abs(Y64) + 2.0 ** -18 * A64 + 1e-30).all()
    # and in norm: bf16 rounding only
    assert np.linalg.norm(Y_dev - Y64) <= 2.0 ** -8 * np.linalg.norm(Y64)


# (tokens, d_in, k): tensor-core shapes with several tiles and a ragged row tail, and shapes of the shape-agnostic path
APPLY_CASES = [(300, 512, 256), (200, 768, 128), (130, 256, 64), (65, 2304, 128), (50, 96, 32), (33, 192, 64)]


@pytest.mark.parametrize("tokens,d_in,k", APPLY_CASES)
@pytest.mark.parametrize("transpose", [False, True])
def test_apply_transform_matches_oracle(cq, tokens, d_in, k, transpose):
    Xb = syn.weight_student_t(tokens, d_in, 71, 3, 5.0)
    T = syn.perturbed_blocks(d_in // k, k, 23, 0.2)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = cq.cafeq_apply_transform(to_dev(Xb), f32_dev(T), trole=cq.APPLY_TT if transpose else cq.APPLY_T, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    Y64 = orc.inference_apply(w64(Xb), T, "in", transpose)
    A64 = orc.inference_apply(np.abs(w64(Xb)), np.abs(T), "in", transpose)
    _bf16_check(Y.float().cpu().numpy().astype(np.float64), Y64, A64)


def test_apply_transform_output_axis(cq):
    Xb = syn.weight_student_t(512, 384, 72, 3, 5.0)
    T = syn.perturbed_blocks(2, 256, 24, 0.2)
    Y = cq.cafeq_apply_transform(to_dev(Xb), f32_dev(T), taxis=cq.AXIS_OUT)
    torch.cuda.synchronize()
    _bf16_check(Y.float().cpu().numpy().astype(np.float64), orc.inference_apply(w64(Xb), T, "out", False),
                orc.inference_apply(np.abs(w64(Xb)), np.abs(T), "out", False))


def test_transformed_quantised_product_is_the_original_up_to_quantisation(cq):
    """End to end on the device: quantise W o M, pack, dequantise, multiply the activations by M^-T: the result is
    W x up to the quantisation error (which the oracle's float64 chain gives), not up to anything else."""
    d_out, d_in, k, bits, g, tokens = 192, 512, 128, 4, 128, 64
    Wb = syn.weight_student_t(d_out, d_in, 81, 2, 10.0)
    Xb = syn.weight_student_t(tokens, d_in, 82, 3, 5.0)
    M = syn.perturbed_blocks(d_in // k, k, 25, 0.1)
    Mc = orc.round_bf16(M.astype(np.float32)).astype(np.float64)
    Minv = np.linalg.inv(Mc)
    codes, scales = cq.cafeq_rtn(to_dev(Wb), f32_dev(M), bits=bits, group=g, tblock=k)
    packed = cq.cafeq_pack(codes, bits=bits)
    What = cq.cafeq_dequant(packed, scales, bits=bits, group=g, d_in=d_in)
    Xp = cq.cafeq_apply_transform(to_dev(Xb), f32_dev(Minv.astype(np.float32)), trole=cq.APPLY_TT)
    torch.cuda.synchronize()
    y_dev = (Xp.double() @ What.double().T).cpu().numpy()
    # oracle chain in float64
    f = orc.single_forward(w64(Wb), M, bits, g, "in")
    Xp64 = orc.inference_apply(w64(Xb), Minv.astype(np.float32), "in", True)
    y_orc = Xp64 @ np.asarray(f["Uhat"], dtype=np.float64).T
    y_exact = w64(Xb) @ w64(Wb).T
    assert np.linalg.norm(y_dev - y_orc) <= 1e-2 * np.linalg.norm(y_orc)          # bf16 storage of both device operands
    # the quantisation error dominates what is left against the unquantised product, on both sides alike
    e_dev, e_orc = np.linalg.norm(y_dev - y_exact), np.linalg.norm(y_orc - y_exact)
    assert abs(e_dev - e_orc) <= 0.05 * e_orc


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("shape", [(64, 256, 128), (37, 384, 64), (5, 48, 16)])
def test_dequant_matches_oracle(cq, bits, shape):
    d_out, d_in, g = shape
    rng = np.random.default_rng(5 + bits)
    qm = 2 ** (bits - 1) - 1
    q = rng.integers(-qm, qm + 1, size=(d_out, d_in)).astype(np.int32)
    s = np.abs(rng.standard_normal((d_out, d_in // g))).astype(np.float32) + 1e-3
    packed = orc.pack_codes(q, bits)
    out = cq.cafeq_dequant(torch.from_numpy(packed).cuda(), torch.from_numpy(s).cuda(), bits=bits, group=g, d_in=d_in)
    torch.cuda.synchronize()
    ref = orc.round_bf16(orc.dequant(packed, s, bits, g, d_in).astype(np.float32))
    assert np.array_equal(out.float().cpu().numpy(), ref.astype(np.float32))     # fp32 product of an fp32 and a small integer is exact
