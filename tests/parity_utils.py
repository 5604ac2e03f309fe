"""Comparison helpers shared by the GPU parity tests (no method arithmetic beyond comparisons)."""
from __future__ import annotations

import numpy as np

import cafeq_synth as syn


def to_dev(bits_u16: np.ndarray):
    """bf16 bit patterns (numpy uint16) -> CUDA bf16 tensor."""
    import torch
    return torch.from_numpy(bits_u16.view(np.int16).copy()).cuda().view(torch.bfloat16)


def f32_dev(x: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()


def w64(bits_u16: np.ndarray) -> np.ndarray:
    return syn.bf16_bits_to_f64(bits_u16)


def rel_err(x, ref) -> float:
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    d = np.linalg.norm(x - ref)
    n = np.linalg.norm(ref)
    return float(d / n) if n > 0 else float(d)


TIE_WINDOW = 2.0 ** -18 * 16.0   # 2^-18 sqrt(k) for the largest block (k = 256): 6.1e-5 in code units
TIE_FRACTIONS = []               # (test id, fraction of codes that differed inside the window), read by conftest


def assert_codes_tie_aware(q_gpu, s_gpu, Q, U64, group, window=TIE_WINDOW, max_frac=1e-4, label=None, scale_rtol=1e-5):
    """Codes may differ from the oracle only where the oracle's quotient U/s sits within `window`
    (relative to max(1,|x|)) of a rounding boundary, then by exactly one; scales to 1e-5 relative.

    The device accumulates the transform product in fp32 on tensor cores / FMA units, the oracle
    in float64: a quotient closer to a half-integer than the accumulated rounding error can round
    either way.  The window is 2^-18 sqrt(k) max(1, |x|): k products of relative error 2^-24 each accumulate to
    about 2^-24 sqrt(k) |U|, a few times that in code units after the division by the scale.  The fraction of
    codes that differed is recorded (TIE_FRACTIONS) so that a run can report it."""
    q_gpu = np.asarray(q_gpu, dtype=np.int64)
    q_ref = np.asarray(Q["q"], dtype=np.int64)
    s_ref = Q["s"].astype(np.float64)
    s_gpu = np.asarray(s_gpu, dtype=np.float64)
    assert s_gpu.shape == s_ref.shape
    assert np.all(np.abs(s_gpu - s_ref) <= scale_rtol * np.abs(s_ref) + 1e-30), "scales differ"
    g = U64.shape[1] if group == 0 else group
    bad = q_gpu != q_ref
    frac = bad.mean()
    if bad.any():
        s_e = np.repeat(s_ref, g, axis=1)
        x = np.where(s_e > 0, U64 / np.where(s_e > 0, s_e, 1.0), 0.0)
        dist = np.abs(np.abs(x - np.floor(x)) - 0.5)
        assert np.all(np.abs(q_gpu - q_ref)[bad] == 1), "a code differs by more than one"
        assert np.all(dist[bad] <= window * np.maximum(1.0, np.abs(x[bad]))), "code differs away from a tie"
    assert frac <= max_frac, f"too many near-tie mismatches: {frac}"
    import os
    TIE_FRACTIONS.append((label or os.environ.get("PYTEST_CURRENT_TEST", "?").split(" ")[0], float(frac), int(bad.size)))
    return float(frac)


# ---------------------------------------------------------------------------------------------------------
# inputs without rounding ties
# ---------------------------------------------------------------------------------------------------------
def near_tie_mask(U64, bits, group, window, boundary="round"):
    """Entries of a transformed matrix whose quotient U/s lies within `window` * max(1, |x|) of a rounding boundary
    (half-integers for round-to-nearest; integers for boundary="floor", the floor + offset codes; the entries
    attaining the group's absmax are exempt there, they are coded +-qmax by rule), and groups whose two largest
    magnitudes are within 1e-5 relative of each other (either would let fp32 and float64 arithmetic disagree about
    an integer decision).  Returns a boolean [d_out, d_in] mask."""
    from oracle import cafeq_oracle as orc
    Q = orc.quant_sym(U64, bits, group)
    d_out, d_in = U64.shape
    g = d_in if group == 0 else group
    s_e = np.repeat(Q["s"].astype(np.float64), g, axis=1)
    x = np.where(s_e > 0, U64 / np.where(s_e > 0, s_e, 1.0), 0.0)
    if boundary == "floor":
        dist = np.abs(x - np.rint(x))
        a_e = np.repeat(Q["a"].astype(np.float64), g, axis=1)
        dist = np.where(np.abs(U64.astype(np.float32)) >= a_e, 1.0, dist)
    else:
        dist = np.abs(np.abs(x - np.floor(x)) - 0.5)
    bad = dist <= window * np.maximum(1.0, np.abs(x))
    A = np.sort(np.abs(U64).reshape(d_out, d_in // g, g), axis=2)
    close = (A[..., -1] - A[..., -2]) <= 1e-5 * A[..., -1]
    return bad | np.repeat(close, g, axis=1)


def tie_free_weight(draw, transform, bits, group, redraw, window=2e-4, max_iter=200, boundary="round"):
    """A seeded weight (bf16 bit patterns) none of whose transformed entries is a near-tie.

    draw(i) -> uint16 [d_out, d_in] bit patterns of the i-th independent draw; transform(W64) -> U64;
    redraw = "rows" when a transformed entry depends only on its own row of W (input-axis transform), "cols" when
    it depends only on its own column (output-axis transform).  Rows / columns holding a near-tie are replaced from
    the next draw until none is left.  Comparing the device with the oracle on such inputs removes the one
    difference that is not an error: an fp32 quotient and a float64 quotient landing on opposite sides of a
    half-integer."""
    Wb = draw(0).copy()
    for it in range(1, max_iter + 1):
        mask = near_tie_mask(transform(w64(Wb)), bits, group, window, boundary)
        lines = mask.any(axis=1) if redraw == "rows" else mask.any(axis=0)
        if not lines.any():
            return Wb
        fresh = draw(it)
        if redraw == "rows":
            Wb[lines] = fresh[lines]
        else:
            Wb[:, lines] = fresh[:, lines]
    raise AssertionError("could not draw a tie-free weight")


def device_inverse(cq, M, generic=False):
    """inv(bf16(M)) as the device computes it from a cold start (float32 numpy [nb,k,k]); the pair calls apply
    bf16 of exactly this to the second factor.  generic: the shape-agnostic kernels (elimination), as with
    FLAG_GENERIC."""
    import torch
    nb, k, _ = M.shape
    Wd = torch.zeros((64, nb * k), dtype=torch.bfloat16, device="cuda")
    out = cq.cafeq_proxy_loss_fwd_bwd(Wd, f32_dev(M), bits=4, group=0,
                                      flags=cq.FLAG_NO_GRAD | (cq.FLAG_GENERIC if generic else 0), want_minv=True)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    return out["Minv"].cpu().numpy()
