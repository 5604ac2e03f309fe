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


def assert_codes_tie_aware(q_gpu, s_gpu, Q, U64, group, window=2e-4, max_frac=2e-3):
    """Codes may differ from the oracle only where the oracle's quotient U/s sits within `window`
    (relative to max(1,|x|)) of a rounding boundary, then by exactly one; scales to 1e-5 relative.

    The device accumulates the transform product in fp32 on tensor cores / FMA units, the oracle
    in float64: a quotient closer to a half-integer than the accumulated rounding error can round
    either way."""
    q_gpu = np.asarray(q_gpu, dtype=np.int64)
    q_ref = np.asarray(Q["q"], dtype=np.int64)
    s_ref = Q["s"].astype(np.float64)
    s_gpu = np.asarray(s_gpu, dtype=np.float64)
    assert s_gpu.shape == s_ref.shape
    assert np.all(np.abs(s_gpu - s_ref) <= 1e-5 * np.abs(s_ref) + 1e-30), "scales differ"
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
    return float(frac)
