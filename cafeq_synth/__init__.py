"""Seeded synthetic inputs for the CafeQ hot path.

This module only *draws numbers*: weight matrices with the shapes and value
distributions of the workloads, random rotation blocks used as the starting
transform, and a few structured transforms (identity, signed permutations,
power-of-two diagonals) that tests use.  It contains none of the method's
arithmetic (no quantiser, no loss, no gradient); both the CPU oracle and the
CUDA path consume what it returns.

Weights are returned as bf16 *bit patterns* (numpy uint16), so that both
consumers start from exactly the same representable values.  The stand-in
recipe (the trained Gemma 2 checkpoints the paper quantises are not available):

* config 1: entries N(0, 0.02^2), a seeded 0.5 % of the entries multiplied by 20;
* configs 2-5: Student-t(df=4) entries scaled to standard deviation 1/sqrt(d_in)
  (a t4 variate has variance 2), with a seeded set of input channels multiplied
  by a constant (config 2: 8 channels x10; configs 4-5: round(0.001*d_in),
  at least 1, channels x15; config 3: none).
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 20251119


# --------------------------------------------------------------------------
# bf16 containers (representation only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bf16 (round-to-nearest-even), return uint16 bits."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([int(k) for k in key])))


# --------------------------------------------------------------------------
# weights
# --------------------------------------------------------------------------
def weight_gauss_outliers(d_out: int, d_in: int, seed: int, std: float = 0.02,
                          frac: float = 0.005, mult: float = 20.0) -> np.ndarray:
    """Config-1 style weight: N(0, std^2) with a seeded fraction of entries x mult."""
    rng = _rng(seed, 1)
    w = rng.standard_normal((d_out, d_in), dtype=np.float32) * np.float32(std)
    n = d_out * d_in
    n_out = int(round(frac * n))
    if n_out:
        pos = _rng(seed, 2).choice(n, size=n_out, replace=False)
        w.reshape(-1)[pos] *= np.float32(mult)
    return f32_to_bf16_bits(w)


def weight_student_t(d_out: int, d_in: int, seed: int, n_outlier_channels: int = 0,
                     mult: float = 1.0) -> np.ndarray:
    """Heavy-tailed weight: t(4) scaled to std 1/sqrt(d_in); outlier input channels x mult."""
    rng = _rng(seed, 1)
    w = np.empty((d_out, d_in), dtype=np.float32)
    rows = max(1, (1 << 22) // d_in)
    scale = 1.0 / np.sqrt(2.0 * d_in)
    for r0 in range(0, d_out, rows):
        r1 = min(d_out, r0 + rows)
        w[r0:r1] = (rng.standard_t(4.0, size=(r1 - r0, d_in)) * scale).astype(np.float32)
    if n_outlier_channels:
        ch = _rng(seed, 2).choice(d_in, size=n_outlier_channels, replace=False)
        w[:, ch] *= np.float32(mult)
    return f32_to_bf16_bits(w)


def weight_small(d_out: int, d_in: int, seed: int, scale: float = 1.0) -> np.ndarray:
    """Small dense Gaussian weight for unit tests."""
    w = _rng(seed, 3).standard_normal((d_out, d_in)).astype(np.float32) * np.float32(scale)
    return f32_to_bf16_bits(w)


# --------------------------------------------------------------------------
# transforms
# --------------------------------------------------------------------------
def haar_blocks(nb: int, k: int, seed: int) -> np.ndarray:
    """nb random rotations of size k (QR of a seeded Gaussian, diag(R) sign fixed)."""
    rng = _rng(seed, 4)
    out = np.empty((nb, k, k), dtype=np.float64)
    for b in range(nb):
        g = rng.standard_normal((k, k))
        q, r = np.linalg.qr(g)
        q = q * np.sign(np.diag(r))[None, :]
        out[b] = q
    return out.astype(np.float32)


def perturbed_blocks(nb: int, k: int, seed: int, eps: float = 0.05) -> np.ndarray:
    """Rotation blocks plus a small dense perturbation (invertible, not orthogonal)."""
    q = haar_blocks(nb, k, seed).astype(np.float64)
    e = _rng(seed, 5).standard_normal((nb, k, k)) * (eps / np.sqrt(k))
    return (q + e).astype(np.float32)


def identity_blocks(nb: int, k: int) -> np.ndarray:
    return np.broadcast_to(np.eye(k, dtype=np.float32), (nb, k, k)).copy()


def signed_perm_blocks(nb: int, k: int, seed: int, within: int | None = None) -> np.ndarray:
    """Signed permutation blocks; `within` keeps each index inside its run of that length."""
    rng = _rng(seed, 6)
    out = np.zeros((nb, k, k), dtype=np.float32)
    w = within or k
    for b in range(nb):
        for s0 in range(0, k, w):
            p = rng.permutation(w) + s0
            sg = rng.choice([-1.0, 1.0], size=w)
            out[b, np.arange(s0, s0 + w), p] = sg
    return out


def pow2_diag_blocks(nb: int, k: int, seed: int, emin: int = -3, emax: int = 3) -> np.ndarray:
    """Diagonal blocks with entries +-2^e (products with bf16 values stay exact)."""
    rng = _rng(seed, 7)
    out = np.zeros((nb, k, k), dtype=np.float32)
    for b in range(nb):
        e = rng.integers(emin, emax + 1, size=k)
        sg = rng.choice([-1.0, 1.0], size=k)
        out[b, np.arange(k), np.arange(k)] = sg * np.exp2(e)
    return out


def hadamard_blocks(nb: int, k: int, seed: int) -> np.ndarray:
    """Randomised Hadamard blocks H diag(+-1) / sqrt(k) (k a power of two; Sylvester construction): the fixed,
    data-independent rotation used as the random baseline.  For k = 4^m every entry is +-2^-m, exact in bf16."""
    assert k > 0 and (k & (k - 1)) == 0
    h = np.ones((1, 1))
    while h.shape[0] < k:
        h = np.block([[h, h], [h, -h]])
    rng = _rng(seed, 8)
    out = np.empty((nb, k, k), dtype=np.float64)
    for b in range(nb):
        out[b] = h * rng.choice([-1.0, 1.0], size=k)[None, :] / np.sqrt(k)
    return out.astype(np.float32)


# --------------------------------------------------------------------------
# workload tables (shapes of the benchmark configurations)
# --------------------------------------------------------------------------
# role: "single" -> axis IN, applies M; "pair" -> (W1 stored [h, d1], W2 stored [d3, r*h])
def layer_spec(config: int) -> dict:
    if config == 1:
        return dict(bits=4, group=128, k=128, steps=50,
                    singles=[("w", 256, 512)], pairs=[])
    if config == 2:
        return dict(bits=4, group=128, k=128, steps=200, singles=[],
                    pairs=[("updown", ("up", 9216, 2304), ("down", 2304, 9216), 128, 1)])
    if config in (3, 4):
        return dict(bits=3, group=128, k=256, steps=500,
                    singles=[("q", 4096, 3584), ("k", 2048, 3584), ("gate", 14336, 3584)],
                    pairs=[("vo", ("v", 2048, 3584), ("o", 3584, 4096), 256, 2),
                           ("updown", ("up", 14336, 3584), ("down", 3584, 14336), 256, 1)])
    if config == 5:
        return dict(bits=3, group=128, k=256, steps=500,
                    singles=[("q", 4096, 4608), ("k", 2048, 4608), ("gate", 36864, 4608)],
                    pairs=[("vo", ("v", 2048, 4608), ("o", 4608, 4096), 128, 2),
                           ("updown", ("up", 36864, 4608), ("down", 4608, 36864), 256, 1)])
    raise ValueError("config must be 1..5")


_MATRIX_ID = {"w": 0, "q": 1, "k": 2, "gate": 3, "v": 4, "o": 5, "up": 6, "down": 7}


def make_weight(config: int, name: str, d_out: int, d_in: int, layer: int = 0) -> np.ndarray:
    """The seeded stand-in weight `name` of `config`, layer `layer` (bf16 bits [d_out, d_in])."""
    seed = BASE_SEED + layer
    mid = _MATRIX_ID[name]
    if config == 1:
        return weight_gauss_outliers(d_out, d_in, seed * 16 + mid)
    if config == 2:
        return weight_student_t(d_out, d_in, seed * 16 + mid, 8, 10.0)
    if config == 3:
        return weight_student_t(d_out, d_in, seed * 16 + mid)
    n_ch = max(1, int(round(0.001 * d_in)))
    return weight_student_t(d_out, d_in, seed * 16 + mid, n_ch, 15.0)


def make_transform(name: str, nb: int, k: int, layer: int = 0) -> np.ndarray:
    return haar_blocks(nb, k, (BASE_SEED + 10**6 + layer) * 16 + _MATRIX_ID[name])
