"""Seeded synthetic inputs for the KroQuant online quantizer.

This module only *draws inputs*: activations as bf16 bit patterns, Kronecker
factors, LU parameters and per-channel scales.  It holds none of the method's
arithmetic (no transform, no MXFP4 encoding), so both the CPU oracle's tests and
the CUDA path can take their inputs from it without sharing any of the code
under test.

The paper's own workloads are DiT activations (PixArt-Sigma, SANA,
FLUX.1-schnell; Section 4.1) that are not available offline.  The tensors here
take their *shapes* from the paper's production-shape latency table (Appendix A)
and their *structure* from what the paper says about DiT activations: a few
channels orders of magnitude larger than the rest (Section 1), and text/image
token heterogeneity in FLUX (Section 4.2).

Draw order is fixed: values, then outlier-channel indices, then spike-row
indices; factors and scales come from ``default_rng(seed + 1000 + layer)``.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

BLOCK = 32  # channels per MX block (paper Section 3.1/3.2: n = 32)


# --------------------------------------------------------------------------
# bf16 bit helpers (input representation only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (round-to-nearest-even) and return the
    16-bit patterns as uint16.  Inputs must be finite."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float32."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32)


def f32_to_fp16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to IEEE binary16 (NumPy's round-to-nearest-even cast) and return
    the 16-bit patterns.  Inputs must be finite and below 65504 in magnitude."""
    return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)


def fp16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(bits, dtype=np.uint16).view(np.float16).astype(np.float32)


# --------------------------------------------------------------------------
# factors, LU parameters, scales
# --------------------------------------------------------------------------
def gen_factors(seed: int, n_sets: int = 1, layer: int = 0) -> np.ndarray:
    """Well-conditioned 2x2 factors ``G[n_sets, 5, 2, 2]`` (float32).

    Each factor is a random orthogonal matrix (QR of a Gaussian 2x2 with the
    sign fixed by diag(R)) times ``diag(u1, u2)``, ``u ~ U[0.5, 2]``.
    """
    rng = np.random.default_rng(seed + 1000 + layer)
    G = np.empty((n_sets, 5, 2, 2), dtype=np.float32)
    for s in range(n_sets):
        for k in range(5):
            Q, R = np.linalg.qr(rng.standard_normal((2, 2)))
            Q = Q * np.sign(np.diag(R))
            u = rng.uniform(0.5, 2.0, size=2)
            G[s, k] = (Q * u[None, :]).astype(np.float32)
    return G


def identity_factors(n_sets: int = 1) -> np.ndarray:
    G = np.zeros((n_sets, 5, 2, 2), dtype=np.float32)
    G[:, :, 0, 0] = 1.0
    G[:, :, 1, 1] = 1.0
    return G


def hadamard_lu_params(n_sets: int = 1) -> np.ndarray:
    """(a, b, c) = (1/sqrt2, 1/sqrt2, 1): the paper's Hadamard initialisation
    (Section 3.2, "Hadamard initialization")."""
    abc = np.empty((n_sets, 5, 3), dtype=np.float32)
    abc[..., 0] = 1.0 / math.sqrt(2.0)
    abc[..., 1] = 1.0 / math.sqrt(2.0)
    abc[..., 2] = 1.0
    return abc


def gen_lu_params(seed: int, n_sets: int = 1, layer: int = 0) -> np.ndarray:
    """Perturbed-Hadamard LU parameters ``abc[n_sets, 5, 3]`` (float32): the
    kind of factor set the paper's calibration produces after a few steps."""
    rng = np.random.default_rng(seed + 1000 + layer)
    a = np.exp(rng.normal(0.0, 0.2, size=(n_sets, 5))) / math.sqrt(2.0)
    b = 1.0 / math.sqrt(2.0) + rng.normal(0.0, 0.2, size=(n_sets, 5))
    c = 1.0 + rng.normal(0.0, 0.2, size=(n_sets, 5))
    return np.stack([a, b, c], axis=-1).astype(np.float32)


def gen_channel_scales(seed: int, d: int, layer: int = 0) -> np.ndarray:
    """Per-channel multipliers ``s[d] ~ U[0.25, 4]`` (float32) for the
    SmoothQuant-style comparison kernel."""
    rng = np.random.default_rng(seed + 1000 + layer)
    return rng.uniform(0.25, 4.0, size=d).astype(np.float32)


# --------------------------------------------------------------------------
# activations
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class ActivationSpec:
    """Recipe for one activation tensor ``X[tokens, d]``."""
    name: str
    tokens: int
    d: int
    seed: int
    outlier_channels: int          # number of channels multiplied by outlier_gain
    outlier_gain: float
    spike_rows: int = 0            # number of random rows multiplied by spike_gain
    spike_gain: float = 1.0
    gelu: bool = False             # pass N(0,1) through exact GELU first
    tail_rows: int = 0             # last `tail_rows` rows multiplied by tail_gain
    tail_gain: float = 1.0


def _gelu(z: np.ndarray) -> np.ndarray:
    from scipy.special import erf  # exact GELU 0.5 z (1 + erf(z / sqrt 2))
    return (0.5 * z * (1.0 + erf(z / math.sqrt(2.0)))).astype(np.float32)


def gen_activations_f32(spec: ActivationSpec) -> np.ndarray:
    rng = np.random.default_rng(spec.seed)
    x = rng.standard_normal((spec.tokens, spec.d), dtype=np.float32)
    if spec.gelu:
        x = _gelu(x)
    if spec.outlier_channels:
        ch = rng.choice(spec.d, size=spec.outlier_channels, replace=False)
        x[:, ch] *= np.float32(spec.outlier_gain)
    if spec.spike_rows:
        rows = rng.choice(spec.tokens, size=spec.spike_rows, replace=False)
        x[rows, :] *= np.float32(spec.spike_gain)
    if spec.tail_rows:
        x[spec.tokens - spec.tail_rows:, :] *= np.float32(spec.tail_gain)
    return x


def gen_activations(spec: ActivationSpec, dtype: str = "bf16") -> np.ndarray:
    """16-bit patterns (uint16) of the activation tensor, shape [tokens, d]; bf16 or fp16."""
    x = gen_activations_f32(spec)
    return f32_to_fp16_bits(x) if dtype == "fp16" else f32_to_bf16_bits(x)


def gen_dense_blocks(seed: int, n_sets: int = 1) -> np.ndarray:
    """Random well-conditioned dense 32x32 blocks (not Kronecker-structured): orthogonal (QR of a
    Gaussian) times diag(U[0.5, 2])."""
    rng = np.random.default_rng(seed + 2000)
    out = np.empty((n_sets, 32, 32), np.float32)
    for s in range(n_sets):
        Q, R = np.linalg.qr(rng.standard_normal((32, 32)))
        Q = Q * np.sign(np.diag(R))
        out[s] = (Q * rng.uniform(0.5, 2.0, size=32)[None, :]).astype(np.float32)
    return out


def gen_weights(seed: int, o: int, d: int) -> np.ndarray:
    """bf16 bit patterns of a synthetic linear-layer weight ``W[o, d]``: N(0, 1/d) entries with a
    log-normal per-input-channel gain (sigma 0.5), the kind of channel imbalance smoothing and
    rotations are meant to even out.  Used by the calibration workload only."""
    rng = np.random.default_rng(seed + 3000)
    w = rng.standard_normal((o, d), dtype=np.float32) / np.float32(math.sqrt(d))
    gain = np.exp(rng.normal(0.0, 0.5, size=d)).astype(np.float32)
    return f32_to_bf16_bits(w * gain[None, :])


def calib_spec(rows: int, d: int, seed: int = 5) -> ActivationSpec:
    """Calibration activations: the rows of all samples stacked, 1 % outlier channels x 50."""
    return ActivationSpec(f"calib-{rows}x{d}", rows, d, seed,
                          outlier_channels=max(1, round(0.01 * d)), outlier_gain=50.0)


def tiny_spec() -> ActivationSpec:
    return ActivationSpec("tiny", 256, 1152, seed=0, outlier_channels=12,
                          outlier_gain=50.0, spike_rows=4, spike_gain=8.0)


def pixart_specs() -> list[ActivationSpec]:
    return [
        ActivationSpec("pixart_attn_in", 8192, 1152, seed=1,
                       outlier_channels=round(0.01 * 1152), outlier_gain=50.0),
        ActivationSpec("pixart_fc2_in", 8192, 4608, seed=1,
                       outlier_channels=round(0.01 * 4608), outlier_gain=50.0, gelu=True),
    ]


def sana_specs() -> list[ActivationSpec]:
    return [
        ActivationSpec("sana_2240", 4096, 2240, seed=2, outlier_channels=22,
                       outlier_gain=50.0, spike_rows=4, spike_gain=8.0),
        ActivationSpec("sana_5600", 4096, 5600, seed=2, outlier_channels=56,
                       outlier_gain=50.0, spike_rows=4, spike_gain=8.0),
    ]


def flux_specs() -> list[ActivationSpec]:
    # 4096 image tokens followed by 512 text tokens whose variance is 4x larger.
    return [
        ActivationSpec("flux_3072", 4608, 3072, seed=3, outlier_channels=15,
                       outlier_gain=100.0, tail_rows=512, tail_gain=2.0),
        ActivationSpec("flux_12288", 4608, 12288, seed=3, outlier_channels=61,
                       outlier_gain=100.0, tail_rows=512, tail_gain=2.0),
    ]


SWEEP_TOKENS = (1024, 4096, 16384, 65536)
SWEEP_D = (1152, 2240, 3072, 12288)


def sweep_spec(tokens: int, d: int) -> ActivationSpec:
    return ActivationSpec(f"sweep_{tokens}x{d}", tokens, d, seed=4, outlier_channels=12,
                          outlier_gain=50.0, spike_rows=4, spike_gain=8.0)


ALGORITHMIC_BYTES_PER_ELEMENT = 2.0 + 0.5 + 1.0 / 32.0  # bf16 read + 4-bit code + scale byte / 32


def algorithmic_bytes(tokens: int, d: int) -> float:
    """Bytes one quantizer call must move: read X once, write codes and scales."""
    return tokens * d * ALGORITHMIC_BYTES_PER_ELEMENT


# --------------------------------------------------------------------------
# token sharding across ranks (no exchange step: token rows are independent)
# --------------------------------------------------------------------------
def shard_rows(tokens: int, world_size: int, rank: int) -> tuple[int, int]:
    """Contiguous [begin, end) token range of `rank`; sizes differ by at most 1."""
    if world_size <= 0 or not (0 <= rank < world_size):
        raise ValueError("bad rank/world_size")
    base, rem = divmod(tokens, world_size)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)
