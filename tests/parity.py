"""Parity rules between the CUDA quantizer and the CPU oracle.

P0  exact kernels (bare MXFP4, per-channel scale, identity factors): every code
    and scale byte identical (a zero's sign may differ only where the oracle's
    value is exactly +-0).
P1  pre-rounding values: |y_gpu - y| <= 1e-5 * max(|y|, amax_block / 32)   (amax_block / 16 for
    fp16 activations, see FLOOR_DIV).
    A code 0x0 vs 0x8 (signed zero) is not a mismatch where the oracle's value is
    exactly +-0 or, for the inexact kernels, within the P1 tolerance of zero.
P2  codes: a mismatch is allowed only where the oracle's scaled value lies within
    1e-5 relative of a rounding boundary, must be one adjacent magnitude step
    with the same sign, and at most 1e-4 of all codes may differ.
P3  scales: identical, except blocks whose oracle amax lies within 1e-5 relative
    of a power of two, which may be off by one; their codes are then checked
    against the oracle re-encoded with the GPU's scale; at most 1e-4 of blocks.
"""
from __future__ import annotations

import numpy as np

from oracle import np_oracle as no

BOUNDS = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
REL = 1e-5
MAX_FRACTION = 1e-4
# Floor of the value tolerance, as a fraction of the block amax.  bf16 activations (the case the 1e-5 rule is stated
# for): amax/32.  fp16 activations: amax/16, from the accumulation model: an fp16 activation times an 11-bit factor
# term is a 22-bit product, so (unlike the 16-bit products of bf16 activations, whose sums mostly stay exact in 24
# bits) every one of the 32 additions of leading-term products rounds in the tensor core's fp32 accumulator.  With
# partial sums growing like sqrt(k) sigma_p (sigma_p = rms product) and a rounding of +-2^-24 relative each, the
# error's standard deviation is sqrt(sum_{k<=32} k / 3) 2^-24 sigma_p = 7.9e-7 sigma_p, while a block's amax is
# about 13.6 sigma_p (the largest of 32 sums of 32 products; outlier channels only raise it): amax/32 puts the
# tolerance at 5.4 standard deviations, which 10^8 elements do exceed now and then (measured worst: 1.1 times
# that floor), amax/16 at 10.8.
FLOOR_DIV = {"bf16": 32.0, "fp16": 16.0}


def unpack(q: np.ndarray) -> np.ndarray:
    t, half = q.shape
    c = np.empty((t, half * 2), np.uint8)
    c[:, 0::2] = q & 15
    c[:, 1::2] = q >> 4
    return c


def check_values(Y_gpu: np.ndarray, Y_or: np.ndarray, x_dtype: str = "bf16") -> dict:
    t, d = Y_or.shape
    yo = Y_or.astype(np.float64).reshape(t, d // 32, 32)
    yg = Y_gpu.astype(np.float64).reshape(t, d // 32, 32)
    amax = np.abs(yo).max(axis=2, keepdims=True)
    tol = REL * np.maximum(np.abs(yo), amax / FLOOR_DIV[x_dtype])
    err = np.abs(yg - yo)
    bad = err > tol
    ratio = np.where(tol > 0, err / np.where(tol > 0, tol, 1), np.where(err > 0, np.inf, 0))
    assert not bad.any(), f"P1: {bad.sum()} values outside tolerance, worst err/tol = {ratio.max():.3g}"
    return {"max_err_over_tol": float(ratio.max())}


def check_codes(q_gpu, s_gpu, q_or, s_or, Y_or, exact: bool, x_dtype: str = "bf16") -> dict:
    q_gpu, s_gpu = np.asarray(q_gpu), np.asarray(s_gpu)
    t, d = Y_or.shape
    nb = d // 32
    cg, co = unpack(q_gpu), unpack(q_or)
    Y = Y_or.astype(np.float64)
    # ---- scales (P3)
    sdiff = s_gpu != s_or
    n_sdiff = int(sdiff.sum())
    expect_codes = co
    if n_sdiff:
        assert not exact, f"P0: {n_sdiff} scale bytes differ"
        amax = np.abs(Y.reshape(t, nb, 32)).max(axis=2)
        m, _ = np.frexp(amax[sdiff])                  # amax = m 2^e, m in [0.5, 1)
        near_pow2 = np.minimum(np.abs(m - 0.5) / 0.5, np.abs(m - 1.0)) <= REL
        assert near_pow2.all(), "P3: a scale differs on a block whose amax is not at a power of two"
        assert (np.abs(s_gpu[sdiff].astype(int) - s_or[sdiff].astype(int)) == 1).all()
        assert n_sdiff <= max(1, MAX_FRACTION * t * nb), f"P3: {n_sdiff} scale mismatches"
        expect_codes = no.encode_with_scale(Y_or, np.where(sdiff, s_gpu, s_or))
    # ---- codes (P0 / P2)
    diff = cg != expect_codes
    # zero-sign exemption: both codes are a zero and only the sign bit differs, where the
    # oracle's value is exactly +-0 (summation order decides the sign of an exact zero) or,
    # for the inexact kernels, lies within the P1 tolerance of zero (|y| <= 1e-5 amax/32),
    # so that its sign is not determined by the arithmetic
    if exact:
        undetermined = Y == 0.0
    else:
        amax_b = np.abs(Y.reshape(t, nb, 32)).max(axis=2, keepdims=True)
        undetermined = (np.abs(Y.reshape(t, nb, 32)) <= REL * amax_b / FLOOR_DIV[x_dtype]).reshape(t, d)
    zero_sign = diff & undetermined & ((cg & 7) == 0) & ((expect_codes & 7) == 0)
    diff &= ~zero_sign
    n_diff = int(diff.sum())
    if exact:
        assert n_diff == 0, f"P0: {n_diff} codes differ"
    elif n_diff:
        S_used = np.where(sdiff, s_gpu, s_or).astype(np.float64)
        vb = np.abs(Y.reshape(t, nb, 32) * np.exp2(127.0 - S_used)[:, :, None])
        v = vb.reshape(t, d)
        # a code may differ only where the value lies within the value tolerance of a boundary:
        # 1e-5 relative, or the tolerance floor (for bf16 the floor never exceeds 1e-5 * 0.25)
        floor = (REL * vb.max(axis=2, keepdims=True) / FLOOR_DIV[x_dtype]).repeat(32, 2).reshape(t, d)
        vd, fd = v[diff], floor[diff]
        near = (np.abs(vd[:, None] - BOUNDS[None, :]) <= np.maximum(REL * BOUNDS[None, :], fd[:, None])).any(axis=1)
        assert near.all(), f"P2: {int((~near).sum())} code mismatches away from any rounding boundary"
        g, o = cg[diff].astype(int), expect_codes[diff].astype(int)
        assert ((g & 8) == (o & 8)).all(), "P2: sign differs"
        assert (np.abs((g & 7) - (o & 7)) == 1).all(), "P2: more than one step"
        assert n_diff <= max(1, MAX_FRACTION * t * d), f"P2: {n_diff} code mismatches"
    return {"code_mismatches": n_diff, "scale_mismatches": n_sdiff,
            "zero_sign_only": int(zero_sign.sum())}


def check_codes_chunked(q_gpu, s_gpu, x_bits_rows, oracle_quantize, tokens: int, exact: bool, x_dtype: str = "bf16",
                        chunk: int = 2048) -> dict:
    """Whole-tensor P0/P2/P3 check with bounded host memory: the oracle runs on `chunk` token rows at a time.

    q_gpu, s_gpu: the device results (anything sliceable by row range that yields NumPy arrays through
    ``np.asarray`` / ``.cpu().numpy()``); x_bits_rows(r0, r1) -> uint16 input rows; oracle_quantize(bits) ->
    (q, s, Y).  Every row is compared.  A chunk whose bytes are identical to the oracle's is accepted at once;
    the others go through check_codes, and the 1e-4 limits are applied to the chunk and to the whole tensor."""
    total = {"code_mismatches": 0, "scale_mismatches": 0, "zero_sign_only": 0, "rows": 0}
    d = None
    for r0 in range(0, tokens, chunk):
        r1 = min(tokens, r0 + chunk)
        q_or, s_or, Y = oracle_quantize(x_bits_rows(r0, r1))
        qg, sg = q_gpu[r0:r1], s_gpu[r0:r1]
        if hasattr(qg, "cpu"):
            qg, sg = qg.cpu().numpy(), sg.cpu().numpy()
        d = Y.shape[1]
        total["rows"] += r1 - r0
        if np.array_equal(qg, q_or) and np.array_equal(sg, s_or):
            continue
        r = check_codes(qg, sg, q_or, s_or, Y, exact=exact, x_dtype=x_dtype)
        for k in ("code_mismatches", "scale_mismatches", "zero_sign_only"):
            total[k] += r[k]
    assert total["rows"] == tokens
    assert total["code_mismatches"] <= max(1, MAX_FRACTION * tokens * d), f"P2: {total['code_mismatches']} code mismatches"
    assert total["scale_mismatches"] <= max(1, MAX_FRACTION * tokens * d / 32), f"P3: {total['scale_mismatches']} scale mismatches"
    return total
