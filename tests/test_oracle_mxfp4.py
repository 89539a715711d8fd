"""Pins for the oracle's MXFP4 half (CPU only): hand-worked encodings, brute
force over every bf16 value in (-8, 8), invariants and degenerate blocks."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import c_oracle as co
from oracle import np_oracle as no
from paper_2607_21446_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "mxfp4_handworked.txt")
GRID = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3),
        Fraction(4), Fraction(6)]


def block32(vals):
    y = np.zeros(32, np.float32)
    y[:len(vals)] = np.asarray(vals, dtype=np.float32)
    return y


def codes_of(q16):
    out = []
    for b in q16:
        out += [int(b) & 15, int(b) >> 4]
    return out


# ---- hand-worked fixtures -----------------------------------------------------
def _golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, vals, S, codes, byts = [p.strip() for p in line.split("|")]
            rows.append((name, [float(v) for v in vals.split()], int(S),
                         [int(c, 16) for c in codes.split()],
                         [int(b, 16) for b in byts.split()]))
    return rows


@pytest.mark.parametrize("row", _golden_rows(), ids=lambda r: r[0])
def test_handworked_blocks(row):
    name, vals, S, codes, byts = row
    q, s = co.encode_block(block32(vals))
    assert s == S
    assert codes_of(q)[:len(codes)] == codes
    assert list(q[:len(byts)]) == byts
    assert not q[(len(vals) + 1) // 2:].any()          # trailing zeros -> code 0
    # the NumPy twin reproduces the same fixture
    q2, s2 = no.mx_encode(block32(vals)[None, :])
    assert list(q2[0]) == list(q) and int(s2[0, 0]) == S


# ---- brute force: nearest of the 16 signed grid values, ties to even code -----
def brute_code(v: float) -> int:
    """Nearest signed E2M1 value by absolute difference (exact rationals), ties to
    the even code, values beyond +-6 saturate; the sign bit follows the input."""
    fv = Fraction(v)
    av = abs(fv)
    best = min(abs(av - g) for g in GRID)
    cands = [i for i, g in enumerate(GRID) if abs(av - g) == best]
    even = [i for i in cands if i % 2 == 0]
    mag = even[0] if even else cands[0]
    sign = 8 if np.signbit(np.float32(v)) else 0
    return sign | mag


def all_bf16_in_open_8():
    bits = np.arange(0, 1 << 16, dtype=np.uint32).astype(np.uint16)
    vals = W.bf16_bits_to_f32(bits)
    ok = np.isfinite(vals) & (np.abs(vals) < 8.0)
    return vals[ok]


def test_e2m1_rounding_brute_force_all_bf16():
    vals = all_bf16_in_open_8()
    # add the 7 rounding boundaries and their float neighbours, both signs
    extra = []
    for b in (0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0):
        f = np.float32(b)
        for s in (1.0, -1.0):
            extra += [s * f, s * np.nextafter(f, np.float32(0)), s * np.nextafter(f, np.float32(9))]
    vals = np.concatenate([vals, np.asarray(extra, np.float32)])
    # anchor element 4.0 keeps amax in [4, 8) -> S = 127 -> scaled value = value
    Y = np.zeros((len(vals), 32), np.float32)
    Y[:, 0] = vals
    Y[:, 1] = 4.0
    q, s = co.mx_encode(Y)
    assert (s == 127).all()
    got = q[:, 0] & 15
    expect = np.array([brute_code(float(v)) for v in vals], dtype=np.uint8)
    assert np.array_equal(got, expect)
    assert ((q[:, 0] >> 4) == 6).all()                 # the anchor itself: 4.0 -> code 6
    qn, sn = no.mx_encode(Y)
    assert np.array_equal(qn, q) and np.array_equal(sn, s)


def test_tie_table_explicit():
    # ties go to the even code: .25->0, .75->1.0, 1.25->1.0, 1.75->2.0, 2.5->2.0, 3.5->4.0, 5->4.0
    ties = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]
    codes = [0, 2, 2, 4, 4, 6, 6]
    for v, c in zip(ties, codes):
        q, s = co.encode_block(block32([v, 4.0]))
        assert s == 127 and (q[0] & 15) == c
        q, s = co.encode_block(block32([-v, 4.0]))
        assert (q[0] & 15) == (8 | c)


# ---- scale byte ------------------------------------------------------------------
@pytest.mark.parametrize("e", [-126, -60, -3, 0, 1, 2, 3, 64, 127])
def test_scale_byte_is_biased_exponent_minus_two(e):
    for m in (1.0, 1.5, 1.9999999):
        amax = np.float32(np.ldexp(np.float32(m), e))
        q, s = co.encode_block(block32([amax]))
        assert s == max(e - 2 + 127, 0)
        # v = amax * 2^(127-S) lies in [4, 8) unless the clamp at 0 was hit
        if e - 2 + 127 >= 0:
            v = float(amax) * 2.0 ** (127 - s)
            assert 4.0 <= v < 8.0
            assert (q[0] & 15) == brute_code(v)


def test_degenerate_blocks():
    q, s = co.encode_block(np.zeros(32, np.float32))
    assert s == 0 and not q.any()
    q, s = co.encode_block(np.full(32, -0.0, np.float32))
    assert s == 0 and (q == 0x88).all()                 # sign of zero is kept
    tiny = np.float32(1e-45)                             # smallest subnormal
    q, s = co.encode_block(block32([tiny, -tiny]))
    assert s == 0 and (q[0] & 15) == 0 and (q[0] >> 4) == 8
    big = np.float32(3.0e38)                             # exponent 127 -> S = 252
    q, s = co.encode_block(block32([big, -big / 2]))
    assert s == 252
    v = float(big) * 2.0 ** (127 - 252)
    assert (q[0] & 15) == brute_code(v) and (q[0] >> 4) == brute_code(-v / 2)
    # subnormal amax below 2^-125 clamps the byte at 0 and scales by 2^127
    sub = np.float32(np.ldexp(1.0, -130))
    q, s = co.encode_block(block32([sub]))
    assert s == 0 and (q[0] & 15) == brute_code(float(sub) * 2.0 ** 127)


# ---- invariants ----------------------------------------------------------------------
@pytest.fixture(scope="module")
def small():
    spec = W.ActivationSpec("inv", 96, 256, seed=17, outlier_channels=3, outlier_gain=50.0,
                            spike_rows=2, spike_gain=8.0)
    Xb = W.gen_activations(spec)
    G = W.gen_factors(17)
    return Xb, G


def test_power_of_two_equivariance(small):
    Xb, G = small
    x = W.bf16_bits_to_f32(Xb)
    q, s, _ = co.quantize(Xb, G)
    for k in (-7, 3, 20):
        q2, s2, _ = co.quantize(W.f32_to_bf16_bits(x * np.float32(2.0 ** k)), G)
        assert np.array_equal(q2, q)
        assert np.array_equal(s2.astype(int), s.astype(int) + k)


def test_negation_flips_only_sign_bits(small):
    Xb, G = small
    q, s, _ = co.quantize(Xb, G)
    qn, sn, _ = co.quantize(Xb ^ np.uint16(0x8000), G)
    assert np.array_equal(sn, s)
    assert np.array_equal(qn, q ^ np.uint8(0x88))


def test_idempotence_with_identity(small):
    Xb, _ = small
    q, s, _ = co.plain_quantize(Xb)
    dec = co.dequantize(q, s)                                  # exact floats
    q2, s2 = co.mx_encode(dec)
    assert np.array_equal(q2, q) and np.array_equal(s2, s)


def test_scaled_amax_in_4_8_and_half_step_bound(small):
    Xb, G = small
    q, s, Y = co.quantize(Xb, G)
    yb = Y.reshape(96, 8, 32).astype(np.float64)
    sc = np.exp2(127.0 - s.astype(np.float64))[:, :, None]
    v = yb * sc
    amax = np.abs(v).max(axis=2)
    assert ((amax >= 4) & (amax < 8)).all()
    dec = no.decode(q, s) * sc                                  # decoded, scaled domain
    err = np.abs(v - dec)
    av = np.abs(v)
    step = np.where(av < 2, 0.5, np.where(av < 4, 1.0, 2.0))
    unsat = av <= 6
    assert (err[unsat] <= step[unsat] / 2).all()
    assert (np.abs(dec[~unsat]) == 6).all()


def test_row_permutation_equivariance(small):
    Xb, G = small
    perm = np.random.default_rng(0).permutation(Xb.shape[0])
    q, s, _ = co.quantize(Xb, G)
    qp, sp, _ = co.quantize(Xb[perm], G)
    assert np.array_equal(qp, q[perm]) and np.array_equal(sp, s[perm])


# ---- decode -----------------------------------------------------------------------------
def test_dequantize_without_factors_is_exact_decode(small):
    Xb, G = small
    q, s, _ = co.quantize(Xb, G)
    dec = co.dequantize(q, s)
    assert np.array_equal(dec.astype(np.float64), no.decode(q, s).reshape(dec.shape))
    # all 16 codes at a few scales, against the grid written out
    codes = np.arange(16, dtype=np.uint8)
    qq = (codes[0::2] | (codes[1::2] << 4))[None, :].repeat(2, 0)
    qq = np.concatenate([qq, np.zeros((2, 8), np.uint8)], axis=1)
    ss = np.array([[127], [120]], np.uint8)
    out = co.dequantize(qq, ss)
    grid = np.array([0, .5, 1, 1.5, 2, 3, 4, 6, -0.0, -.5, -1, -1.5, -2, -3, -4, -6], np.float32)
    assert np.array_equal(out[0, :16], grid)
    assert np.array_equal(out[1, :16], grid * np.float32(2.0 ** -7))
    assert np.signbit(out[0, 8])


def test_dequantize_with_factors_inverts_transform(small):
    Xb, G = small
    q, s, Y = co.quantize(Xb, G)
    back = co.dequantize(q, s, G)
    # equals (decoded y) @ K^-1 computed with the library inverse
    Kinv = np.linalg.inv(co.dense_k(G[0]))
    ref = (no.decode(q, s) @ Kinv).reshape(back.shape)
    assert np.allclose(back, ref, rtol=1e-6, atol=1e-6 * np.abs(ref).max())
    # identity factors: same as no factors
    qi, si, _ = co.plain_quantize(Xb)
    assert np.array_equal(co.dequantize(qi, si, W.identity_factors(1)), co.dequantize(qi, si))
    # reconstruction error is bounded by the quantization step times ||K^-1||
    x = W.bf16_bits_to_f32(Xb).astype(np.float64)
    rel = np.linalg.norm(back - x) / np.linalg.norm(x)
    assert rel < 0.25


def test_dequantize_bf16_rounding_matches_torch(small):
    Xb, G = small
    q, s, _ = co.quantize(Xb, G)
    f = co.dequantize(q, s, G)
    b = co.dequantize(q, s, G, out_bf16=True)
    # float -> bf16 by the library's RNE cast; differs from single rounding of the
    # double only on float-level ties, which these data do not hit
    tb = torch.from_numpy(f.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (tb != b).mean() < 1e-3
    assert np.abs(W.bf16_bits_to_f32(b) - f).max() <= np.abs(f).max() * 2.0 ** -8
    # without factors every decoded value is exactly representable in bf16
    b0 = co.dequantize(q, s, None, out_bf16=True)
    assert np.array_equal(W.bf16_bits_to_f32(b0), co.dequantize(q, s))


# ---- codes under an imposed scale byte (the helper of parity rule P3) ----------------------
IMPOSED = os.path.join(os.path.dirname(__file__), "golden", "mxfp4_imposed_scale.txt")


def _imposed_rows():
    rows = []
    with open(IMPOSED) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, vals, S, codes = [p.strip() for p in line.split("|")]
            rows.append((name, [float(v) for v in vals.split()], int(S), [int(c, 16) for c in codes.split()]))
    return rows


@pytest.mark.parametrize("row", _imposed_rows(), ids=lambda r: r[0])
def test_encode_with_scale_handworked(row):
    name, vals, S, codes = row
    got = no.encode_with_scale(block32(vals)[None, :], np.array([[S]], np.uint8))
    assert list(got[0, :len(codes)]) == codes
    assert not got[0, len(vals):].any()


def test_encode_with_scale_at_own_scale_is_the_encoder(small):
    # with S = the block's own scale byte it must reproduce the C oracle's encoder on whole tensors
    Xb, G = small
    q, s, Y = co.quantize(Xb, G)
    codes = np.empty(Y.shape, np.uint8)
    codes[:, 0::2] = q & 15
    codes[:, 1::2] = q >> 4
    assert np.array_equal(no.encode_with_scale(Y, s), codes)
    spec = W.tiny_spec()
    Xt = W.gen_activations(spec)
    qt, st, Yt = co.quantize(Xt, W.gen_factors(0))
    ct = np.empty(Yt.shape, np.uint8)
    ct[:, 0::2] = qt & 15
    ct[:, 1::2] = qt >> 4
    assert np.array_equal(no.encode_with_scale(Yt, st), ct)


def test_encode_with_scale_brute_force_neighbouring_scales():
    # every bf16 value in (-8, 8) at S = 126, 127, 128 against the exact-rational nearest-code search
    vals = all_bf16_in_open_8()
    Y = np.zeros((len(vals), 32), np.float32)
    Y[:, 0] = vals
    for S in (126, 127, 128):
        got = no.encode_with_scale(Y, np.full((len(vals), 1), S, np.uint8))[:, 0]
        expect = np.array([brute_code(float(v) * 2.0 ** (127 - S)) for v in vals], dtype=np.uint8)
        assert np.array_equal(got, expect)
