"""Pins for the oracle's transform half (CPU only).

Each test checks the oracle against something other than itself: a library
Kronecker product, hand vectors, the Hadamard closed form, exact rational
arithmetic, or an algebraic identity the paper states.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import c_oracle as co
from oracle import np_oracle as no
from paper_2607_21446_b200 import workloads as W


def bits_of(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


# ---- Section 3.5 entry-wise formula vs the library Kronecker product ---------
@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_bit_formula_equals_np_kron_chain(seed):
    G = W.gen_factors(seed)[0]
    K_bits = co.dense_k(G)                      # prod_k G_k[r_{5-k}, c_{5-k}]
    K = G[0].astype(np.float64)
    for k in range(1, 5):
        K = np.kron(K, G[k].astype(np.float64))  # G1 (x) G2 (x) ... (x) G5
    assert np.allclose(K_bits, K, rtol=1e-15, atol=0)


# ---- convention: y = x K (row vector), G1 <-> bit 4, G5 <-> bit 0 -----------
def _shear_set(which):
    G = W.identity_factors(1)
    G[0, which] = np.array([[1, 2], [0, 1]], np.float32)
    return G


def test_convention_G1_acts_on_msb():
    x = np.arange(32, dtype=np.float32)[None, :]
    y = co.transform(bits_of(x), _shear_set(0))[0]
    # K = [[1,2],[0,1]] (x) I16 :  y[i] = x[i], y[16+i] = x[16+i] + 2 x[i]
    expect = x[0].copy()
    expect[16:] += 2 * x[0, :16]
    assert np.array_equal(y, expect)
    assert list(y[16:19]) == [16.0, 19.0, 22.0]


def test_convention_G5_acts_on_lsb():
    x = np.arange(32, dtype=np.float32)[None, :]
    y = co.transform(bits_of(x), _shear_set(4))[0]
    # K = I16 (x) [[1,2],[0,1]] :  y[2i] = x[2i], y[2i+1] = x[2i+1] + 2 x[2i]
    assert list(y[:6]) == [0.0, 1.0, 2.0, 7.0, 4.0, 13.0]
    expect = x[0].copy()
    expect[1::2] += 2 * x[0, 0::2]
    assert np.array_equal(y, expect)


def test_transposed_operand_would_fail():
    # x K and x K^T differ for a shear; guards against a transposed K.
    x = np.zeros((1, 32), np.float32)
    x[0, 0] = 1.0
    y = co.transform(bits_of(x), _shear_set(4))[0]
    # row 0 of K = e0 + 2 e1
    assert y[0] == 1.0 and y[1] == 2.0 and not y[2:].any()


# ---- Section 3.2: LU parametrisation and Hadamard initialisation -------------
def test_lu_formula_and_unit_determinant():
    abc = W.gen_lu_params(7, n_sets=3)
    G = co.lu_to_factors(abc)
    a, b, c = (abc[..., i].astype(np.float64) for i in range(3))
    assert np.allclose(G[..., 0, 0], a, rtol=1e-7)
    assert np.allclose(G[..., 0, 1], b, rtol=1e-7)
    assert np.allclose(G[..., 1, 0], a * c, rtol=1e-6)
    assert np.allclose(G[..., 1, 1], b * c - 1 / a, rtol=1e-6, atol=1e-7)
    det = np.linalg.det(G.astype(np.float64))
    assert np.allclose(det, -1.0, atol=1e-5)
    assert np.allclose(G, no.lu_to_factors(abc), rtol=1e-6, atol=1e-7)
    for s in range(3):
        sign, logdet = np.linalg.slogdet(co.dense_k(G[s]))
        assert abs(logdet) < 1e-4          # |det K| = 1


def test_hadamard_closed_form():
    G = co.lu_to_factors(W.hadamard_lu_params(1))
    K = co.dense_k(G[0])
    r = np.arange(32)
    pop = np.array([[bin(a & b).count("1") for b in r] for a in r])
    H = (-1.0) ** pop / np.sqrt(32.0)
    assert np.allclose(K, H, atol=2e-7)
    assert np.allclose(K @ K, np.eye(32), atol=1e-6)
    y = co.transform(bits_of(np.ones((1, 32))), G)[0]
    assert abs(y[0] - np.sqrt(32.0)) < 1e-5 and np.abs(y[1:]).max() < 1e-6


# ---- Section 3.2: inverse = Kronecker product of the 2x2 inverses -----------
@pytest.mark.parametrize("seed", [0, 5, 9])
def test_inverse_and_round_trip(seed):
    G = W.gen_factors(seed)
    K = co.dense_k(G[0])
    Kinv = co.dense_kinv(G[0])
    assert np.allclose(K @ Kinv, np.eye(32), atol=1e-12 * np.linalg.cond(K))
    assert np.allclose(Kinv, np.linalg.inv(K), rtol=1e-9, atol=1e-12)
    spec = W.ActivationSpec("rt", 64, 256, seed=seed, outlier_channels=3, outlier_gain=50.0)
    Xb = W.gen_activations(spec)
    x = W.bf16_bits_to_f32(Xb).astype(np.float64)
    Y = co.transform(Xb, G).astype(np.float64)          # float-rounded y
    back = (Y.reshape(64, 8, 32) @ Kinv).reshape(64, 256)
    scale = np.abs(x.reshape(64, 8, 32)).max(axis=2, keepdims=True).repeat(32, 2).reshape(64, 256)
    assert (np.abs(back - x) <= 1e-5 * scale).all()


# ---- identity factors reduce to the bare quantizer ---------------------------
def test_identity_factors_reduce_to_plain():
    Xb = W.gen_activations(W.ActivationSpec("id", 32, 128, seed=11, outlier_channels=2,
                                            outlier_gain=50.0))
    G = W.identity_factors(1)
    assert np.array_equal(co.transform(Xb, G), co.widen(Xb))
    q1, s1, _ = co.quantize(Xb, G)
    q2, s2, _ = co.plain_quantize(Xb)
    assert np.array_equal(q1, q2) and np.array_equal(s1, s2)
    assert np.array_equal(co.widen(Xb), W.bf16_bits_to_f32(Xb))


# ---- exact rational brute force on a tiny input ------------------------------
def test_transform_against_exact_rationals():
    rng = np.random.default_rng(3)
    Xb = bits_of(rng.standard_normal((2, 64)) * 3)
    G = W.gen_factors(21, n_sets=2)
    Y = co.transform(Xb, G)
    x = W.bf16_bits_to_f32(Xb)
    for t in range(2):
        for j in range(2):
            g = [[[Fraction(float(G[j, k, a, b])) for b in range(2)] for a in range(2)]
                 for k in range(5)]
            for c in range(32):
                acc = Fraction(0)
                for r in range(32):
                    p = Fraction(float(x[t, 32 * j + r]))
                    for k in range(5):
                        p *= g[k][(r >> (4 - k)) & 1][(c >> (4 - k)) & 1]
                    acc += p
                exact = float(acc)                       # correctly rounded double
                got = float(Y[t, 32 * j + c])
                # oracle = float(double sum): within one float ulp of the exact value
                ulp = np.spacing(np.float32(abs(exact))) if exact else 1e-45
                assert abs(got - exact) <= ulp, (t, j, c, got, exact)


# ---- regroupings: pair form and five-stage butterfly equal the dense product --
def test_pair_form_and_butterfly_equal_dense():
    G = W.gen_factors(4)[0].astype(np.float64)
    K = co.dense_k(G.astype(np.float32))
    P = np.kron(G[0], G[1])                     # 4x4 on bits 4,3
    Q = np.kron(np.kron(G[2], G[3]), G[4])      # 8x8 on bits 2,1,0
    rng = np.random.default_rng(0)
    x = rng.standard_normal(32)
    dense = x @ K
    pair = (P.T @ x.reshape(4, 8) @ Q).reshape(32)
    assert np.allclose(pair, dense, rtol=1e-12, atol=1e-13)
    v = x.copy()
    for k in range(5):                           # stage k mixes index bit 4-k
        bit = 4 - k
        w = np.empty_like(v)
        for i in range(32):
            lo, hi = i & ~(1 << bit), i | (1 << bit)
            cb = (i >> bit) & 1
            w[i] = v[lo] * G[k][0][cb] + v[hi] * G[k][1][cb]
        v = w
    assert np.allclose(v, dense, rtol=1e-12, atol=1e-13)


# ---- per-block factor sets: block j uses set j -------------------------------
def test_per_block_sets_are_indexed_by_block():
    nb = 5
    G = W.identity_factors(nb)
    for j in range(nb):
        G[j, 0] *= np.float32(j + 1)            # K_j = (j+1) I
    x = np.ones((3, nb * 32), np.float32)
    Y = co.transform(bits_of(x), G)
    expect = np.repeat(np.arange(1, nb + 1, dtype=np.float32), 32)[None, :].repeat(3, 0)
    assert np.array_equal(Y, expect)
    with pytest.raises(ValueError):
        co.transform(bits_of(x), G[:3])          # n_sets must be 1 or d/32
    with pytest.raises(ValueError):
        co.transform(bits_of(np.ones((1, 48))), W.identity_factors(1))


def test_shared_set_equals_replicated_per_block_sets():
    Xb = W.gen_activations(W.ActivationSpec("rep", 16, 160, seed=2, outlier_channels=2,
                                            outlier_gain=50.0))
    G = W.gen_factors(2)
    assert np.array_equal(co.transform(Xb, G), co.transform(Xb, np.repeat(G, 5, axis=0)))


# ---- linearity in x (power-of-two scaling is exact) ---------------------------
def test_power_of_two_scaling_is_exact():
    Xb = W.gen_activations(W.ActivationSpec("p2", 8, 64, seed=5, outlier_channels=1,
                                            outlier_gain=50.0))
    G = W.gen_factors(5)
    x = W.bf16_bits_to_f32(Xb)
    Y1 = co.transform(Xb, G)
    Y2 = co.transform(bits_of(x * 8.0), G)
    assert np.array_equal(Y2, Y1 * np.float32(8.0))


# ---- the two oracle implementations agree bit for bit -------------------------
def test_c_and_numpy_oracles_agree_on_tiny():
    Xb = W.gen_activations(W.tiny_spec())
    G = W.gen_factors(0)
    q, s, Y = co.quantize(Xb, G)
    q2, s2, Y2 = no.quantize(Xb, G)
    assert np.array_equal(Y, Y2)
    assert np.array_equal(q, q2) and np.array_equal(s, s2)
    assert q.shape == (256, 576) and s.shape == (256, 36)
    # per-block factors on a smaller tensor
    Xs = Xb[:32, :320]
    Gb = W.gen_factors(0, n_sets=10)
    qa, sa, Ya = co.quantize(Xs, Gb)
    qb, sb, Yb = no.quantize(Xs, Gb)
    assert np.array_equal(Ya, Yb) and np.array_equal(qa, qb) and np.array_equal(sa, sb)
    # scale path
    sv = W.gen_channel_scales(0, 320)
    assert np.array_equal(co.scale_transform(Xs, sv), no.scale_transform(Xs, sv))
