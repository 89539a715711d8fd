"""Pins for the oracle's fp16-input and dense-block variants (CPU only)."""
import numpy as np
import pytest

from oracle import c_oracle as co
from paper_2607_21446_b200 import workloads as W


def kron_chain(G1):
    K = G1[0].astype(np.float64)
    for k in range(1, 5):
        K = np.kron(K, G1[k].astype(np.float64))
    return K


def test_fp16_widening_matches_numpy_for_every_finite_pattern():
    bits = np.arange(0, 1 << 16, dtype=np.uint32).astype(np.uint16)
    ref = bits.view(np.float16).astype(np.float32)           # library conversion
    fin = np.isfinite(ref)
    pad = (-fin.sum()) % 32
    b = np.concatenate([bits[fin], np.zeros(pad, np.uint16)]).reshape(-1, 32)
    got = co.widen(b, x_dtype="fp16").reshape(-1)[:fin.sum()]
    assert np.array_equal(got.view(np.uint32), ref[fin].view(np.uint32))   # also the sign of zero


def test_fp16_and_bf16_inputs_agree_on_values_both_formats_hold():
    # values with <= 8 significant bits and small exponents are exact in both formats
    rng = np.random.default_rng(0)
    x = (rng.integers(-255, 256, size=(16, 128)) * 2.0 ** rng.integers(-6, 3, size=(16, 128))).astype(np.float32)
    G = W.gen_factors(3)
    a = co.quantize(W.f32_to_bf16_bits(x), G, x_dtype="bf16")
    b = co.quantize(W.f32_to_fp16_bits(x), G, x_dtype="fp16")
    for u, v in zip(a, b):
        assert np.array_equal(u, v)


def test_dense_blocks_equal_factor_path_when_the_product_is_exact_in_float():
    # dyadic factor entries: every K entry is exactly representable in float32
    rng = np.random.default_rng(5)
    G = (rng.integers(-3, 4, size=(2, 5, 2, 2)) / 2.0).astype(np.float32)
    for s in range(2):
        for k in range(5):
            if abs(np.linalg.det(G[s, k])) < 0.2:
                G[s, k] = np.array([[1, 0.5], [-0.5, 1]], np.float32)
    Kd = np.stack([kron_chain(G[s]) for s in range(2)]).astype(np.float32)
    assert np.array_equal(Kd.astype(np.float64), np.stack([kron_chain(G[s]) for s in range(2)]))
    Xb = W.gen_activations(W.ActivationSpec("d", 8, 64, seed=1, outlier_channels=2, outlier_gain=50.0))
    assert np.array_equal(co.transform(Xb, G), co.transform(Xb, K_dense=Kd))


@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
def test_dense_transform_equals_library_matmul(dtype):
    Kd = W.gen_dense_blocks(7, n_sets=3)
    Xb = W.gen_activations(W.ActivationSpec("m", 24, 96, seed=7, outlier_channels=2, outlier_gain=50.0), dtype)
    x = (W.fp16_bits_to_f32(Xb) if dtype == "fp16" else W.bf16_bits_to_f32(Xb)).astype(np.float64)
    Y = co.transform(Xb, K_dense=Kd, x_dtype=dtype)
    ref = np.einsum("tjr,jrc->tjc", x.reshape(24, 3, 32), Kd.astype(np.float64)).reshape(24, 96)
    err = np.abs(Y.astype(np.float64) - ref)
    assert (err <= np.spacing(np.abs(ref).astype(np.float32)).astype(np.float64)).all()
    # shared dense block = the same block replicated
    assert np.array_equal(co.transform(Xb, K_dense=Kd[:1]), co.transform(Xb, K_dense=np.repeat(Kd[:1], 3, 0)))
    with pytest.raises(ValueError):
        co.transform(Xb, K_dense=Kd[:2])


def test_scale_and_plain_paths_with_fp16_input():
    Xb = W.gen_activations(W.ActivationSpec("s", 8, 64, seed=2, outlier_channels=1, outlier_gain=50.0), "fp16")
    x = W.fp16_bits_to_f32(Xb)
    sv = W.gen_channel_scales(2, 64)
    assert np.array_equal(co.widen(Xb, "fp16"), x)
    assert np.array_equal(co.scale_transform(Xb, sv, "fp16"),
                          (x.astype(np.float64) * sv.astype(np.float64)[None, :]).astype(np.float32))


# ---- tiled scale layout for block-scaled GEMM consumers --------------------------------------
def test_tiled_scale_layout_hand_indices():
    # 128 x 4 tiles of 512 bytes; inside a tile: (r % 32) * 16 + (r % 128 // 32) * 4 + j % 4
    kb = 9                                    # 3 column tiles per row tile
    assert co.tiled_scale_index(0, 0, kb) == 0
    assert co.tiled_scale_index(0, 1, kb) == 1
    assert co.tiled_scale_index(0, 3, kb) == 3
    assert co.tiled_scale_index(0, 4, kb) == 512             # next column tile
    assert co.tiled_scale_index(1, 0, kb) == 16
    assert co.tiled_scale_index(31, 0, kb) == 31 * 16
    assert co.tiled_scale_index(32, 0, kb) == 4               # second 32-row quarter
    assert co.tiled_scale_index(96, 2, kb) == 12 + 2
    assert co.tiled_scale_index(127, 3, kb) == 31 * 16 + 12 + 3 == 511
    assert co.tiled_scale_index(128, 0, kb) == 3 * 512        # next row tile
    assert co.tiled_scale_index(130, 8, kb) == 3 * 512 + 2 * 512 + 2 * 16


@pytest.mark.parametrize("rows,kb", [(1, 1), (128, 4), (130, 9), (257, 36), (300, 175)])
def test_tiled_scale_layout_equals_reshape_permute(rows, kb):
    """Independent statement with library reshapes: pad to [R*128, C*4], split into tiles
    [R, C, 128, 4], split the 128 rows into [4, 32] and store each tile as [32, 4, 4]."""
    rng = np.random.default_rng(rows + kb)
    s = rng.integers(1, 255, size=(rows, kb), dtype=np.uint8)
    got = co.scales_to_tiled(s, fill=0)
    R, Cb = (rows + 127) // 128, (kb + 3) // 4
    p = np.zeros((R * 128, Cb * 4), np.uint8)
    p[:rows, :kb] = s
    t = p.reshape(R, 128, Cb, 4).transpose(0, 2, 1, 3)          # [R, C, 128, 4]
    t = t.reshape(R, Cb, 4, 32, 4).transpose(0, 1, 3, 2, 4)      # [R, C, 32, 4, 4]
    assert np.array_equal(got, t.reshape(-1))
    # a bijection on the real entries: every (r, j) lands on a distinct byte
    idx = {co.tiled_scale_index(r, j, kb) for r in range(min(rows, 140)) for j in range(kb)}
    assert len(idx) == min(rows, 140) * kb


# ---- 16-bit copy of the transformed activations ---------------------------------------------------
def test_rounding_y_to_16_bits_matches_library_casts():
    import torch
    rng = np.random.default_rng(3)
    y = np.concatenate([
        (rng.standard_normal(20000) * np.exp(rng.uniform(-12, 8, 20000))).astype(np.float32),
        np.array([0.0, -0.0, 65504.0, 65519.9, 65520.0, -70000.0, 2.0 ** -24, 2.0 ** -25, 1.5 * 2.0 ** -25,
                  2.0 ** -14, 1.00048828125, 1.0009765625, 1.00146484375], np.float32)])
    # every float that is exactly half-way between two fp16 / bf16 neighbours around 1..2
    ties16 = (1.0 + (np.arange(0, 2048, 2) + 1) / 2048.0).astype(np.float32)
    tiesb = (1.0 + (np.arange(0, 256, 2) + 1) / 256.0).astype(np.float32)
    y = np.concatenate([y, ties16, tiesb, -ties16])
    got16 = co.round_y_to_16bit(y, "fp16")
    with np.errstate(over="ignore"):
        ref16 = y.astype(np.float16).view(np.uint16)                 # NumPy: round to nearest even
    assert np.array_equal(got16, ref16)
    gotb = co.round_y_to_16bit(y, "bf16")
    refb = torch.from_numpy(y.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(gotb, refb)


# ---- full-d Hadamard baseline -------------------------------------------------------------------------
@pytest.mark.parametrize("d", [32, 64, 256, 1024])
def test_hadamard_transform_against_scipy(d):
    from scipy.linalg import hadamard
    Xb = W.gen_activations(W.ActivationSpec("h", 5, d, seed=d, outlier_channels=2, outlier_gain=50.0))
    x = W.bf16_bits_to_f32(Xb).astype(np.float64)
    Y = co.hadamard_transform(Xb)
    ref = x @ (hadamard(d).astype(np.float64) / np.sqrt(d))            # Sylvester construction, library
    assert np.allclose(Y, ref, rtol=2e-7, atol=2e-7 * np.abs(ref).max())
    # orthogonal and symmetric: applying it twice gives x back
    back = Y.astype(np.float64) @ (hadamard(d) / np.sqrt(d))
    assert np.allclose(back, x, atol=1e-5 * np.abs(x).max())
    # d = 32 coincides with the block transform at the paper's Hadamard initialisation
    if d == 32:
        G = co.lu_to_factors(W.hadamard_lu_params(1))
        assert np.allclose(Y, co.transform(Xb, G), rtol=1e-6, atol=1e-6 * np.abs(Y).max())
    with pytest.raises(ValueError):
        co.hadamard_transform(np.zeros((1, 96), np.uint16))


def test_hadamard_constant_row_and_single_spike():
    d = 128
    ones = W.f32_to_bf16_bits(np.ones((1, d), np.float32))
    y = co.hadamard_transform(ones)[0]
    assert y[0] == np.float32(np.sqrt(d)) and not y[1:].any()
    spike = np.zeros((1, d), np.float32)
    spike[0, 5] = 3.0
    y = co.hadamard_transform(W.f32_to_bf16_bits(spike))[0]
    signs = np.array([(-1.0) ** bin(5 & c).count("1") for c in range(d)])
    assert np.array_equal(y, (3.0 * signs / np.sqrt(d)).astype(np.float32))
