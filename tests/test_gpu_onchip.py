"""The tensor-core quantizer with its operand built on chip from the factor scalars (path "onchip": Section 3.5,
the "K2" kernel; Appendix B; bf16 and fp16 activations) against the CPU oracle, and next to the path that copies ready-made operand images.

The operand itself is pinned through the transform output: unit-vector activations make row r of a block's output
the row K[r][:] that the kernel holds (three bf16 terms summed in the fp32 accumulator), which is compared with the
Kronecker product formed in float64 by the oracle -- a transposed or mis-swizzled image, a factor taken with the
wrong bit, or a lost low-order term all fail it."""
import numpy as np
import pytest
import torch

from oracle import c_oracle as co
from paper_2607_21446_b200 import workloads as W
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2607_21446_b200 import binding
    binding.load_library()
    return binding


def dev(bits, dtype="bf16"):
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.float16 if dtype == "fp16" else torch.bfloat16)


def spec(tokens, d, seed):
    return W.ActivationSpec(f"k2_{tokens}x{d}", tokens, d, seed=seed, outlier_channels=max(1, d // 100),
                            outlier_gain=50.0, spike_rows=min(2, tokens), spike_gain=8.0)


def untile(s_tiled, tokens, nb):
    """Row-major scale bytes out of the 128 x 4 tiled layout: the oracle's layout routine, run on the three bytes of
    every row-major index, says where each byte lives."""
    assert tokens * nb < 0xFFFFFF
    idx = np.arange(tokens * nb).reshape(tokens, nb)
    pos = sum(co.scales_to_tiled(((idx >> (8 * b)) & 255).astype(np.uint8), fill=255).astype(np.int64) << (8 * b) for b in range(3))
    live = pos != 0xFFFFFF                       # padding bytes carry the fill value in all three passes
    out = np.empty(tokens * nb, np.uint8)
    out[pos[live]] = s_tiled[: pos.size][live]
    return out.reshape(tokens, nb)


@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("n_sets", [1, 3, 36, 175])
def test_operand_built_on_chip_is_the_kronecker_product(B, n_sets, dtype):
    d = 32 * n_sets
    G = W.gen_factors(21 + n_sets, n_sets=n_sets)
    if dtype == "fp16":
        G[::2, 0] *= np.float32(2.0 ** 9)        # fp16 operands are normalised per set: make the sets' exponents differ
        G[1::3, 1] *= np.float32(2.0 ** -7)
    # token r carries the unit vector e_r in every block: Y[r, 32 j + c] = K_j[r][c]
    X = torch.zeros(32, d, dtype=torch.float16 if dtype == "fp16" else torch.bfloat16)
    for r in range(32):
        X[r, r::32] = 1.0
    f = B.Factors.create(G)
    Y = B.kroquant_transform_f32(X.cuda(), f, path="onchip").cpu().numpy().astype(np.float64)
    assert B.kroquant_last_device_error() == 0
    for j in range(n_sets):
        K = co.dense_k(G[j:j + 1]).reshape(32, 32)
        got = Y[:, 32 * j:32 * j + 32]
        # bf16: the three terms hold the leading 24 bits of every entry (8 + 8 + 8, each rounded to nearest: 2^-27
        # relative); what is read back is their sum in the tensor core's fp32 accumulator, which need not round to
        # nearest: one ulp.  fp16: terms of K 2^e (largest entry in [1, 2)) down to fp16's smallest step 2^-24, so a
        # small entry keeps an absolute 2^-25 of the set's largest; again one ulp of the accumulator on top
        tol = 2.0 ** -23 * np.abs(K)
        if dtype == "fp16":
            tol += 2.0 ** -25 * 2.0 ** np.floor(np.log2(np.abs(K).max()))
        assert np.all(np.abs(got - K) <= tol), (j, (np.abs(got - K) / tol).max())
    # and entry by entry it is the image path's operand up to that last bit
    Y_img = B.kroquant_transform_f32(X.cuda(), f, path="tensor").cpu().numpy().astype(np.float64)
    assert np.all(np.abs(Y - Y_img) <= 2.0 ** -22 * np.abs(Y_img) + (1e-7 * np.abs(Y_img).max() if dtype == "fp16" else 0))
    assert (Y == Y_img).mean() > 0.99


# ragged and multi-tile shapes, shared and per-block sets; 4608 x 3072 takes the large CTA shape, 1500 x 3072 and
# 700 x 5600 several tiles per CTA with a ragged last tile, 129 x 2240 a ragged column group
SHAPES = [(1, 32, False), (33, 1152, False), (1500, 3072, False), (4608, 3072, False),
          (1, 32, True), (3, 1152, True), (129, 2240, True), (700, 5600, True), (1200, 1152, True)]


@pytest.mark.parametrize("tokens,d,per_block", SHAPES)
@pytest.mark.parametrize("layout,dtype", [("rowmajor", "bf16"), ("tiled", "bf16"), ("rowmajor", "fp16")])
def test_onchip_path_against_the_oracle(B, tokens, d, per_block, layout, dtype):
    Xb = W.gen_activations(spec(tokens, d, 7 + tokens), dtype)
    G = W.gen_factors(13 + d, n_sets=d // 32 if per_block else 1)
    if dtype == "fp16":
        G[::2, 0] *= np.float32(2.0 ** 5)        # per-set normalisation exponents that differ
    X, f = dev(Xb, dtype), B.Factors.create(G)
    q, s = B.kroquant_quantize(X, f, path="onchip", scale_layout=layout)
    Yg = B.kroquant_transform_f32(X, f, path="onchip")
    qo, so, Y = co.quantize(Xb, G, dtype)
    P.check_values(Yg.cpu().numpy(), Y, dtype)
    s_rm = s.cpu().numpy()
    if layout == "tiled":
        s_rm = untile(s_rm.reshape(-1), tokens, d // 32)
    P.check_codes(q.cpu().numpy(), s_rm, qo, so, Y, exact=False, x_dtype=dtype)
    assert B.kroquant_last_device_error() == 0
    # next to the image path: the same bytes except where a value sits on a rounding boundary
    q2, s2 = B.kroquant_quantize(X, f, path="tensor", scale_layout=layout)
    assert (q != q2).float().mean().item() <= 1e-4 and (s != s2).float().mean().item() <= 1e-4


@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
def test_onchip_identity_factors_are_exact(B, dtype):
    Xb = W.gen_activations(spec(257, 96, 3), dtype)
    q_or, s_or, Y = co.plain_quantize(Xb, dtype)
    for n_sets in (1, 3):
        f = B.Factors.create(W.identity_factors(n_sets))
        q, s = B.kroquant_quantize(dev(Xb, dtype), f, path="onchip")
        P.check_codes(q.cpu().numpy(), s.cpu().numpy(), q_or, s_or, Y, exact=True)


@pytest.mark.parametrize("per_block", [False, True])
def test_onchip_factor_sets_of_extreme_scale(B, per_block):
    """Factor entries far from 1 (K scaled by 2^+-20, one factor nearly singular): the compensated products and the
    three-term split must hold up, and the scale bytes move with the factor of two."""
    tokens, d = 300, 1152
    Xb = W.gen_activations(spec(tokens, d, 17))
    for pw in (20, -20):
        G = W.gen_factors(31, n_sets=d // 32 if per_block else 1)
        G[:, 0] *= np.float32(2.0 ** pw)
        G[:, 3, 1, :] *= np.float32(1e-3)                      # a small second row: |det G4| shrinks a thousandfold
        X, f = dev(Xb), B.Factors.create(G)
        q, s = B.kroquant_quantize(X, f, path="onchip")
        Yg = B.kroquant_transform_f32(X, f, path="onchip")
        qo, so, Y = co.quantize(Xb, G)
        P.check_values(Yg.cpu().numpy(), Y)
        P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=False)
    assert B.kroquant_last_device_error() == 0


def test_onchip_back_to_back_and_tuned_calls_agree(B):
    # the builders run ahead of and behind the dependency wait of chained launches: every call must give the same bytes
    tokens, d = 2500, 2240
    X = dev(W.gen_activations(spec(tokens, d, 9)))
    for per_block in (False, True):
        f = B.Factors.create(W.gen_factors(5, n_sets=d // 32 if per_block else 1))
        ref = B.kroquant_quantize(X, f, path="onchip")
        outs = [B.kroquant_quantize(X, f, path="onchip") for _ in range(8)]
        outs += [B.kroquant_quantize(X, f, path="onchip", tuning=B.Tuning(dynamic=dyn, unit_tiles=u, trigger=tr, prefetch_tiles=pf,
                                                                           ctas_per_sm=cps))
                 for dyn, u, tr, pf, cps in [(0, 1, 1, 0, 3), (1, 2, 2, 4, 2), (0, 3, 0, 1, 1), (1, 1, 1, 2, 3)]]
        for q, s in outs:
            assert torch.equal(q, ref[0]) and torch.equal(s, ref[1])
    assert B.kroquant_last_device_error() == 0


def test_onchip_refusals_launch_nothing(B):
    X = dev(W.gen_activations(spec(64, 64, 3)))
    n0 = B.kroquant_launch_count()
    dense = B.Factors.create_dense(np.eye(32, dtype=np.float32)[None])
    with pytest.raises(RuntimeError):
        B.kroquant_quantize(X, dense, path="onchip")
    with pytest.raises(RuntimeError):
        B.kroquant_transform_f32(X, dense, path="onchip")
    assert B.kroquant_launch_count() == n0
