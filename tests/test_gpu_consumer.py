"""The quantizer's output feeds a block-scaled MXFP4 tensor-core GEMM directly (paper Section 3.4:
O = Q(A T) Q(W~)^T + low-rank branch): packed codes as they are, scale bytes in the 128 x 4 tiled
layout.  The consumer here is the library GEMM behind torch.nn.functional.scaled_mm."""
import numpy as np
import pytest
import torch

from oracle import c_oracle as co
from paper_2607_21446_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2607_21446_b200 import binding
    binding.load_library()
    return binding


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def spec(tokens, d, seed):
    return W.ActivationSpec("c", tokens, d, seed=seed, outlier_channels=max(1, d // 100), outlier_gain=50.0,
                            spike_rows=min(2, tokens), spike_gain=8.0)


@pytest.mark.parametrize("tokens,d,per_block", [(1, 32, False), (130, 288, False), (257, 1152, False),
                                                (300, 5600, False), (129, 2240, True), (640, 1152, True)])
def test_tiled_layout_is_a_reindexing_of_the_row_major_scales(B, tokens, d, per_block):
    Xb = W.gen_activations(spec(tokens, d, seed=tokens))
    X = dev_bf16(Xb)
    G = W.gen_factors(3, n_sets=d // 32 if per_block else 1)
    f = B.Factors.create(G)
    sv = torch.from_numpy(W.gen_channel_scales(3, d)).cuda()
    calls = {
        "kroquant": lambda **kw: B.kroquant_quantize(X, f, **kw),
        "kroquant_alu": lambda **kw: B.kroquant_quantize(X, f, path="alu", **kw),
        "scale": lambda **kw: B.kroquant_scale_quantize(X, sv, **kw),
        "plain": lambda **kw: B.kroquant_mxfp4_quantize(X, **kw),
    }
    for name, fn in calls.items():
        q0, s0 = fn()
        q1, s1 = fn(scale_layout="tiled")
        assert torch.equal(q0, q1), name
        expect = co.scales_to_tiled(s0.cpu().numpy(), fill=0)       # padding stays at the buffer's zeros
        assert s1.numel() == B.tiled_scale_bytes(tokens, d) == expect.size
        assert np.array_equal(s1.cpu().numpy(), expect), name


def _scaled_mm_mxfp4(qa, sa_tiled, qw, sw_tiled):
    F = torch.nn.functional
    if not hasattr(F, "scaled_mm"):
        pytest.skip("torch.nn.functional.scaled_mm not available")
    return F.scaled_mm(qa.view(torch.float4_e2m1fn_x2), qw.view(torch.float4_e2m1fn_x2).t(),
                       sa_tiled.view(torch.float8_e8m0fnu), F.ScalingType.BlockWise1x32,
                       sw_tiled.view(torch.float8_e8m0fnu), F.ScalingType.BlockWise1x32,
                       swizzle_a=F.SwizzleType.SWIZZLE_32_4_4, swizzle_b=F.SwizzleType.SWIZZLE_32_4_4,
                       output_dtype=torch.bfloat16)


@pytest.mark.parametrize("tokens,d,o", [(512, 1152, 256), (300, 3072, 384), (1024, 2240, 128)])
def test_w4a4_layer_through_the_block_scaled_gemm(B, tokens, d, o):
    """Q(A T) Q(W T^-T)^T computed by the tensor-core MXFP4 GEMM from the quantizer's raw outputs
    equals the product of the decoded operands (up to the GEMM's bf16 output rounding), and
    approximates A W^T."""
    A_bits = W.gen_activations(spec(tokens, d, seed=41))
    W_bits = W.f32_to_bf16_bits((np.random.default_rng(42).standard_normal((o, d)) * 0.05).astype(np.float32))
    A, Wt = dev_bf16(A_bits), dev_bf16(W_bits)
    fh = B.Factors.create_lu(W.hadamard_lu_params(1))       # orthogonal, symmetric: T^-T = T
    qa, sa = B.kroquant_quantize(A, fh, scale_layout="tiled")
    qw, sw = B.kroquant_quantize(Wt, fh, scale_layout="tiled")
    out = _scaled_mm_mxfp4(qa, sa, qw, sw).double()
    # reference: decode the same codes with the row-major scales of a second call
    qa2, sa2 = B.kroquant_quantize(A, fh)
    qw2, sw2 = B.kroquant_quantize(Wt, fh)
    assert torch.equal(qa, qa2) and torch.equal(qw, qw2)
    ref = B.kroquant_dequantize(qa2, sa2).double() @ B.kroquant_dequantize(qw2, sw2).double().T
    err = (out - ref).abs().max() / ref.abs().max()
    assert err < 2.0 ** -7, float(err)                       # bf16 output rounding (+ fp32 accumulation)
    exact = A.double() @ Wt.double().T
    rel = (out - exact).norm() / exact.norm()
    print(f"{tokens}x{d}x{o}: GEMM vs decoded product {float(err):.2e}; W4A4 vs bf16 layer {float(rel):.3f}")
    assert rel < 0.3


def _ulp16(y, dtype):
    """Spacing of the 16-bit format at |y| (float64 arrays)."""
    mant = 10 if dtype == "fp16" else 7
    emin = -14 if dtype == "fp16" else -126
    e = np.floor(np.log2(np.maximum(np.abs(y), 2.0 ** emin)))
    return 2.0 ** (e - mant)


@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("tokens,d,per_block", [(3, 1152, False), (640, 1152, False), (300, 2240, True)])
def test_dual_output_codes_and_16bit_transformed_activations(B, dtype, tokens, d, per_block):
    from tests import parity as P
    Xb = W.gen_activations(spec(tokens, d, seed=tokens + 7), dtype)
    X = torch.from_numpy(Xb.view(np.int16).copy()).cuda().view(torch.float16 if dtype == "fp16" else torch.bfloat16)
    G = W.gen_factors(5, n_sets=d // 32 if per_block else 1)
    f = B.Factors.create(G)
    q, s, AT = B.kroquant_quantize_dual(X, f)
    q0, s0 = B.kroquant_quantize(X, f, path="tensor")
    assert torch.equal(q, q0) and torch.equal(s, s0)                       # same codes as the plain call
    qo, so, Y = co.quantize(Xb, G, dtype)
    P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=False, x_dtype=dtype)
    at_bits = AT.view(torch.int16).cpu().numpy().view(np.uint16)
    at = (W.fp16_bits_to_f32(at_bits) if dtype == "fp16" else W.bf16_bits_to_f32(at_bits)).astype(np.float64)
    ref_bits = co.round_y_to_16bit(Y, dtype)
    # identical to the oracle's rounding except where the GPU's float value sits on the other side of a
    # 16-bit rounding boundary: then one unit in the last place, and rare
    diff = at_bits != ref_bits
    assert diff.mean() < 2e-3, diff.mean()
    y = Y.astype(np.float64)
    amax = np.abs(y.reshape(tokens, d // 32, 32)).max(axis=2, keepdims=True).repeat(32, 2).reshape(y.shape)
    tol = 0.5 * _ulp16(y, dtype) + 1e-5 * np.maximum(np.abs(y), amax / P.FLOOR_DIV[dtype])
    assert (np.abs(at - y) <= tol * (1 + 1e-9)).all()
    assert B.kroquant_last_device_error() == 0


def test_low_rank_branch_and_w4a4_branch_from_one_pass(B):
    """O = Q(A T) Q(W~)^T + (A T) L R with both activations operands from kroquant_quantize_dual."""
    tokens, d, o, r = 256, 1152, 128, 16
    A_bits = W.gen_activations(spec(tokens, d, seed=51))
    rng = np.random.default_rng(52)
    W_bits = W.f32_to_bf16_bits((rng.standard_normal((o, d)) * 0.05).astype(np.float32))
    A, Wt = dev_bf16(A_bits), dev_bf16(W_bits)
    fh = B.Factors.create_lu(W.hadamard_lu_params(1))
    # low-rank part of the transformed weight W~ = W T^-T (= W T for the Hadamard): best rank-r piece
    WT = B.kroquant_transform_f32(Wt, fh).double()
    U, S, Vh = torch.linalg.svd(WT, full_matrices=False)
    L, R = (U[:, :r] * S[:r]), Vh[:r]                                   # W~ ~ L R + residual
    resid = (WT - L @ R).to(torch.bfloat16)
    qa, sa, AT = B.kroquant_quantize_dual(A, fh, scale_layout="tiled")
    qw, sw = B.kroquant_mxfp4_quantize(resid, scale_layout="tiled")     # residual is already transformed
    main = _scaled_mm_mxfp4(qa, sa, qw, sw).double()
    low = (AT.double() @ R.T) @ L.T
    exact = A.double() @ Wt.double().T
    rel_with = ((main + low) - exact).norm() / exact.norm()
    qw0, sw0 = B.kroquant_quantize(Wt, fh, scale_layout="tiled")
    rel_without = (_scaled_mm_mxfp4(qa, sa, qw0, sw0).double() - exact).norm() / exact.norm()
    print("W4A4 + rank-16 branch:", float(rel_with), "W4A4 alone:", float(rel_without))
    assert rel_with < rel_without
