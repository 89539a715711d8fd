"""The transform pair the quantizer serves (paper Section 1, first equation; Section 3.4
inference formula):  A -> A T,  W -> W T^-T  leaves  A W^T  unchanged, and the W4A4 product
Q(A T) Q(W T^-T)^T approximates it.  T^-T is itself block-diagonal Kronecker, with factors
G_k^-T, so both operands go through the same library calls."""
import numpy as np
import pytest
import torch

from paper_2607_21446_b200 import workloads as W

pytestmark = pytest.mark.gpu


def inverse_transpose_factors(G):
    Gi = np.linalg.inv(G.astype(np.float64))          # [n_sets, 5, 2, 2], each 2x2 inverted
    return np.ascontiguousarray(np.swapaxes(Gi, -1, -2)).astype(np.float32)


@pytest.mark.parametrize("n_sets_kind", ["shared", "per_block"])
def test_transform_pair_leaves_the_linear_map_invariant(n_sets_kind):
    from paper_2607_21446_b200 import binding as B
    tokens, d, o = 512, 1152, 256
    A_bits = W.gen_activations(W.ActivationSpec("A", tokens, d, seed=21, outlier_channels=12, outlier_gain=50.0))
    rngw = np.random.default_rng(22)
    W_bits = W.f32_to_bf16_bits((rngw.standard_normal((o, d)) * 0.05).astype(np.float32))
    n_sets = 1 if n_sets_kind == "shared" else d // 32
    G = W.gen_factors(21, n_sets=n_sets)
    Ginvt = inverse_transpose_factors(G)
    A = torch.from_numpy(A_bits.view(np.int16)).cuda().view(torch.bfloat16)
    Wt = torch.from_numpy(W_bits.view(np.int16)).cuda().view(torch.bfloat16)
    fa, fw = B.Factors.create(G), B.Factors.create(Ginvt)
    ref = A.double() @ Wt.double().T
    # (1) without quantization the pair is invariant (up to fp32 rounding of the transforms)
    AT = B.kroquant_transform_f32(A, fa).double()
    WT = B.kroquant_transform_f32(Wt, fw).double()
    inv_err = ((AT @ WT.T) - ref).abs().max() / ref.abs().max()
    assert inv_err < 2e-5, inv_err
    # (2) W4A4: quantize both, decode, multiply
    qa, sa = B.kroquant_quantize(A, fa)
    qw, sw = B.kroquant_quantize(Wt, fw)
    out = B.kroquant_dequantize(qa, sa).double() @ B.kroquant_dequantize(qw, sw).double().T
    rel = (out - ref).norm() / ref.norm()
    # (3) the same without any transform (bare MXFP4 on both operands)
    qa0, sa0 = B.kroquant_mxfp4_quantize(A)
    qw0, sw0 = B.kroquant_mxfp4_quantize(Wt)
    out0 = B.kroquant_dequantize(qa0, sa0).double() @ B.kroquant_dequantize(qw0, sw0).double().T
    rel0 = (out0 - ref).norm() / ref.norm()
    print(n_sets_kind, "invariance", float(inv_err), "W4A4 rel err with T", float(rel), "without", float(rel0))
    # 4-bit products with uncalibrated random factors: tens of percent either way (the factors
    # here are random, not learned; this is a sanity bound, not a quality claim)
    assert rel < 0.5 and rel0 < 0.5
    # (4) decoding with the inverse factors recovers A up to the quantization error
    back = B.kroquant_dequantize(qa, sa, fa).double()
    assert (back - A.double()).norm() / A.double().norm() < 0.25
    assert B.kroquant_last_device_error() == 0


def test_hadamard_transform_reduces_the_w4a4_error_on_outlier_activations():
    """The paper's premise (Section 1; Section 3.2 Hadamard initialisation): mixing channels
    inside each 32-block spreads outlier channels and lowers the W4A4 error of A W^T."""
    from paper_2607_21446_b200 import binding as B
    tokens, d, o = 1024, 1152, 256
    A_bits = W.gen_activations(W.ActivationSpec("A", tokens, d, seed=31, outlier_channels=12, outlier_gain=50.0))
    W_bits = W.f32_to_bf16_bits((np.random.default_rng(32).standard_normal((o, d)) * 0.05).astype(np.float32))
    A = torch.from_numpy(A_bits.view(np.int16)).cuda().view(torch.bfloat16)
    Wt = torch.from_numpy(W_bits.view(np.int16)).cuda().view(torch.bfloat16)
    ref = A.double() @ Wt.double().T
    fh = B.Factors.create_lu(W.hadamard_lu_params(1))     # orthogonal and symmetric: T^-T = T
    qa, sa = B.kroquant_quantize(A, fh)
    qw, sw = B.kroquant_quantize(Wt, fh)
    out = B.kroquant_dequantize(qa, sa).double() @ B.kroquant_dequantize(qw, sw).double().T
    qa0, sa0 = B.kroquant_mxfp4_quantize(A)
    qw0, sw0 = B.kroquant_mxfp4_quantize(Wt)
    out0 = B.kroquant_dequantize(qa0, sa0).double() @ B.kroquant_dequantize(qw0, sw0).double().T
    rel, rel0 = float((out - ref).norm() / ref.norm()), float((out0 - ref).norm() / ref.norm())
    print("W4A4 rel err: hadamard", rel, "none", rel0)
    assert rel < rel0
