"""GPU parity for fp16 activations and for dense 32x32 blocks given directly."""
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


def dev(bits, dtype):
    t = torch.from_numpy(bits.view(np.int16).copy()).cuda()
    return t.view(torch.float16 if dtype == "fp16" else torch.bfloat16)


def spec(tokens, d, seed=5):
    return W.ActivationSpec(f"v{tokens}x{d}", tokens, d, seed=seed, outlier_channels=max(1, d // 100),
                            outlier_gain=50.0, spike_rows=min(2, tokens), spike_gain=8.0)


SHAPES = [(1, 32), (3, 1152), (129, 2240), (640, 1152), (256, 1152)]


@pytest.mark.parametrize("tokens,d", SHAPES)
def test_fp16_exact_kernels(B, tokens, d):
    Xb = W.gen_activations(spec(tokens, d), "fp16")
    X = dev(Xb, "fp16")
    q, s = B.kroquant_mxfp4_quantize(X)
    qo, so, Y = co.plain_quantize(Xb, "fp16")
    P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=True)
    sv = W.gen_channel_scales(3, d)
    q, s = B.kroquant_scale_quantize(X, torch.from_numpy(sv).cuda())
    qo, so, Y = co.scale_quantize(Xb, sv, "fp16")
    P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=True)
    f = B.Factors.create(W.identity_factors(1))
    for path in ("tensor", "alu", "auto"):
        q, s = B.kroquant_quantize(X, f, path=path)
        qo, so, Y = co.plain_quantize(Xb, "fp16")
        P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=True)


@pytest.mark.parametrize("path", ["tensor", "alu"])
@pytest.mark.parametrize("per_block", [False, True])
@pytest.mark.parametrize("tokens,d", SHAPES)
def test_fp16_kroquant(B, path, per_block, tokens, d):
    Xb = W.gen_activations(spec(tokens, d, seed=tokens + d), "fp16")
    G = W.gen_factors(tokens, n_sets=d // 32 if per_block else 1)
    X = dev(Xb, "fp16")
    f = B.Factors.create(G)
    q, s = B.kroquant_quantize(X, f, path=path)
    Yg = B.kroquant_transform_f32(X, f, path=path)
    qo, so, Y = co.quantize(Xb, G, "fp16")
    P.check_values(Yg.cpu().numpy(), Y, "fp16")
    P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=False, x_dtype="fp16")
    assert B.kroquant_last_device_error() == 0


def test_fp16_factor_scaling_is_folded_exactly(B):
    """Factor sets whose K is very large or very small exercise the normalisation exponent of
    the fp16 image (fast path) and, with tiny activations, the clamped slow path."""
    Xb = W.gen_activations(spec(256, 1152, seed=8), "fp16")
    x = W.fp16_bits_to_f32(Xb)
    for scale_pow, xpow in ((12, 0), (-12, 0), (-3, -10), (16, 3)):
        G = W.gen_factors(8)
        G[0, 0] *= np.float32(2.0 ** scale_pow)                   # K scales by 2^scale_pow
        Xs = W.f32_to_fp16_bits(x * np.float32(2.0 ** xpow))
        f = B.Factors.create(G)
        X = dev(Xs, "fp16")
        q, s = B.kroquant_quantize(X, f)
        Yg = B.kroquant_transform_f32(X, f)
        qo, so, Y = co.quantize(Xs, G, "fp16")
        P.check_values(Yg.cpu().numpy(), Y, "fp16")
        P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=False, x_dtype="fp16")


@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
def test_hadamard_fp16_and_bf16(B, dtype):
    Xb = W.gen_activations(spec(512, 1152, seed=9), dtype)
    abc = W.hadamard_lu_params(1)
    f = B.Factors.create_lu(abc)
    G = co.lu_to_factors(abc)
    X = dev(Xb, dtype)
    q, s = B.kroquant_quantize(X, f)
    Yg = B.kroquant_transform_f32(X, f)
    qo, so, Y = co.quantize(Xb, G, dtype)
    P.check_values(Yg.cpu().numpy(), Y, dtype)
    P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=False, x_dtype=dtype)


@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("n_sets_kind", ["shared", "per_block"])
def test_dense_blocks(B, dtype, n_sets_kind):
    tokens, d = 300, 1152
    Xb = W.gen_activations(spec(tokens, d, seed=12), dtype)
    Kd = W.gen_dense_blocks(12, n_sets=1 if n_sets_kind == "shared" else d // 32)
    f = B.Factors.create_dense(Kd)
    X = dev(Xb, dtype)
    q, s = B.kroquant_quantize(X, f)
    Yg = B.kroquant_transform_f32(X, f)
    qo, so, Y = co.quantize(Xb, x_dtype=dtype, K_dense=Kd)
    print(dtype, n_sets_kind, P.check_values(Yg.cpu().numpy(), Y, dtype))
    P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=False, x_dtype=dtype)
    # what dense handles do not support is refused with a status, nothing is launched
    n0 = B.kroquant_launch_count()
    with pytest.raises(B.KroQuantError) as e:
        B.kroquant_quantize(X, f, path="alu")
    assert e.value.status == 5
    with pytest.raises(B.KroQuantError):
        B.kroquant_dequantize(q, s, f)
    assert B.kroquant_launch_count() == n0
    bad = Kd.copy()
    bad[0] = 0
    with pytest.raises(B.KroQuantError):
        B.Factors.create_dense(bad)


def test_dense_blocks_built_from_factors_match_the_factor_handle(B):
    G = W.gen_factors(14)
    K = G[0, 0].astype(np.float64)
    for k in range(1, 5):
        K = np.kron(K, G[0, k].astype(np.float64))
    Kd = K.astype(np.float32)[None]
    Xb = W.gen_activations(spec(256, 1152, seed=14))
    X = dev(Xb, "bf16")
    Ya = B.kroquant_transform_f32(X, B.Factors.create(G)).cpu().numpy()
    Yb = B.kroquant_transform_f32(X, B.Factors.create_dense(Kd)).cpu().numpy()
    amax = np.abs(Ya.reshape(256, 36, 32)).max(axis=2, keepdims=True).repeat(32, 2).reshape(Ya.shape)
    assert (np.abs(Ya - Yb) <= 2e-7 * amax * 32).all()       # K rounded to float32 once


def test_pixart_shaped_fp16_full_size(B):
    """PixArt-Sigma runs in FP16 (paper Appendix D): the [8192,1152] tensor at full size."""
    sp = W.pixart_specs()[0]
    Xb = W.gen_activations(sp, "fp16")
    G = W.gen_factors(1)
    X = dev(Xb, "fp16")
    f = B.Factors.create(G)
    q, s = B.kroquant_quantize(X, f)
    Yg = B.kroquant_transform_f32(X, f)
    qo, so, Y = co.quantize(Xb, G, "fp16")
    print(P.check_values(Yg.cpu().numpy(), Y, "fp16"),
          P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=False, x_dtype="fp16"))


# ---- full-d Walsh-Hadamard comparison kernel -------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
@pytest.mark.parametrize("tokens,d", [(1, 32), (70, 64), (33, 256), (130, 1024), (37, 4096), (9, 8192), (5, 16384),
                                      (3000, 128), (1111, 2048), (700, 4096), (2500, 512), (300, 8192), (200, 16384)])
def test_fwht_quantize(B, dtype, tokens, d):
    Xb = W.gen_activations(spec(tokens, d, seed=d + tokens), dtype)
    X = dev(Xb, dtype)
    q, s = B.kroquant_fwht_quantize(X)
    Yg = B.kroquant_fwht_transform_f32(X)
    qo, so, Y = co.hadamard_quantize(Xb, dtype)
    print(d, P.check_values(Yg.cpu().numpy(), Y, dtype))
    P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=False, x_dtype=dtype)


def test_fwht_tensor_core_and_multi_pass_kernels_agree(B):
    """The comparison runs on the tensor-core pipeline (one product across the blocks of a token -- from d = 8192 on
    across its rows of 2 or 4 blocks, which a pass through tensor memory then mixes -- and a butterfly inside each
    block); the multi-pass kernel stays reachable through the tuning struct.  Both are held to
    the oracle, and to each other where no value sits on a rounding boundary."""
    for tokens, d in [(1500, 1024), (300, 4096), (150, 8192), (100, 16384)]:
        Xb = W.gen_activations(spec(tokens, d, seed=d), "bf16")
        X = dev(Xb, "bf16")
        qo, so, Y = co.hadamard_quantize(Xb, "bf16")
        outs = []
        for staged in (1, 0):
            n0 = B.kroquant_launch_count()
            q, s = B.kroquant_fwht_quantize(X, tuning=B.Tuning(compare_staged=staged))
            assert B.kroquant_launch_count() == n0 + 1
            P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=False)
            outs.append((q, s))
        assert (outs[0][0] != outs[1][0]).float().mean().item() <= 1e-4
    assert B.kroquant_last_device_error() == 0


def test_fwht_back_to_back_and_tuned_calls_agree(B):
    """Chained launches (programmatic dependent launch, dynamic and static tile distribution, several tiles per CTA) of
    the tensor-core Hadamard kernels must all give the same bytes."""
    for tokens, d in [(6000, 1024), (3000, 4096), (1200, 16384)]:
        X = dev(W.gen_activations(spec(tokens, d, seed=tokens), "bf16"), "bf16")
        ref = B.kroquant_fwht_quantize(X)
        outs = [B.kroquant_fwht_quantize(X) for _ in range(6)]
        outs += [B.kroquant_fwht_quantize(X, tuning=B.Tuning(dynamic=dyn, unit_tiles=u, trigger=tr, prefetch_tiles=pf))
                 for dyn, u, tr, pf in [(0, 1, 1, 0), (1, 2, 2, 4), (0, 3, 0, 1), (1, 1, 1, 2)]]
        for q, s in outs:
            assert torch.equal(q, ref[0]) and torch.equal(s, ref[1])
    assert B.kroquant_last_device_error() == 0


def test_fwht_rejects_other_sizes(B):
    import ctypes as C
    L = B.load_library()
    X = torch.zeros((4, 96), dtype=torch.bfloat16, device="cuda")
    q = torch.zeros((4, 48), dtype=torch.uint8, device="cuda")
    s = torch.zeros((4, 3), dtype=torch.uint8, device="cuda")
    args = lambda d: (C.c_void_p(X.data_ptr()), 0, 4, d, C.c_void_p(q.data_ptr()), C.c_void_p(s.data_ptr()), None)
    assert L.kroquant_fwht_quantize(*args(96)) == 2          # not a power of two
    assert L.kroquant_fwht_quantize(*args(16)) == 2
    assert L.kroquant_fwht_quantize(*args(32768)) == 2
