"""kroquant_gemm_mxfp4: the W4A4 product of the quantized layer (Section 3.4) on the block-scaled FP4
tensor-core path, fed by the quantizer's own outputs (packed codes + tiled scale bytes).

Every product a*b*2^(sa+sb) is exact in fp32, so the only error is the order of the fp32 accumulation:
the tolerance is 1e-6 of sum |a||b| per output (measured: 0 on most shapes, 2e-8 at K = 3072).
"""
import numpy as np
import pytest
import torch

from oracle import c_oracle as co
from oracle import calib_oracle as cal
from paper_2607_21446_b200 import binding as kb
from paper_2607_21446_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL = 1e-6


@pytest.fixture(autouse=True, params=["pair", "single"])
def gemm_variant(request):
    """Every test runs with both kernels: CTA pairs on 256 x 256 tiles (default) and one CTA per 128 x 128 tile."""
    kb.set_gemm_pair(request.param == "pair")
    yield request.param
    kb.set_gemm_pair(True)


def _operand(rows, K, seed, spread=True):
    """bf16 tensor whose 32-blocks have scales spread over 2^-3 .. 2^3 (so that scale bytes differ)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    x = torch.randn(rows, K, device="cuda", generator=g)
    if spread:
        e = torch.randint(-3, 4, (rows, K // 32), device="cuda", generator=g).float()
        x = x * torch.exp2(e).repeat_interleave(32, 1)
    return x.to(torch.bfloat16).contiguous()


def _decoded(x_bf16):
    """-> (codes, tiled scales) from the GPU quantizer and the oracle's decode of the same operand."""
    q_t, s_t = kb.kroquant_mxfp4_quantize(x_bf16, scale_layout="tiled")
    q_r, s_r = kb.kroquant_mxfp4_quantize(x_bf16)
    assert torch.equal(q_t, q_r)
    dec = co.dequantize(q_r.cpu().numpy(), s_r.cpu().numpy()).astype(np.float64)
    return q_t, s_t, dec


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (1, 32, 32), (130, 96, 288), (257, 160, 1152), (300, 512, 5600),
                                   (1000, 1056, 2240)])
def test_against_the_decoded_float64_product(M, N, K):
    A, W = _operand(M, K, 1), _operand(N, K, 2)
    qa, sa, Ad = _decoded(A)
    qw, sw, Wd = _decoded(W)
    ref = Ad @ Wd.T
    bound = np.abs(Ad) @ np.abs(Wd).T
    out = kb.kroquant_gemm_mxfp4(qa, sa, qw, sw, out_dtype=torch.float32)
    torch.cuda.synchronize()
    o = out.double().cpu().numpy()
    assert np.all(np.isfinite(o))
    assert np.all(np.abs(o - ref) <= TOL * bound + 1e-300)
    assert kb.kroquant_last_device_error() == 0
    # bf16 output = the fp32 result rounded once
    out16 = kb.kroquant_gemm_mxfp4(qa, sa, qw, sw, out_dtype=torch.bfloat16)
    assert torch.equal(out16, out.to(torch.bfloat16))


def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    return [(int(rng.integers(1, 700)), 32 * int(rng.integers(1, 34)), 32 * int(rng.integers(1, 66))) for _ in range(n)]


@pytest.mark.parametrize("M,N,K", _random_shapes(14, 2024))
def test_seeded_random_shapes(M, N, K):
    A, W = _operand(M, K, M + K), _operand(N, K, N + K)
    qa, sa, Ad = _decoded(A)
    qw, sw, Wd = _decoded(W)
    out = kb.kroquant_gemm_mxfp4(qa, sa, qw, sw, out_dtype=torch.float32).double().cpu().numpy()
    assert np.all(np.abs(out - Ad @ Wd.T) <= TOL * (np.abs(Ad) @ np.abs(Wd).T) + 1e-300)
    low = kb.kroquant_gemm_bf16(A, W, out_dtype=torch.float32).double().cpu().numpy()
    Af, Wf = A.double().cpu().numpy(), W.double().cpu().numpy()
    # 16-bit operands with outlier channels: the products span many binades, and the tensor core drops the bits
    # below its accumulator's last place once per 16-deep instruction, so the bound grows with K/16 roundings of
    # at most 2^-23 of the running sum of magnitudes (seen: 1.7e-6 of that sum at K = 2048)
    low_tol = (K // 16 + 2) * 2.0 ** -23
    assert np.all(np.abs(low - Af @ Wf.T) <= low_tol * (np.abs(Af) @ np.abs(Wf).T) + 1e-300)
    assert kb.kroquant_last_device_error() == 0


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_output_base_that_is_only_16_byte_aligned(dtype):
    """The epilogue uses 32-byte stores when the output base allows it and 16-byte stores otherwise."""
    M, N, K = 200, 288, 256
    A, W = _operand(M, K, 21), _operand(N, K, 22)
    qa, sa, _ = _decoded(A)
    qw, sw, _ = _decoded(W)
    ref = kb.kroquant_gemm_mxfp4(qa, sa, qw, sw, out_dtype=dtype)
    shift = 16 // ref.element_size()
    flat = torch.zeros(M * N + shift, dtype=dtype, device="cuda")
    out = flat[shift:].view(M, N)
    assert out.data_ptr() % 32 == 16
    kb.kroquant_gemm_mxfp4(qa, sa, qw, sw, out=out)
    assert torch.equal(out, ref)
    assert float(flat[:shift].abs().max()) == 0.0


def test_low_rank_branch_is_added_before_the_single_rounding():
    M, N, K = 384, 256, 512
    A, W = _operand(M, K, 3), _operand(N, K, 4)
    qa, sa, Ad = _decoded(A)
    qw, sw, Wd = _decoded(W)
    add = _operand(M, N, 5, spread=False)
    out = kb.kroquant_gemm_mxfp4(qa, sa, qw, sw, add=add, out_dtype=torch.float32)
    ref = Ad @ Wd.T + add.double().cpu().numpy()
    bound = np.abs(Ad) @ np.abs(Wd).T + np.abs(add.double().cpu().numpy())
    assert np.all(np.abs(out.double().cpu().numpy() - ref) <= TOL * bound)


def test_same_result_as_the_library_block_scaled_gemm():
    F = torch.nn.functional
    if not hasattr(F, "scaled_mm"):
        pytest.skip("torch.nn.functional.scaled_mm not available")
    M, N, K = 512, 384, 1152
    A, W = _operand(M, K, 6), _operand(N, K, 7)
    qa, sa, _ = _decoded(A)
    qw, sw, _ = _decoded(W)
    lib = F.scaled_mm(qa.view(torch.float4_e2m1fn_x2), qw.view(torch.float4_e2m1fn_x2).t(),
                      sa.view(torch.float8_e8m0fnu), F.ScalingType.BlockWise1x32,
                      sw.view(torch.float8_e8m0fnu), F.ScalingType.BlockWise1x32,
                      swizzle_a=F.SwizzleType.SWIZZLE_32_4_4, swizzle_b=F.SwizzleType.SWIZZLE_32_4_4,
                      output_dtype=torch.bfloat16)
    ours = kb.kroquant_gemm_mxfp4(qa, sa, qw, sw, out_dtype=torch.bfloat16)
    # both round an (almost) identical fp32 sum to bf16: at most one bf16 step apart, and rarely
    diff = (ours.float() - lib.float()).abs()
    assert float((diff > 0).float().mean()) < 1e-3
    assert float((diff / lib.float().abs().clamp_min(1e-30)).max()) <= 2.0 ** -7


@pytest.mark.parametrize("per_block", [False, True])
def test_quantized_layer_from_activations_to_output(per_block):
    """The inference form of Section 3.4 with this library's own kernels end to end: KroQuant quantizer on
    the activations (factors G), the same quantizer on the weights with the Kronecker set of T^-T, then the
    FP4 GEMM; compared with the oracle's Q(A T) Q(W T^-T)^T."""
    M, o, d, seed = 640, 384, 1152, 9
    n_sets = d // 32 if per_block else 1
    A_bits = wl.gen_activations(wl.calib_spec(M, d, seed))
    W_bits = wl.gen_weights(seed, o, d)
    theta = wl.gen_lu_params(seed, n_sets).astype(np.float64)
    G = cal.lu_factors(theta).astype(np.float32)
    H = np.stack([[np.linalg.inv(G[s, k].astype(np.float64)).T for k in range(5)] for s in range(n_sets)]).astype(np.float32)
    dev = torch.device("cuda:0")
    A_t = torch.from_numpy(A_bits.view(np.int16)).to(dev).view(torch.bfloat16)
    W_t = torch.from_numpy(W_bits.view(np.int16)).to(dev).view(torch.bfloat16)
    fa, fw = kb.Factors.create(G), kb.Factors.create(H)
    qa, sa = kb.kroquant_quantize(A_t, fa, scale_layout="tiled")
    qw, sw = kb.kroquant_quantize(W_t, fw, scale_layout="tiled")
    out = kb.kroquant_gemm_mxfp4(qa, sa, qw, sw, out_dtype=torch.float32).double().cpu().numpy()
    # (1) the GEMM on the codes the GPU quantizer produced: exact up to the accumulation order
    qa_r, sa_r = kb.kroquant_quantize(A_t, fa)
    qw_r, sw_r = kb.kroquant_quantize(W_t, fw)
    assert torch.equal(qa_r, qa) and torch.equal(qw_r, qw)
    Ad = co.dequantize(qa_r.cpu().numpy(), sa_r.cpu().numpy()).astype(np.float64)
    Wd = co.dequantize(qw_r.cpu().numpy(), sw_r.cpu().numpy()).astype(np.float64)
    assert np.all(np.abs(out - Ad @ Wd.T) <= TOL * (np.abs(Ad) @ np.abs(Wd).T))
    # (2) the whole chain against the oracle's own quantizer: a code within 1e-5 of a rounding boundary
    # may differ (parity rule of the quantizer); each such code moves one output row or column by one grid
    # step of one element (large for an outlier channel), so the comparison is in the Frobenius norm
    qa_o, sa_o, _ = co.quantize(A_bits, G)
    qw_o, sw_o, _ = co.quantize(W_bits, H)
    ref = co.dequantize(qa_o, sa_o).astype(np.float64) @ co.dequantize(qw_o, sw_o).astype(np.float64).T
    assert np.linalg.norm(out - ref) <= 5e-3 * np.linalg.norm(ref)
    assert (qa.cpu().numpy() != qa_o).mean() <= 1e-4 and (qw.cpu().numpy() != qw_o).mean() <= 1e-4
    fa.destroy()
    fw.destroy()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_linear_layer_call_equals_the_two_separate_calls(dtype):
    M, o, d, seed = 300, 256, 1152, 13
    A_bits = wl.gen_activations(wl.calib_spec(M, d, seed), "fp16" if dtype == torch.float16 else "bf16")
    A_t = torch.from_numpy(A_bits.view(np.int16)).cuda().view(dtype)
    W_t = torch.from_numpy(wl.gen_weights(seed, o, d).view(np.int16)).cuda().view(torch.bfloat16)
    theta = wl.gen_lu_params(seed, 1).astype(np.float64)
    G = cal.lu_factors(theta).astype(np.float32)
    H = np.stack([[np.linalg.inv(G[0, k].astype(np.float64)).T for k in range(5)]]).astype(np.float32)
    layer = kb.LinearW4A4.from_weights(W_t, G, H)
    add = _operand(M, o, 14, spread=False)
    out = layer(A_t, add=add)
    out_again = layer(A_t, add=add)          # work buffers reused
    qa, sa = kb.kroquant_quantize(A_t, layer.factors, scale_layout="tiled")
    ref = kb.kroquant_gemm_mxfp4(qa, sa, layer.w_codes, layer.w_scales, add=add)
    assert torch.equal(out, ref) and torch.equal(out_again, ref)
    assert kb.kroquant_last_device_error() == 0


@pytest.mark.parametrize("M,N,K", [(300, 128, 1152), (257, 96, 136), (1000, 512, 128), (64, 32, 8)])
def test_bf16_gemm_for_the_low_rank_branch(M, N, K):
    g = torch.Generator(device="cuda")
    g.manual_seed(M + N + K)
    A = torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16)
    Bm = torch.randn(N, K, device="cuda", generator=g).to(torch.bfloat16)
    add = torch.randn(M, N, device="cuda", generator=g)
    ref = A.double().cpu().numpy() @ Bm.double().cpu().numpy().T
    bound = np.abs(A.double().cpu().numpy()) @ np.abs(Bm.double().cpu().numpy()).T
    out = kb.kroquant_gemm_bf16(A, Bm, out_dtype=torch.float32).double().cpu().numpy()
    assert np.all(np.abs(out - ref) <= 1e-6 * bound + 1e-30)          # exact products, fp32 accumulation
    out2 = kb.kroquant_gemm_bf16(A, Bm, add=add, out_dtype=torch.float32).double().cpu().numpy()
    assert np.all(np.abs(out2 - (ref + add.double().cpu().numpy())) <= 1e-6 * (bound + np.abs(add.double().cpu().numpy())))
    out16 = kb.kroquant_gemm_bf16(A, Bm)
    assert torch.equal(out16, kb.kroquant_gemm_bf16(A, Bm, out_dtype=torch.float32).to(torch.bfloat16))
    assert kb.kroquant_last_device_error() == 0


def test_whole_layer_with_low_rank_branch():
    """Section 3.4's inference form with this library's kernels only:
    O = Q(A T) Q(W~ - L R)^T + (A T) R^T L^T, the second term in 16 bit with rank 128."""
    M, o, d, r, seed = 384, 256, 1152, 128, 17
    rng = np.random.default_rng(seed)
    A_bits = wl.gen_activations(wl.calib_spec(M, d, seed))
    A_t = torch.from_numpy(A_bits.view(np.int16)).cuda().view(torch.bfloat16)
    W = wl.bf16_bits_to_f32(wl.gen_weights(seed, o, d)).astype(np.float64)
    theta = wl.gen_lu_params(seed, 1).astype(np.float64)
    G = cal.lu_factors(theta).astype(np.float32)
    K_, P_ = cal.blocks_of(theta)
    Wt = cal.apply_blocks(W, P_)                                   # W~ = W T^-T
    U_, s_, Vt_ = np.linalg.svd(Wt, full_matrices=False)            # a rank-r split of W~ stands in for LoRaQ's L, R
    Lm = (U_[:, :r] * s_[:r]).astype(np.float32)                    # [o, r]
    Rm = Vt_[:r].astype(np.float32)                                 # [r, d]
    L_t = torch.from_numpy(Lm).cuda().to(torch.bfloat16).contiguous()
    R_t = torch.from_numpy(Rm).cuda().to(torch.bfloat16).contiguous()
    resid = torch.from_numpy((Wt - L_t.double().cpu().numpy() @ R_t.double().cpu().numpy()).astype(np.float32)).cuda().to(torch.bfloat16)
    qw, sw = kb.kroquant_mxfp4_quantize(resid.contiguous(), scale_layout="tiled")       # Q(W~ - L R), offline
    fa = kb.Factors.create(G)
    qa, sa, AT = kb.kroquant_quantize_dual(A_t, fa, scale_layout="tiled")               # codes, scales, A T in bf16
    low = kb.kroquant_gemm_bf16(kb.kroquant_gemm_bf16(AT, R_t), L_t)                    # (A T R^T) L^T, bf16 [M, o]
    out = kb.kroquant_gemm_mxfp4(qa, sa, qw, sw, add=low, out_dtype=torch.float32).double().cpu().numpy()
    # oracle: decode both quantized operands, float64 products; the 16-bit branch from the same bf16 inputs
    qa_r, sa_r = kb.kroquant_quantize(A_t, fa)
    qw_r, sw_r = kb.kroquant_mxfp4_quantize(resid.contiguous())
    main = co.dequantize(qa_r.cpu().numpy(), sa_r.cpu().numpy()).astype(np.float64) @ \
        co.dequantize(qw_r.cpu().numpy(), sw_r.cpu().numpy()).astype(np.float64).T
    branch = (AT.double().cpu().numpy() @ R_t.double().cpu().numpy().T) @ L_t.double().cpu().numpy().T
    ref = main + branch
    # two bf16 roundings on the branch (2^-9 relative each); the W4A4 part is exact up to accumulation order
    assert np.abs(out - ref).max() <= 1e-2 * np.abs(branch).max() + 1e-6 * np.abs(main).max()
    # and the layer does what it is for: close to the unquantized product A W^T
    exact = wl.bf16_bits_to_f32(A_bits).astype(np.float64) @ W.T
    assert np.linalg.norm(out - exact) < 0.25 * np.linalg.norm(exact)
    fa.destroy()


def test_argument_checks():
    A, W = _operand(128, 128, 1), _operand(128, 128, 2)
    qa, sa, _ = _decoded(A)
    qw, sw, _ = _decoded(W)
    L = kb.load_library()
    import ctypes as C
    out = torch.empty((128, 128), dtype=torch.float32, device="cuda")
    p = lambda t: C.c_void_p(t.data_ptr())
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert L.kroquant_gemm_mxfp4(p(qa), p(sa), p(qw), p(sw), 128, 128, 100, None, p(out), 0, st) == 2      # K % 32
    assert L.kroquant_gemm_mxfp4(p(qa), p(sa), p(qw), p(sw), 128, 100, 128, None, p(out), 0, st) == 2      # N % 32
    assert L.kroquant_gemm_mxfp4(p(qa), None, p(qw), p(sw), 128, 128, 128, None, p(out), 0, st) == 1       # null
    assert L.kroquant_gemm_mxfp4(p(qa), p(sa), p(qw), p(sw), 128, 128, 128, None, p(out), 7, st) == 5      # dtype
    assert L.kroquant_gemm_mxfp4(p(qa), p(sa), p(qw), p(sw), 0, 128, 128, None, p(out), 0, st) == 0        # empty
    with pytest.raises(ValueError):
        kb.kroquant_gemm_mxfp4(qa, sa[:100], qw, sw)
