"""GPU parity tests: the CUDA path, called through the C ABI (ctypes binding), against
the CPU oracle on the same seeded inputs.  Rules P0-P3 are in tests/parity.py."""
import numpy as np
import pytest
import torch

from oracle import c_oracle as co
from paper_2607_21446_b200 import workloads as W
from tests import parity as P
from tests.test_oracle_mxfp4 import brute_code

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2607_21446_b200 import binding
    binding.load_library()
    assert torch.cuda.is_available()
    return binding


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def host(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy()


def spec(tokens, d, seed=5):
    return W.ActivationSpec(f"t{tokens}x{d}", tokens, d, seed=seed,
                            outlier_channels=max(1, d // 100), outlier_gain=50.0,
                            spike_rows=min(2, tokens), spike_gain=8.0)


RAGGED = [(1, 32), (2, 64), (3, 1152), (31, 64), (33, 1152), (257, 96), (129, 2240), (640, 1152)]


# ---- hardware convert ------------------------------------------------------------------
def test_e2m1_convert_matches_oracle_table(B):
    bits = np.arange(0, 1 << 16, dtype=np.uint32).astype(np.uint16)
    vals = W.bf16_bits_to_f32(bits)
    vals = vals[np.isfinite(vals)]
    extra = []
    for b in (0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0):
        f = np.float32(b)
        for s in (1.0, -1.0):
            extra += [s * f, s * np.nextafter(f, np.float32(0)), s * np.nextafter(f, np.float32(9))]
    vals = np.concatenate([vals, np.asarray(extra, np.float32)])
    got = host(B.kroquant_debug_e2m1_codes(torch.from_numpy(vals).cuda()))
    expect = np.array([brute_code(float(v)) for v in vals], dtype=np.uint8)
    bad = got != expect
    assert not bad.any(), (vals[bad][:8], got[bad][:8], expect[bad][:8])


# ---- P0: exact kernels -----------------------------------------------------------------
@pytest.mark.parametrize("tokens,d", RAGGED + [(256, 1152)])
def test_plain_mxfp4_bit_exact(B, tokens, d):
    Xb = W.gen_activations(spec(tokens, d))
    q_or, s_or, Y = co.plain_quantize(Xb)
    q, s = B.kroquant_mxfp4_quantize(dev_bf16(Xb))
    P.check_codes(host(q), host(s), q_or, s_or, Y, exact=True)


@pytest.mark.parametrize("tokens,d", RAGGED + [(256, 1152)])
def test_scale_quantize_bit_exact(B, tokens, d):
    Xb = W.gen_activations(spec(tokens, d))
    sv = W.gen_channel_scales(7, d)
    q_or, s_or, Y = co.scale_quantize(Xb, sv)
    q, s = B.kroquant_scale_quantize(dev_bf16(Xb), torch.from_numpy(sv).cuda())
    P.check_codes(host(q), host(s), q_or, s_or, Y, exact=True)


@pytest.mark.parametrize("path", ["auto", "tensor", "alu"])
@pytest.mark.parametrize("tokens,d", [(3, 1152), (129, 2240), (256, 1152)])
def test_identity_factors_bit_exact_on_every_path(B, path, tokens, d):
    Xb = W.gen_activations(spec(tokens, d))
    q_or, s_or, Y = co.plain_quantize(Xb)
    f = B.Factors.create(W.identity_factors(1))
    q, s = B.kroquant_quantize(dev_bf16(Xb), f, path=path)
    P.check_codes(host(q), host(s), q_or, s_or, Y, exact=True)


# ---- P1/P2/P3: the KroQuant quantizer ----------------------------------------------------
def run_kroquant(B, Xb, G, path):
    f = B.Factors.create(G)
    X = dev_bf16(Xb)
    q, s = B.kroquant_quantize(X, f, path=path)
    Yg = B.kroquant_transform_f32(X, f, path=path)
    q_or, s_or, Y = co.quantize(Xb, G)
    v = P.check_values(host(Yg), Y)
    c = P.check_codes(host(q), host(s), q_or, s_or, Y, exact=False)
    assert B.kroquant_last_device_error() == 0
    return {**v, **c}


@pytest.mark.parametrize("path", ["auto", "tensor", "alu"])
def test_tiny_config(B, path):
    Xb = W.gen_activations(W.tiny_spec())
    r = run_kroquant(B, Xb, W.gen_factors(0), path)
    print(path, r)


@pytest.mark.parametrize("path", ["tensor", "alu"])
@pytest.mark.parametrize("tokens,d", RAGGED)
def test_ragged_shapes(B, path, tokens, d):
    Xb = W.gen_activations(spec(tokens, d, seed=tokens + d))
    run_kroquant(B, Xb, W.gen_factors(tokens), path)


@pytest.mark.parametrize("path", ["auto", "tensor", "alu"])
def test_hadamard_and_lu_factors(B, path):
    Xb = W.gen_activations(spec(512, 1152, seed=9))
    X = dev_bf16(Xb)
    for abc in (W.hadamard_lu_params(1), W.gen_lu_params(3, 1)):
        f = B.Factors.create_lu(abc)
        G = co.lu_to_factors(abc)
        assert np.array_equal(f.get(), G)          # the library's LU helper = the oracle's
        q, s = B.kroquant_quantize(X, f, path=path)
        Yg = B.kroquant_transform_f32(X, f, path=path)
        q_or, s_or, Y = co.quantize(Xb, G)
        P.check_values(host(Yg), Y)
        P.check_codes(host(q), host(s), q_or, s_or, Y, exact=False)


@pytest.mark.parametrize("path", ["tensor", "alu"])
@pytest.mark.parametrize("tokens,d", [(1, 32), (64, 320), (33, 2240), (128, 5600), (300, 1152)])
def test_per_block_factor_sets(B, path, tokens, d):
    Xb = W.gen_activations(spec(tokens, d, seed=2))
    run_kroquant(B, Xb, W.gen_factors(2, n_sets=d // 32), path)


def test_outputs_stay_inside_their_buffers(B):
    tokens, d = 130, 1152
    Xb = W.gen_activations(spec(tokens, d))
    f = B.Factors.create(W.gen_factors(1))
    pad = 4096
    qbuf = torch.full((tokens * d // 2 + 2 * pad,), 0xAB, dtype=torch.uint8, device="cuda")
    sbuf = torch.full((tokens * d // 32 + 2 * pad,), 0xCD, dtype=torch.uint8, device="cuda")
    q = qbuf[pad:pad + tokens * d // 2].view(tokens, d // 2)
    s = sbuf[pad:pad + tokens * d // 32].view(tokens, d // 32)
    for path in ("tensor", "alu"):
        B.kroquant_quantize(dev_bf16(Xb), f, q, s, path=path)
        torch.cuda.synchronize()
        assert (qbuf[:pad] == 0xAB).all() and (qbuf[-pad:] == 0xAB).all()
        assert (sbuf[:pad] == 0xCD).all() and (sbuf[-pad:] == 0xCD).all()


def test_power_of_two_equivariance_on_gpu(B):
    Xb = W.gen_activations(spec(256, 1152, seed=4))
    x = W.bf16_bits_to_f32(Xb)
    f = B.Factors.create(W.gen_factors(4))
    q0, s0 = B.kroquant_quantize(dev_bf16(Xb), f)
    q1, s1 = B.kroquant_quantize(dev_bf16(W.f32_to_bf16_bits(x * np.float32(2.0 ** 9))), f)
    assert torch.equal(q0, q1)
    assert torch.equal(s1.int(), s0.int() + 9)


# ---- decode ----------------------------------------------------------------------------------
def test_decode_every_code_under_every_scale_byte(B):
    """All 256 code bytes under all 255 valid scale bytes (S = 0 decodes to subnormal floats, S = 254 to 6 * 2^127),
    both output types, bit for bit; and shapes whose size is no multiple of what a thread or a CTA takes."""
    codes = np.arange(256, dtype=np.uint8)
    q_or = np.tile(codes, (255, 1)).reshape(255, 16, 16)               # row S: 16 blocks, every byte value once
    q_or = np.ascontiguousarray(q_or.reshape(255, 256))                # tokens = 255, d = 512
    s_or = np.repeat(np.arange(255, dtype=np.uint8)[:, None], 16, axis=1)
    q, s = torch.from_numpy(q_or).cuda(), torch.from_numpy(s_or).cuda()
    out = host(B.kroquant_dequantize(q, s))
    ref = co.dequantize(q_or, s_or)
    assert np.array_equal(out.view(np.uint32), ref.view(np.uint32))     # bit patterns: signed zeros and subnormals included
    outb = host(B.kroquant_dequantize(q, s, out_dtype=torch.bfloat16).view(torch.int16)).view(np.uint16)
    assert np.array_equal(outb, co.dequantize(q_or, s_or, out_bf16=True))
    for tokens, d in [(1, 32), (3, 96), (257, 1152), (1000, 2240)]:
        rng = np.random.default_rng(tokens)
        q_or = rng.integers(0, 256, (tokens, d // 2), dtype=np.uint8)
        s_or = rng.integers(100, 150, (tokens, d // 32), dtype=np.uint8)
        q, s = torch.from_numpy(q_or).cuda(), torch.from_numpy(s_or).cuda()
        guard = torch.full((tokens * d + 64,), -7.0, dtype=torch.float32, device="cuda")
        out = guard[32:32 + tokens * d].view(tokens, d)                 # 128-byte offset: canaries on both sides
        B.kroquant_dequantize(q, s, out=out)
        assert np.array_equal(host(out).view(np.uint32), co.dequantize(q_or, s_or).view(np.uint32))
        assert (guard[:32] == -7.0).all() and (guard[32 + tokens * d:] == -7.0).all()
        out4 = guard[4:4 + tokens * d].view(tokens, d)                  # 16-byte but not 32-byte aligned: the narrow stores
        B.kroquant_dequantize(q, s, out=out4)
        assert np.array_equal(host(out4).view(np.uint32), co.dequantize(q_or, s_or).view(np.uint32))


def test_dequantize(B):
    Xb = W.gen_activations(spec(200, 1152, seed=6))
    G = W.gen_factors(6)
    q_or, s_or, _ = co.quantize(Xb, G)
    q, s = torch.from_numpy(q_or).cuda(), torch.from_numpy(s_or).cuda()
    # without factors: exact
    out = host(B.kroquant_dequantize(q, s))
    assert np.array_equal(out, co.dequantize(q_or, s_or))
    outb = host(B.kroquant_dequantize(q, s, out_dtype=torch.bfloat16).view(torch.int16)).view(np.uint16)
    assert np.array_equal(outb, co.dequantize(q_or, s_or, out_bf16=True))
    # with factors: fp32 butterfly vs fp64 oracle
    f = B.Factors.create(G)
    ref = co.dequantize(q_or, s_or, G)
    got = host(B.kroquant_dequantize(q, s, f))
    scale = np.abs(ref.reshape(200, 36, 32)).max(axis=2, keepdims=True).repeat(32, 2).reshape(ref.shape)
    assert (np.abs(got - ref) <= 1e-5 * np.maximum(np.abs(ref), scale / 32)).all()
    gotb = W.bf16_bits_to_f32(host(B.kroquant_dequantize(q, s, f, out_dtype=torch.bfloat16)
                                   .view(torch.int16)).view(np.uint16))
    assert (np.abs(gotb - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-5 * scale).all()
    # per-block inverse
    Gb = W.gen_factors(6, n_sets=36)
    qb, sb, _ = co.quantize(Xb, Gb)
    fb = B.Factors.create(Gb)
    refb = co.dequantize(qb, sb, Gb)
    gotp = host(B.kroquant_dequantize(torch.from_numpy(qb).cuda(), torch.from_numpy(sb).cuda(), fb))
    scale = np.abs(refb.reshape(200, 36, 32)).max(axis=2, keepdims=True).repeat(32, 2).reshape(refb.shape)
    assert (np.abs(gotp - refb) <= 1e-5 * np.maximum(np.abs(refb), scale / 32)).all()
    # special scale bytes: 0 (2^-127, subnormal) and 254
    codes = np.arange(16, dtype=np.uint8)
    qq = np.zeros((2, 16), np.uint8)
    qq[:, :8] = codes[0::2] | (codes[1::2] << 4)
    ss = np.array([[0], [254]], np.uint8)
    got = host(B.kroquant_dequantize(torch.from_numpy(qq).cuda(), torch.from_numpy(ss).cuda()))
    assert np.array_equal(got, co.dequantize(qq, ss))


# ---- argument validation: status codes, nothing launched ----------------------------------
def test_error_codes(B):
    import ctypes as C
    L = B.load_library()
    X = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    q = torch.zeros((4, 32), dtype=torch.uint8, device="cuda")
    s = torch.zeros((4, 2), dtype=torch.uint8, device="cuda")
    f = B.Factors.create(W.gen_factors(0))
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    px, pq, ps = (C.c_void_p(t.data_ptr()) for t in (X, q, s))
    n0 = B.kroquant_launch_count()
    assert L.kroquant_quantize(None, 4, 64, f._h, pq, ps, st) == 1
    assert L.kroquant_quantize(px, 4, 64, None, pq, ps, st) == 1
    assert L.kroquant_quantize(px, 4, 48, f._h, pq, ps, st) == 2
    assert L.kroquant_quantize(px, -1, 64, f._h, pq, ps, st) == 2
    assert L.kroquant_quantize(px, 4, 0, f._h, pq, ps, st) == 2
    assert L.kroquant_quantize(C.c_void_p(X.data_ptr() + 2), 4, 64, f._h, pq, ps, st) == 3
    f3 = B.Factors.create(W.gen_factors(0, n_sets=3))
    assert L.kroquant_quantize(px, 4, 64, f3._h, pq, ps, st) == 4
    assert L.kroquant_quantize_path(px, 4, 64, f._h, pq, ps, 7, st) == 5
    assert L.kroquant_quantize(px, 0, 64, f._h, pq, ps, st) == 0            # empty input: ok, no launch
    # tiled scale bytes leave by 16-byte vector stores: a misaligned buffer is refused, never launched
    big = torch.zeros(4096 + 16, dtype=torch.uint8, device="cuda")
    ps_odd = C.c_void_p(big.data_ptr() + 4)
    pat = C.c_void_p(torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda").data_ptr())
    f2 = B.Factors.create(W.gen_factors(0, n_sets=2))
    for h in (f._h, f2._h):
        assert L.kroquant_quantize_ex(px, 0, 4, 64, h, pq, ps_odd, 1, 0, st) == 3
        assert L.kroquant_quantize_dual(px, 0, 4, 64, h, pq, ps_odd, 1, pat, st) == 3
    assert L.kroquant_mxfp4_quantize_ex(px, 0, 4, 64, pq, ps_odd, 1, st) == 3
    assert B.kroquant_launch_count() == n0
    assert L.kroquant_quantize_ex(px, 0, 4, 64, f._h, pq, ps_odd, 0, 0, st) == 0     # row-major scales: any address
    torch.cuda.synchronize()
    assert B.kroquant_launch_count() == n0 + 1
    n0 += 1
    bad = W.gen_factors(0)
    bad[0, 2] = np.array([[1, 2], [2, 4]], np.float32)                       # singular
    with pytest.raises(B.KroQuantError) as e:
        B.Factors.create(bad)
    assert e.value.status == 4
    bad[0, 2] = np.array([[1, np.inf], [0, 1]], np.float32)
    with pytest.raises(B.KroQuantError):
        B.Factors.create(bad)
    abc = W.hadamard_lu_params(1)
    abc[0, 0, 0] = 0.0
    with pytest.raises(B.KroQuantError):
        B.Factors.create_lu(abc)
    assert L.kroquant_quantize(px, 4, 64, f._h, pq, ps, st) == 0
    assert B.kroquant_launch_count() == n0 + 1
    torch.cuda.synchronize()


def test_host_buffer_entry_point_equals_device_path(B):
    """kroquant_quantize_host: pinned host tensors in and out through caller-owned device work buffers, one C call."""
    Xb = W.gen_activations(spec(300, 1152, seed=12))
    f = B.Factors.create(W.gen_factors(12))
    X = dev_bf16(Xb)
    q_ref, s_ref = B.kroquant_quantize(X, f)
    hx = torch.from_numpy(Xb.view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    hq = torch.empty((300, 576), dtype=torch.uint8).pin_memory()
    hs = torch.empty((300, 36), dtype=torch.uint8).pin_memory()
    xw, qw, sw = torch.empty_like(X), torch.empty_like(q_ref), torch.empty_like(s_ref)
    st = torch.cuda.Stream()
    n0 = B.kroquant_launch_count()
    for _ in range(2):
        B.kroquant_quantize_host(hx, f, hq, hs, xw, qw, sw, stream=st)
    st.synchronize()
    assert B.kroquant_launch_count() == n0 + 2
    assert np.array_equal(hq.numpy(), host(q_ref)) and np.array_equal(hs.numpy(), host(s_ref))


@pytest.mark.parametrize("tokens,d", [(3, 1152), (257, 96), (640, 1152), (2048, 2240)])
def test_grid_stride_comparison_kernels_bit_exact(B, tokens, d):
    """The plain grid-stride kernels (tuning field compare_staged = 0; also the fall-back for a multiplier vector
    that does not fit shared memory) give the same bits as the staged ones and as the oracle."""
    Xb = W.gen_activations(spec(tokens, d, seed=31))
    sv = W.gen_channel_scales(31, d)
    X, svd = dev_bf16(Xb), torch.from_numpy(sv).cuda()
    qs, ss = B.kroquant_scale_quantize(X, svd)
    qp, sp = B.kroquant_mxfp4_quantize(X)
    plain = B.Tuning(compare_staged=0)
    qs0, ss0 = B.kroquant_scale_quantize(X, svd, tuning=plain)
    qp0, sp0 = B.kroquant_mxfp4_quantize(X, tuning=plain)
    assert torch.equal(qs, qs0) and torch.equal(ss, ss0) and torch.equal(qp, qp0) and torch.equal(sp, sp0)
    q_or, s_or, Y = co.scale_quantize(Xb, sv)
    P.check_codes(host(qs0), host(ss0), q_or, s_or, Y, exact=True)


def test_scale_vector_too_long_for_shared_memory_falls_back(B):
    # d = 20480: 80 KB of multipliers do not fit beside the stages: the grid-stride kernel serves the call
    tokens, d = 64, 20480
    Xb = W.gen_activations(spec(tokens, d, seed=32))
    sv = W.gen_channel_scales(32, d)
    q, s = B.kroquant_scale_quantize(dev_bf16(Xb), torch.from_numpy(sv).cuda())
    q_or, s_or, Y = co.scale_quantize(Xb, sv)
    P.check_codes(host(q), host(s), q_or, s_or, Y, exact=True)
    assert B.kroquant_last_device_error() == 0
