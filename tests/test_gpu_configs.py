"""GPU parity at the full sizes of the five workload configs, in the launch configuration
the bench times (default tensor-core path, default grid).  Tensors up to FLUX size are
compared whole in one piece, the sweep points whole in chunks of 2048 token rows."""
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


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def whole(B, spec, G, exact=False, check_y=True):
    Xb = W.gen_activations(spec)
    X = dev_bf16(Xb)
    f = B.Factors.create(G)
    q, s = B.kroquant_quantize(X, f)
    q_or, s_or, Y = co.quantize(Xb, G)
    r = P.check_codes(q.cpu().numpy(), s.cpu().numpy(), q_or, s_or, Y, exact=exact)
    if check_y:
        Yg = B.kroquant_transform_f32(X, f)
        r.update(P.check_values(Yg.cpu().numpy(), Y))
        del Yg
    assert B.kroquant_last_device_error() == 0
    # comparison kernels on the same input: bit exact
    sv = W.gen_channel_scales(spec.seed, spec.d)
    q2, s2 = B.kroquant_scale_quantize(X, torch.from_numpy(sv).cuda())
    qo, so, Yo = co.scale_quantize(Xb, sv)
    P.check_codes(q2.cpu().numpy(), s2.cpu().numpy(), qo, so, Yo, exact=True)
    q3, s3 = B.kroquant_mxfp4_quantize(X)
    qo, so, Yo = co.plain_quantize(Xb)
    P.check_codes(q3.cpu().numpy(), s3.cpu().numpy(), qo, so, Yo, exact=True)
    return r


def test_config_tiny(B):
    print(whole(B, W.tiny_spec(), W.gen_factors(0)))


@pytest.mark.parametrize("i", [0, 1])
def test_config_pixart(B, i):
    sp = W.pixart_specs()[i]
    print(sp.name, whole(B, sp, W.gen_factors(1, layer=i)))


@pytest.mark.parametrize("i", [0, 1])
@pytest.mark.parametrize("per_block", [False, True])
def test_config_sana(B, i, per_block):
    sp = W.sana_specs()[i]
    G = W.gen_factors(2, n_sets=sp.d // 32 if per_block else 1, layer=i)
    print(sp.name, per_block, whole(B, sp, G))


@pytest.mark.parametrize("i", [0, 1])
def test_config_flux(B, i):
    sp = W.flux_specs()[i]
    print(sp.name, whole(B, sp, W.gen_factors(3, layer=i), check_y=(i == 0)))


@pytest.mark.parametrize("tokens,d", [(1024, 1152), (16384, 2240), (65536, 3072), (16384, 12288)])
def test_config_sweep_whole_tensor(B, tokens, d):
    """Sweep points: the generator runs on the host once; EVERY row goes through the oracle, in chunks of 2048 rows so
    that host memory stays bounded; the comparison kernels are checked the same way (bit exact)."""
    sp = W.sweep_spec(tokens, d)
    Xb = W.gen_activations(sp)
    G = W.gen_factors(4)
    X = dev_bf16(Xb)
    f = B.Factors.create(G)
    q, s = B.kroquant_quantize(X, f)
    r = P.check_codes_chunked(q, s, lambda r0, r1: Xb[r0:r1], lambda b: co.quantize(b, G), tokens, exact=False)
    sv = W.gen_channel_scales(4, d)
    q2, s2 = B.kroquant_scale_quantize(X, torch.from_numpy(sv).cuda())
    P.check_codes_chunked(q2, s2, lambda r0, r1: Xb[r0:r1], lambda b: co.scale_quantize(b, sv), tokens, exact=True)
    q3, s3 = B.kroquant_mxfp4_quantize(X)
    P.check_codes_chunked(q3, s3, lambda r0, r1: Xb[r0:r1], co.plain_quantize, tokens, exact=True)
    # properties that hold at any size: every scale byte follows from the decoded block maximum
    # (a non-zero block always holds a code 6 or 7)
    codes = torch.maximum(q & 7, (q >> 4) & 7).view(tokens, d // 32, 16).amax(dim=2)
    assert bool(((codes >= 6) | (s == 0)).all())
    assert B.kroquant_last_device_error() == 0
    print(sp.name, r)


def test_largest_sweep_point_generated_on_device(B):
    """X[65536, 12288] (1.6 GB) is drawn on the device with torch's seeded generator (the host generator would
    need > 10 GB of temporaries) and read back 2048 rows at a time: every row goes through the oracle.  Same
    structure as the sweep recipe: N(0,1), 12 outlier channels x50, 4 spike rows x8."""
    tokens, d = 65536, 12288
    g = torch.Generator(device="cuda").manual_seed(4)
    X = torch.empty((tokens, d), dtype=torch.bfloat16, device="cuda")
    for r0 in range(0, tokens, 8192):
        blk = torch.randn((8192, d), generator=g, device="cuda")
        blk[:, torch.arange(12, device="cuda") * 1000 + 7] *= 50.0
        X[r0:r0 + 8192] = blk.to(torch.bfloat16)
    X[torch.tensor([5, 4099, 30000, 65535], device="cuda")] *= 8.0
    G = W.gen_factors(4)
    f = B.Factors.create(G)
    q, s = B.kroquant_quantize(X, f)

    def rows(r0, r1):
        return X[r0:r1].view(torch.int16).cpu().numpy().view(np.uint16)

    print(P.check_codes_chunked(q, s, rows, lambda b: co.quantize(b, G), tokens, exact=False))
    assert B.kroquant_last_device_error() == 0
