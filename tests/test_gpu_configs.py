"""GPU parity at the full sizes of the five workload configs, in the launch configuration
the bench times (default tensor-core path, default grid).  Tensors up to FLUX size are
compared whole; the largest sweep point is compared on sampled token rows."""
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
def test_config_sweep_sampled_rows(B, tokens, d):
    """Sweep points: the generator runs on the host once; the oracle checks 256 sampled
    token rows (all of their blocks), plus the first and the last row."""
    sp = W.sweep_spec(tokens, d)
    Xb = W.gen_activations(sp)
    G = W.gen_factors(4)
    X = dev_bf16(Xb)
    f = B.Factors.create(G)
    q, s = B.kroquant_quantize(X, f)
    rng = np.random.default_rng(1)
    rows = np.unique(np.concatenate([[0, tokens - 1], rng.choice(tokens, 256, replace=False)]))
    q_or, s_or, Y = co.quantize(Xb[rows], G)
    ridx = torch.from_numpy(rows).cuda()
    r = P.check_codes(q[ridx].cpu().numpy(), s[ridx].cpu().numpy(), q_or, s_or, Y, exact=False)
    # properties that hold at any size: every scale byte follows from the decoded block maximum
    # (a non-zero block always holds a code 6 or 7), and identity factors give the bare encoder
    codes = torch.maximum(q & 7, (q >> 4) & 7).view(tokens, d // 32, 16).amax(dim=2)
    assert bool(((codes >= 6) | (s == 0)).all())
    fi = B.Factors.create(W.identity_factors(1))
    qa, sa = B.kroquant_quantize(X, fi, path="tensor")
    qb, sb = B.kroquant_mxfp4_quantize(X)
    assert torch.equal(sa, sb)
    diff = qa != qb                                  # only signed zeros may differ
    if bool(diff.any()):
        a, b = qa[diff], qb[diff]
        x = a ^ b
        assert bool(((x & 0x77) == 0).all())                       # magnitudes agree
        assert bool((((x & 0x08) == 0) | ((a & 0x07) == 0)).all())  # a flipped sign only on a zero
        assert bool((((x & 0x80) == 0) | ((a & 0x70) == 0)).all())
    assert B.kroquant_last_device_error() == 0
    print(sp.name, r)


def test_largest_sweep_point_generated_on_device(B):
    """X[65536, 12288] (1.6 GB) is drawn on the device with torch's seeded generator (the
    host generator would need > 10 GB of temporaries); 192 sampled rows go back to the host
    and through the oracle.  Same structure as the sweep recipe: N(0,1), 12 outlier
    channels x50, 4 spike rows x8."""
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
    rows = np.unique(np.concatenate([[0, 5, 65535], np.random.default_rng(2).choice(tokens, 189, replace=False)]))
    ridx = torch.from_numpy(rows).cuda()
    Xb = X[ridx].view(torch.int16).cpu().numpy().view(np.uint16)
    q_or, s_or, Y = co.quantize(Xb, G)
    print(P.check_codes(q[ridx].cpu().numpy(), s[ridx].cpu().numpy(), q_or, s_or, Y, exact=False))
    assert B.kroquant_last_device_error() == 0
