"""The tensor-core quantizer's work distribution and kernel-boundary settings change nothing in the results.

Static strides or hardware-assisted dynamic distribution (running CTAs take over the units of CTAs that have
not started), any unit size, any trigger point of the programmatic launch and any L2 prefetch depth must give
bit-identical codes and scales; one setting of each kind is also checked against the oracle on shapes whose
CTAs own several tiles each (the other parity tests mostly have one tile per CTA)."""
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
    yield binding
    binding.kroquant_debug_set_distribution(True, 0)         # back to the library's own choices
    binding.kroquant_debug_set_boundary(2, 4)
    binding.kroquant_debug_set_umma_config(2, 0, True)


def dev(bits):
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def spec(tokens, d, seed):
    return W.ActivationSpec(f"dist{tokens}x{d}", tokens, d, seed=seed, outlier_channels=max(1, d // 100),
                            outlier_gain=50.0, spike_rows=min(2, tokens), spike_gain=8.0)


# (dynamic, unit_tiles, trigger, prefetch_tiles, ctas_per_sm, config); unit_tiles 0 and ctas_per_sm 0: automatic
MODES = [(False, 1, 1, 0, 3, 5), (False, 3, 2, 4, 3, 5), (False, 2, 0, 1, 2, 5), (True, 1, 2, 2, 3, 5), (True, 2, 1, 0, 3, 5),
         (True, 4, 0, 3, 2, 5), (True, 1, 2, 1, 4, 5), (True, 16, 2, 64, 1, 5), (True, 0, 2, 4, 0, 2), (True, 3, 2, 4, 2, 2),
         (False, 1, 1, 0, 2, 2), (True, 5, 1, 2, 2, 1)]


def set_mode(B, mode):
    dyn, unit, trigger, prefetch, cps, cfg = mode
    B.kroquant_debug_set_umma_config(cfg, cps, True)
    B.kroquant_debug_set_boundary(trigger, prefetch)
    B.kroquant_debug_set_distribution(dyn, unit)


# 4608 x 3072: 3456 tiles (7 to 8 per CTA of a 444-CTA grid); 2500 x 2240: ragged last tile; 700 x 5600 per block
@pytest.mark.parametrize("tokens,d,per_block", [(4608, 3072, False), (2500, 2240, False), (700, 5600, True),
                                                (1200, 1152, True), (129, 64, False)])
def test_every_mode_gives_the_same_bits(B, tokens, d, per_block):
    Xb = W.gen_activations(spec(tokens, d, tokens + d))
    X = dev(Xb)
    f = B.Factors.create(W.gen_factors(7, n_sets=d // 32 if per_block else 1))
    ref = None
    for mode in MODES:
        set_mode(B, mode)
        for layout in ("rowmajor", "tiled"):
            outs = [B.kroquant_quantize(X, f, path="tensor", scale_layout=layout) for _ in range(3)]   # back to back
            dual = B.kroquant_quantize_dual(X, f, scale_layout=layout)
            got = [t.clone() for t in outs[-1]] + [dual[2].clone()]
            for q, s in outs[:-1]:
                assert torch.equal(q, got[0]) and torch.equal(s, got[1])
            assert torch.equal(dual[0], got[0]) and torch.equal(dual[1], got[1])
            if ref is None:
                ref = {}
            if layout not in ref:
                ref[layout] = got
            else:
                for a, b in zip(ref[layout], got):
                    assert torch.equal(a, b), (mode, layout)
        assert B.kroquant_last_device_error() == 0, mode


@pytest.mark.parametrize("mode", [MODES[0], MODES[3], MODES[5], MODES[8], MODES[9]])
def test_multi_tile_ctas_against_the_oracle(B, mode):
    tokens, d = 1500, 3072           # 1125 tiles: 2 to 3 per CTA of a 444-CTA grid, ragged last tile
    Xb = W.gen_activations(spec(tokens, d, 11))
    G = W.gen_factors(11)
    set_mode(B, mode)
    X, f = dev(Xb), B.Factors.create(G)
    q, s = B.kroquant_quantize(X, f, path="tensor")
    Yg = B.kroquant_transform_f32(X, f, path="tensor")
    qo, so, Y = co.quantize(Xb, G)
    P.check_values(Yg.cpu().numpy(), Y)
    P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=False)
    assert B.kroquant_last_device_error() == 0


def test_dynamic_launches_that_overlap_on_two_streams(B):
    """A running CTA may only take over CTAs of its own grid: two dynamic launches that share the GPU must
    each produce their own complete result."""
    set_mode(B, MODES[3])
    shapes = [(4608, 3072), (3000, 2240)]
    X = [dev(W.gen_activations(spec(t, d, 40 + i))) for i, (t, d) in enumerate(shapes)]
    f = [B.Factors.create(W.gen_factors(50 + i)) for i in range(2)]
    ref = [B.kroquant_quantize(X[i], f[i], path="tensor") for i in range(2)]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in range(2)]
    outs = [[], []]
    for rep in range(12):
        for i in range(2):
            with torch.cuda.stream(streams[i]):
                outs[i].append(B.kroquant_quantize(X[i], f[i], path="tensor", stream=streams[i]))
    torch.cuda.synchronize()
    for i in range(2):
        for q, s in outs[i]:
            assert torch.equal(q, ref[i][0]) and torch.equal(s, ref[i][1])
    assert B.kroquant_last_device_error() == 0


def test_knob_ranges(B):
    for args in [(-1, 0), (3, 0), (0, -1), (0, 65)]:
        with pytest.raises(RuntimeError):
            B.kroquant_debug_set_boundary(*args)
    for args in [(True, -1), (True, 17)]:
        with pytest.raises(RuntimeError):
            B.kroquant_debug_set_distribution(*args)
