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
    return binding


def dev(bits):
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def spec(tokens, d, seed):
    return W.ActivationSpec(f"dist{tokens}x{d}", tokens, d, seed=seed, outlier_channels=max(1, d // 100),
                            outlier_gain=50.0, spike_rows=min(2, tokens), spike_gain=8.0)


# (dynamic, unit_tiles, trigger, prefetch_tiles, ctas_per_sm, config); unit_tiles 0 and ctas_per_sm 0: automatic
MODES = [(False, 1, 1, 0, 3, 5), (False, 3, 2, 4, 3, 5), (False, 2, 0, 1, 2, 5), (True, 1, 2, 2, 3, 5), (True, 2, 1, 0, 3, 5),
         (True, 4, 0, 3, 2, 5), (True, 1, 2, 1, 4, 5), (True, 16, 2, 64, 1, 5), (True, 0, 2, 4, 0, 2), (True, 3, 2, 4, 2, 2),
         (False, 1, 1, 0, 2, 2), (True, 5, 1, 2, 2, 1)]


def tuning_of(B, mode):
    """The per-call tuning struct of a mode: nothing in the library is changed for anybody else."""
    dyn, unit, trigger, prefetch, cps, cfg = mode
    return B.Tuning(config=cfg, ctas_per_sm=cps, use_pdl=1, trigger=trigger, prefetch_tiles=prefetch, dynamic=dyn, unit_tiles=unit)


# 4608 x 3072: 3456 tiles (7 to 8 per CTA of a 444-CTA grid); 2500 x 2240: ragged last tile; 700 x 5600 per block
@pytest.mark.parametrize("tokens,d,per_block", [(4608, 3072, False), (2500, 2240, False), (700, 5600, True),
                                                (1200, 1152, True), (129, 64, False)])
def test_every_mode_gives_the_same_bits(B, tokens, d, per_block):
    Xb = W.gen_activations(spec(tokens, d, tokens + d))
    X = dev(Xb)
    f = B.Factors.create(W.gen_factors(7, n_sets=d // 32 if per_block else 1))
    ref = None
    for mode in MODES:
        tn = tuning_of(B, mode)
        for layout in ("rowmajor", "tiled"):
            outs = [B.kroquant_quantize(X, f, path="tensor", scale_layout=layout, tuning=tn) for _ in range(3)]   # back to back
            dual = B.kroquant_quantize_dual(X, f, scale_layout=layout, tuning=tn)
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
    tn = tuning_of(B, mode)
    X, f = dev(Xb), B.Factors.create(G)
    q, s = B.kroquant_quantize(X, f, path="tensor", tuning=tn)
    Yg = B.kroquant_transform_f32(X, f, path="tensor", tuning=tn)
    qo, so, Y = co.quantize(Xb, G)
    P.check_values(Yg.cpu().numpy(), Y)
    P.check_codes(q.cpu().numpy(), s.cpu().numpy(), qo, so, Y, exact=False)
    assert B.kroquant_last_device_error() == 0


def test_dynamic_launches_that_overlap_on_two_streams(B):
    """A running CTA may only take over CTAs of its own grid: two dynamic launches that share the GPU must
    each produce their own complete result."""
    tn = tuning_of(B, MODES[3])
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
                outs[i].append(B.kroquant_quantize(X[i], f[i], path="tensor", stream=streams[i], tuning=tn))
    torch.cuda.synchronize()
    for i in range(2):
        for q, s in outs[i]:
            assert torch.equal(q, ref[i][0]) and torch.equal(s, ref[i][1])
    assert B.kroquant_last_device_error() == 0


def test_tuning_ranges_and_scope(B):
    X = dev(W.gen_activations(spec(64, 64, 3)))
    f = B.Factors.create(W.gen_factors(3))
    n0 = B.kroquant_launch_count()
    for bad in [dict(trigger=-1), dict(trigger=3), dict(prefetch_tiles=-1), dict(prefetch_tiles=65), dict(unit_tiles=-1),
                dict(unit_tiles=17), dict(dynamic=2), dict(config=8), dict(ctas_per_sm=9), dict(use_pdl=2), dict(compare_staged=-1)]:
        with pytest.raises(RuntimeError):
            B.kroquant_quantize(X, f, tuning=B.Tuning(**bad))
    assert B.kroquant_launch_count() == n0                     # refused: nothing launched
    # a tuned call leaves no trace: the next plain call runs with the defaults and gives the same bits
    a = B.kroquant_quantize(X, f, tuning=B.Tuning(dynamic=0, unit_tiles=1, ctas_per_sm=1, config=3, use_pdl=0))
    b = B.kroquant_quantize(X, f)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
