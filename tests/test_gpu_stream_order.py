"""Stream order behind the quantizer's programmatic launches.

The quantizer kernels are launched with programmatic stream serialization and signal launch completion at
their start.  A consumer in the same stream must still see complete outputs.  The hard case is a short
quantizer call queued behind a long one (so that it really starts early) followed at once by a consumer;
the consumers here are this library's own GEMM kernels (cluster launches), the one-call layer, and an
ordinary framework kernel.
"""
import numpy as np
import pytest
import torch

from paper_2607_21446_b200 import binding as kb
from paper_2607_21446_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def long_call():
    """A quantizer call that runs for a few hundred microseconds."""
    g = torch.Generator(device="cuda")
    g.manual_seed(0)
    big = torch.randn(32768, 12288, device="cuda", generator=g).to(torch.bfloat16)
    f = kb.Factors.create(wl.gen_factors(3, 1))
    q = torch.empty((32768, 12288 // 2), dtype=torch.uint8, device="cuda")
    s = torch.empty((32768, 12288 // 32), dtype=torch.uint8, device="cuda")
    yield lambda: kb.kroquant_quantize(big, f, q, s)
    f.destroy()


@pytest.mark.parametrize("pair", [True, False])
def test_own_gemms_behind_a_chain_of_quantizer_calls(long_call, pair):
    kb.set_gemm_pair(pair)
    try:
        t, d, r, o = 256, 1024, 128, 256
        g = torch.Generator(device="cuda")
        g.manual_seed(1)
        xs = [torch.randn(t, d, device="cuda", generator=g).to(torch.bfloat16) for _ in range(3)]
        R = torch.randn(r, d, device="cuda", generator=g).to(torch.bfloat16)
        Wt = torch.randn(o, d, device="cuda", generator=g).to(torch.bfloat16)
        qw, sw = kb.kroquant_mxfp4_quantize(Wt, scale_layout="tiled")
        f = kb.Factors.create(wl.gen_factors(3, 1, layer=1))
        layer = kb.LinearW4A4(kb.Factors.create(wl.gen_factors(3, 1, layer=1)), qw, sw)
        refs = []
        for x in xs:
            qa, sa, AT = kb.kroquant_quantize_dual(x, f, scale_layout="tiled")
            torch.cuda.synchronize()
            refs.append((kb.kroquant_gemm_bf16(AT, R, out_dtype=torch.float32).clone(),
                         kb.kroquant_gemm_mxfp4(qa, sa, qw, sw, out_dtype=torch.float32).clone(), qa.clone()))
            torch.cuda.synchronize()
        for rep in range(12):
            i = rep % 3
            AT = torch.zeros((t, d), dtype=torch.bfloat16, device="cuda")
            qa = torch.zeros((t, d // 2), dtype=torch.uint8, device="cuda")
            sa = torch.zeros(kb.tiled_scale_bytes(t, d), dtype=torch.uint8, device="cuda")
            torch.cuda.synchronize()
            long_call()                                                        # keeps the GPU busy
            kb.kroquant_quantize_dual(xs[i], f, qa, sa, AT, scale_layout="tiled")   # starts early, waits inside
            low = kb.kroquant_gemm_bf16(AT, R, out_dtype=torch.float32)             # consumers, queued at once
            main = kb.kroquant_gemm_mxfp4(qa, sa, qw, sw, out_dtype=torch.float32)
            copy = qa.clone()                                                  # an ordinary framework kernel
            long_call()
            whole = layer(xs[i], out_dtype=torch.float32)                      # quantizer + GEMM behind a long call
            torch.cuda.synchronize()
            assert torch.equal(low, refs[i][0]), rep
            assert torch.equal(main, refs[i][1]), rep
            assert torch.equal(copy, refs[i][2]), rep
            assert torch.equal(whole, refs[i][1]), rep
        assert kb.kroquant_last_device_error() == 0
        f.destroy()
    finally:
        kb.set_gemm_pair(True)
