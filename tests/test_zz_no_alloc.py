"""kroquant_block_grad_static: the block-gradient reduction for callers that cannot allocate.

Some users of the C ABI have no device memory to hand over as scratch: the memory was claimed up
front by a framework's pool, an allocation would stall a latency-bound loop, or the host program has
no allocator at all.  For them the library carries its own fixed scratch array.  This file checks that
entry point against kroquant_block_grad (the one that takes a caller-supplied scratch buffer), twice in
a row because all calls share the array and the second call finds the first one's leftovers in it.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import calib_oracle as co
from paper_2607_21446_b200 import binding as kb
from paper_2607_21446_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _inputs(rows, d, seed):
    rng = np.random.default_rng(seed)
    X_bits = wl.gen_activations(wl.calib_spec(rows, d, seed))
    G = rng.standard_normal((rows, d)).astype(np.float32)
    dev = torch.device("cuda:0")
    X_t = torch.from_numpy(X_bits.view(np.int16)).to(dev).view(torch.bfloat16)
    return X_bits, G, X_t, torch.from_numpy(G).to(dev)


@pytest.mark.parametrize("shared", [True, False])
def test_static_scratch_matches_caller_scratch_on_two_calls_in_a_row(shared):
    L = kb.load_library()
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    # two different problems back to back: the second reuses the array the first one filled,
    # with a different number of partial blocks
    for rows, d, seed in ((1000, 256, 91), (4104, 1152, 92)):
        n_sets = 1 if shared else d // 32
        X_bits, G, X_t, G_t = _inputs(rows, d, seed)
        expect = kb.kroquant_block_grad(X_t, G_t, n_sets)          # existing entry point
        out = torch.full((n_sets, 32, 32), float("nan"), dtype=torch.float32, device=X_t.device)
        # straight through the C ABI: plain pointers and sizes
        rc = L.kroquant_block_grad_static(C.c_void_p(X_t.data_ptr()), C.c_void_p(G_t.data_ptr()), rows, d, n_sets,
                                          C.c_void_p(out.data_ptr()), stream)
        assert rc == 0, kb.status_string(rc)
        torch.cuda.synchronize()
        got, want = out.cpu().numpy(), expect.cpu().numpy()
        # same kernels, same chunking, fixed summation order: identical, and within the tolerance the
        # oracle comparison of kroquant_block_grad uses
        X = wl.bf16_bits_to_f32(X_bits).astype(np.float64)
        bound = 1e-5 * (np.abs(X).T @ np.abs(G).astype(np.float64)).max()
        assert np.abs(got - want).max() <= bound
        assert np.array_equal(got, want)
        assert np.abs(got - co._block_grads(X, G.astype(np.float64), n_sets)).max() <= bound
        # and once more on the same inputs through the Python wrapper
        out2 = torch.empty_like(out)
        kb.kroquant_block_grad_static(X_t, G_t, n_sets, out2)
        torch.cuda.synchronize()
        assert np.array_equal(out2.cpu().numpy(), want)
    assert kb.kroquant_last_device_error() == 0


def test_static_scratch_refuses_what_does_not_fit_and_handles_empty_input():
    L = kb.load_library()
    dev = torch.device("cuda:0")
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    # d/32 = 2080 partial blocks even with a single chunk of rows: larger than the built-in 2048
    rows, d = 8, 66560
    X = torch.zeros((rows, d), dtype=torch.bfloat16, device=dev)
    G = torch.zeros((rows, d), dtype=torch.float32, device=dev)
    out = torch.zeros((1, 32, 32), dtype=torch.float32, device=dev)
    before = kb.kroquant_launch_count()
    rc = L.kroquant_block_grad_static(C.c_void_p(X.data_ptr()), C.c_void_p(G.data_ptr()), rows, d, 1,
                                      C.c_void_p(out.data_ptr()), stream)
    assert rc == 5 and "unsupported" in kb.status_string(rc).lower()
    assert kb.kroquant_launch_count() == before                     # nothing was launched
    # no rows: zeros, no kernel
    out.fill_(7.0)
    rc = L.kroquant_block_grad_static(None, None, 0, 64, 1, C.c_void_p(out.data_ptr()), stream)
    assert rc == 0
    torch.cuda.synchronize()
    assert float(out.abs().max()) == 0.0
    # bad arguments
    assert L.kroquant_block_grad_static(C.c_void_p(X.data_ptr()), C.c_void_p(G.data_ptr()), 8, 48, 1,
                                        C.c_void_p(out.data_ptr()), stream) == 2      # d % 32
    assert L.kroquant_block_grad_static(C.c_void_p(X.data_ptr()), C.c_void_p(G.data_ptr()), 8, 64, 3,
                                        C.c_void_p(out.data_ptr()), stream) == 4      # n_sets
