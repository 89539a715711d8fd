"""The give-up path of the kernels' bounded waits, exercised without a fault or a hang: in the diagnostic build of
the library one CTA withholds the arrival of its first tile (a flag that nothing sets), the waits on it run out after
20 ms, and the kernel must come back with an error code, a usable context and complete outputs everywhere else."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r"""
import sys, time
sys.path.insert(0, %r)
import numpy as np, torch
from paper_2607_21446_b200 import binding as B, build as kbuild, workloads as W
B.use_library(kbuild.build_timeline())
Xb = W.gen_activations(W.tiny_spec())
X = torch.from_numpy(Xb.view(np.int16)).cuda().view(torch.bfloat16)
f = B.Factors.create(W.gen_factors(0))
q_ref, s_ref = B.kroquant_quantize(X, f, path="tensor")
torch.cuda.synchronize()
assert B.kroquant_last_device_error() == 0
B.kroquant_debug_withhold_arrival(True)
t0 = time.perf_counter()
q, s = B.kroquant_quantize(X, f, path="tensor")
torch.cuda.synchronize()                       # returns: every wait is bounded
dt = time.perf_counter() - t0
err = B.kroquant_last_device_error()
B.kroquant_debug_withhold_arrival(False)
assert err == 2, err                           # KQ_DEV_TIMEOUT_MMA_FULL: the MMA warp gave up on the withheld tile
assert 0.015 < dt < 5.0, dt
# every tile but the withheld one (CTA 0's: flat rows 0..127) is complete
assert torch.equal(q.view(-1, 16)[128:], q_ref.view(-1, 16)[128:]) and torch.equal(s.view(-1)[128:], s_ref.view(-1)[128:])
# the context is usable and the error word was cleared by the read
q2, s2 = B.kroquant_quantize(X, f, path="tensor")
torch.cuda.synchronize()
assert B.kroquant_last_device_error() == 0
assert torch.equal(q2, q_ref) and torch.equal(s2, s_ref)
# the comparison kernels (no tensor-core stage) leave the same way: their epilogue is the waiter (code 4)
B.kroquant_debug_withhold_arrival(True)
B.kroquant_mxfp4_quantize(X)
torch.cuda.synchronize()
err = B.kroquant_last_device_error()
B.kroquant_debug_withhold_arrival(False)
assert err == 4, err
q3, s3 = B.kroquant_mxfp4_quantize(X)
torch.cuda.synchronize()
assert B.kroquant_last_device_error() == 0
# the kernel that builds its operand on chip (per-block sets): the builder warps wait for the withheld tile's
# announcement, the issuing warp for the tile itself, the producer for the slot to come back -- whichever limit runs
# out first reports (7, 2 or 1)
fp = B.Factors.create(W.gen_factors(0, n_sets=X.shape[1] // 32))
qk_ref, sk_ref = B.kroquant_quantize(X, fp, path="onchip")
torch.cuda.synchronize()
assert B.kroquant_last_device_error() == 0
B.kroquant_debug_withhold_arrival(True)
B.kroquant_quantize(X, fp, path="onchip")
torch.cuda.synchronize()
err = B.kroquant_last_device_error()
B.kroquant_debug_withhold_arrival(False)
assert err in (1, 2, 7), err
qk, sk = B.kroquant_quantize(X, fp, path="onchip")
torch.cuda.synchronize()
assert B.kroquant_last_device_error() == 0
assert torch.equal(qk, qk_ref) and torch.equal(sk, sk_ref)
print("ok", round(dt, 3))
""" % ROOT


def test_withheld_arrival_times_out_and_the_context_survives():
    res = subprocess.run([sys.executable, "-c", SCRIPT], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert res.returncode == 0, res.stdout[-1500:] + res.stderr[-3000:]
    assert res.stdout.strip().startswith("ok")


def test_ordinary_build_refuses_the_diagnostic_calls():
    from paper_2607_21446_b200 import binding as B
    L = B.load_library()
    assert L.kroquant_debug_withhold_arrival(1) == 5          # KQ_ERR_UNSUPPORTED
    assert L.kroquant_debug_set_timeline(None) == 5
    assert L.kroquant_debug_boundary_probe(0, 1, 1, 0, 1, None, None) == 5
