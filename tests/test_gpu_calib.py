"""Calibration loop on the GPU against the float64 oracle (Section 3.3, Appendix D).

Tolerances (derived in the design notes): the forward contraction has exact products and fp32
accumulation, the transform is fp32 FMA, so the three loss terms agree to ~1e-5 relative; codes that
sit on a rounding boundary may flip, which moves L_out by O(1/(M d)) relative.  The output error is
rounded to bf16 (2^-9 relative per element, independent signs) before the two backward contractions;
over the o M terms of a block-gradient entry that averages down to ~1e-5 of the largest component.
"""
import numpy as np
import pytest
import torch

from oracle import calib_oracle as co
from paper_2607_21446_b200 import binding as kb
from paper_2607_21446_b200 import workloads as wl

pytestmark = pytest.mark.gpu

LOSS_RTOL = 1e-4         # measured 2e-7 ... 3e-5 (largest at the Hadamard start, where values sit on ties)
GRAD_TOL = 5e-4          # of max |g|; measured 2e-6 ... 9e-5


@pytest.fixture(autouse=True, params=["pair", "single"])
def gemm_variant(request):
    """Every test runs with both tensor-core GEMM kernels: CTA pairs on 256 x 256 tiles (the default)
    and one CTA per 128 x 256 tile."""
    kb.set_gemm_pair(request.param == "pair")
    yield request.param
    kb.set_gemm_pair(True)


def _case(M, o, d, seed):
    A_bits = wl.gen_activations(wl.calib_spec(M, d, seed))
    W_bits = wl.gen_weights(seed, o, d)
    A = wl.bf16_bits_to_f32(A_bits).astype(np.float64)
    W = wl.bf16_bits_to_f32(W_bits).astype(np.float64)
    dev = torch.device("cuda:0")
    A_t = torch.from_numpy(A_bits.view(np.int16)).to(dev).view(torch.bfloat16)
    W_t = torch.from_numpy(W_bits.view(np.int16)).to(dev).view(torch.bfloat16)
    return A, W, A_t, W_t


def _no_device_error():
    code = kb.kroquant_last_device_error()
    assert code == 0, f"device error {code}"


SHAPES = [(512, 96, 320, 31), (1000, 288, 256, 32), (256, 512, 128, 33)]


@pytest.mark.parametrize("M,o,d,seed", SHAPES)
@pytest.mark.parametrize("shared", [True, False])
def test_initial_losses_and_lambdas(M, o, d, seed, shared):
    A, W, A_t, W_t = _case(M, o, d, seed)
    n_sets = 1 if shared else d // 32
    cal = kb.Calibrator(A_t, W_t, n_sets)
    lam_A, lam_W, l0 = co.auto_lambda(A, W, n_sets)
    losses, _ = cal.loss_grad(grad=False)
    assert np.allclose(losses, l0, rtol=LOSS_RTOL, atol=0), (losses, l0)
    lam = cal.lambdas
    assert np.allclose(lam, [lam_A, lam_W], rtol=2 * LOSS_RTOL)
    assert np.allclose(cal.theta, co.hadamard_theta(n_sets), rtol=1e-7)
    _no_device_error()
    cal.destroy()


@pytest.mark.parametrize("M,o,d,seed", SHAPES)
@pytest.mark.parametrize("shared", [True, False])
def test_loss_and_gradient_at_random_parameters(M, o, d, seed, shared):
    A, W, A_t, W_t = _case(M, o, d, seed)
    n_sets = 1 if shared else d // 32
    theta = wl.gen_lu_params(seed, n_sets)
    cal = kb.Calibrator(A_t, W_t, n_sets)
    cal.theta = theta
    cal.lambdas = (2.5, 40.0)
    lam = cal.lambdas.astype(np.float64)
    losses, g = cal.loss_grad()
    total, terms, g_ref = co.loss_and_grad(A, W, theta.astype(np.float64), lam[0], lam[1])
    assert np.allclose(losses, terms, rtol=LOSS_RTOL, atol=0), (losses, terms)
    scale = np.abs(g_ref).max()
    err = np.abs(g - g_ref).max()
    assert err <= GRAD_TOL * scale, (err, scale)
    # the parameters were not touched by the evaluation
    assert np.array_equal(cal.theta, theta)
    _no_device_error()
    cal.destroy()


@pytest.mark.parametrize("M,o,d,seed", [(8, 32, 32, 1), (16, 32, 64, 2), (136, 160, 96, 3), (264, 32, 4608, 4)])
@pytest.mark.parametrize("shared", [True, False])
def test_smallest_and_ragged_shapes(M, o, d, seed, shared):
    """One row tile or less, one block, d far larger than M: every tile is ragged.  With so few rows the bf16
    rounding of the output error averages over few terms, hence the wider gradient tolerance (measured
    up to 6.4e-4 at M = 16)."""
    A, W, A_t, W_t = _case(M, o, d, seed)
    n_sets = 1 if shared else d // 32
    theta = wl.gen_lu_params(seed, n_sets)
    cal = kb.Calibrator(A_t, W_t, n_sets)
    cal.theta = theta
    cal.lambdas = (2.5, 40.0)
    lam = cal.lambdas.astype(np.float64)
    losses, g = cal.loss_grad()
    _, terms, g_ref = co.loss_and_grad(A, W, theta.astype(np.float64), lam[0], lam[1])
    assert np.allclose(losses, terms, rtol=LOSS_RTOL, atol=0), (losses, terms)
    assert np.abs(g - g_ref).max() <= 2e-3 * np.abs(g_ref).max()
    _no_device_error()
    cal.destroy()


def test_gradient_of_the_regularisers_alone():
    """W = 0 makes the output term and its gradient vanish: what is left is lambda_A dL_A/dtheta,
    which involves no bf16 rounding of the output error."""
    M, o, d, seed = 512, 64, 256, 41
    A, W, A_t, W_t = _case(M, o, d, seed)
    W_t.zero_()
    W[:] = 0.0
    theta = wl.gen_lu_params(seed, 1)
    cal = kb.Calibrator(A_t, W_t, 1)
    cal.theta = theta
    cal.lambdas = (1.0, 0.0)
    losses, g = cal.loss_grad()
    _, terms, g_ref = co.loss_and_grad(A, W, theta.astype(np.float64), 1.0, 0.0)
    assert losses[0] == 0.0 and terms[0] == 0.0
    assert np.isclose(losses[1], terms[1], rtol=LOSS_RTOL)
    assert np.abs(g - g_ref).max() <= 1e-4 * np.abs(g_ref).max()
    cal.destroy()


@pytest.mark.parametrize("shared", [True, False])
def test_first_adam_step(shared):
    M, o, d, seed = 512, 96, 320, 31
    A, W, A_t, W_t = _case(M, o, d, seed)
    n_sets = 1 if shared else d // 32
    cal = kb.Calibrator(A_t, W_t, n_sets)
    lam = cal.lambdas.astype(np.float64)
    theta0 = cal.theta.astype(np.float64)
    _, g = cal.loss_grad()
    hist = cal.run(1, lr=1e-2)
    expect = co.Adam(theta0.shape, lr=1e-2).step(theta0, g.astype(np.float64))
    assert np.allclose(cal.theta, expect, rtol=0, atol=2e-6)
    # history row 0 = the terms at theta0, row 1 = at the new parameters
    _, terms0, _ = co.loss_and_grad(A, W, theta0, lam[0], lam[1])
    assert np.allclose(hist[0], terms0, rtol=LOSS_RTOL)
    assert np.allclose(hist[1], co.losses(A, W, cal.theta.astype(np.float64)), rtol=LOSS_RTOL)
    cal.destroy()


@pytest.mark.parametrize("shared", [True, False])
def test_calibration_run_lowers_the_objective_like_the_oracle(shared):
    M, o, d, seed = 512, 96, 256, 51
    A, W, A_t, W_t = _case(M, o, d, seed)
    n_sets = 1 if shared else d // 32
    steps = 40
    cal = kb.Calibrator(A_t, W_t, n_sets)
    lam = cal.lambdas.astype(np.float64)
    hist = cal.run(steps, lr=1e-2)
    total = hist[:, 0] + lam[0] * hist[:, 1] + lam[1] * hist[:, 2]
    theta_ref, (la, lw), hist_ref = co.calibrate(A, W, n_sets, steps=steps, lr=1e-2)
    total_ref = hist_ref[:, 0] + la * hist_ref[:, 1] + lw * hist_ref[:, 2]
    assert np.isclose(total[0], total_ref[0], rtol=1e-3)
    assert total[-1] < total[0]
    # the two trajectories see different rounding (a flipped code changes the path), so they are
    # compared by where they end up, not step by step
    assert abs(total[-1] - total_ref[-1]) <= 0.15 * total_ref[0]
    # the final row of the history is the objective at the returned parameters
    assert np.allclose(hist[-1], co.losses(A, W, cal.theta.astype(np.float64)), rtol=LOSS_RTOL)
    _no_device_error()
    cal.destroy()


@pytest.mark.parametrize("shared", [True, False])
def test_run_on_a_side_stream_replays_a_captured_step(shared):
    """On a capturable stream one Adam step is captured once and replayed; the result must be the same as
    on the default stream, where every step is launched directly."""
    M, o, d, seed = 512, 96, 256, 52
    A, W, A_t, W_t = _case(M, o, d, seed)
    n_sets = 1 if shared else d // 32
    ref = kb.Calibrator(A_t, W_t, n_sets)
    h_ref = ref.run(7, lr=1e-2)
    h_ref2 = ref.run(3, lr=5e-3)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        cal = kb.Calibrator(A_t, W_t, n_sets, stream=side)
        h = cal.run(7, lr=1e-2, stream=side)
        h2 = cal.run(3, lr=5e-3, stream=side)          # second run: replay of the same graph, new learning rate
        side.synchronize()
    # same kernels in the same order; only atomics on the loss sums may reorder
    assert np.allclose(h, h_ref, rtol=1e-9) and np.allclose(h2, h_ref2, rtol=1e-9)
    assert np.allclose(cal.theta, ref.theta, rtol=0, atol=1e-6)
    _no_device_error()
    cal.destroy()
    ref.destroy()


def test_calibrated_factors_feed_the_quantizer():
    """get_factors -> factors_create -> quantize equals the oracle quantizer with the same G."""
    from oracle import c_oracle
    M, o, d, seed = 512, 96, 256, 61
    A, W, A_t, W_t = _case(M, o, d, seed)
    cal = kb.Calibrator(A_t, W_t, d // 32)
    cal.run(5, lr=1e-2, history=False)
    torch.cuda.synchronize()
    G = cal.factors()
    theta = cal.theta
    G_ref = co.lu_factors(theta.astype(np.float64)).astype(np.float32)
    assert np.allclose(G, G_ref, rtol=1e-6, atol=1e-7)
    f = kb.Factors.create(G)
    q = torch.empty((M, d // 2), dtype=torch.uint8, device=A_t.device)
    s = torch.empty((M, d // 32), dtype=torch.uint8, device=A_t.device)
    kb.kroquant_quantize(A_t, f, q, s)
    torch.cuda.synchronize()
    A_bits = A_t.view(torch.int16).cpu().numpy().view(np.uint16)
    q_ref, s_ref, _ = c_oracle.quantize(A_bits, G)
    assert (s.cpu().numpy() != s_ref).mean() <= 1e-4
    assert (q.cpu().numpy() != q_ref).mean() <= 1e-3
    f.destroy()
    cal.destroy()


@pytest.mark.parametrize("rows,d", [(1000, 256), (64, 96), (8, 32), (4104, 1152)])
@pytest.mark.parametrize("shared", [True, False])
def test_block_grad_against_the_oracle(rows, d, shared):
    rng = np.random.default_rng(rows + d)
    X_bits = wl.gen_activations(wl.calib_spec(rows, d, 81))
    X = wl.bf16_bits_to_f32(X_bits).astype(np.float64)
    Gm = rng.standard_normal((rows, d)).astype(np.float32)
    n_sets = 1 if shared else d // 32
    dev = torch.device("cuda:0")
    X_t = torch.from_numpy(X_bits.view(np.int16)).to(dev).view(torch.bfloat16)
    out = kb.kroquant_block_grad(X_t, torch.from_numpy(Gm).to(dev), n_sets).cpu().numpy()
    ref = co._block_grads(X, Gm.astype(np.float64), n_sets)
    # fp32 products and partial sums: error of a sum of n terms ~ sqrt(n) 2^-24 of its absolute sum
    bound = 1e-5 * (np.abs(X).T @ np.abs(Gm).astype(np.float64)).max()
    assert np.abs(out - ref).max() <= bound
    again = kb.kroquant_block_grad(X_t, torch.from_numpy(Gm).to(dev), n_sets).cpu().numpy()
    assert np.array_equal(out, again)                   # fixed summation order


@pytest.mark.parametrize("shared", [True, False])
def test_calibrated_layer_through_the_quantizer_and_the_block_scaled_gemm(shared):
    """End of the pipeline (Section 3.3 objective, Section 3.4 inference form): calibrate, hand the
    activation factors and the weight factors (T^-T is again a Kronecker set) to the quantizer,
    multiply the two MXFP4 operands with the library's block-scaled tensor-core GEMM, and find the
    output error the calibrator reported."""
    F = torch.nn.functional
    if not hasattr(F, "scaled_mm"):
        pytest.skip("torch.nn.functional.scaled_mm not available")
    M, o, d, seed = 512, 256, 512, 77
    A, W, A_t, W_t = _case(M, o, d, seed)
    n_sets = 1 if shared else d // 32
    cal = kb.Calibrator(A_t, W_t, n_sets)
    hist = cal.run(10, lr=1e-2)
    theta = cal.theta.astype(np.float64)
    G, H = cal.factors(), cal.weight_factors()
    K_ref, P_ref = co.blocks_of(theta)
    for s_ in range(n_sets):
        assert np.allclose(co.kron5(G[s_].astype(np.float64)), K_ref[s_], rtol=1e-5, atol=1e-6)
        assert np.allclose(co.kron5(H[s_].astype(np.float64)), P_ref[s_], rtol=1e-5, atol=1e-6)
    fa, fw = kb.Factors.create(G), kb.Factors.create(H)
    qa, sa = kb.kroquant_quantize(A_t, fa, scale_layout="tiled")
    qw, sw = kb.kroquant_quantize(W_t, fw, scale_layout="tiled")
    out = F.scaled_mm(qa.view(torch.float4_e2m1fn_x2), qw.view(torch.float4_e2m1fn_x2).t(),
                      sa.view(torch.float8_e8m0fnu), F.ScalingType.BlockWise1x32,
                      sw.view(torch.float8_e8m0fnu), F.ScalingType.BlockWise1x32,
                      swizzle_a=F.SwizzleType.SWIZZLE_32_4_4, swizzle_b=F.SwizzleType.SWIZZLE_32_4_4,
                      output_dtype=torch.bfloat16).double().cpu().numpy()
    # the oracle's forward pass with the float32 factors the quantizer was given
    f = co.forward(A, W, theta)
    ref = f["Yq"] @ f["Zq"].T
    # bf16 output of the library GEMM (2^-9 relative); a few codes may differ (float32 factors)
    assert np.abs(out - ref).max() <= 6e-3 * np.abs(ref).max()
    L_out = np.sum((out - A @ W.T) ** 2) / (M * o)
    assert np.isclose(L_out, hist[-1, 0], rtol=2e-2)
    assert np.isclose(f["L_out"], hist[-1, 0], rtol=LOSS_RTOL)
    fa.destroy()
    fw.destroy()
    cal.destroy()


def test_argument_checks():
    A, W, A_t, W_t = _case(256, 64, 128, 71)
    with pytest.raises(kb.KroQuantError):
        kb.Calibrator(A_t, W_t, 3)                      # neither 1 nor d/32
    with pytest.raises(kb.KroQuantError):
        kb.Calibrator(A_t[:252].contiguous(), W_t, 1)   # M not a multiple of 8
    with pytest.raises(kb.KroQuantError):
        kb.Calibrator(A_t, W_t[:40].contiguous(), 1)    # o not a multiple of 32
    cal = kb.Calibrator(A_t, W_t, 1)
    bad = co.hadamard_theta(1).astype(np.float32)
    bad[0, 2, 0] = 0.0
    with pytest.raises(kb.KroQuantError):
        cal.theta = bad
    with pytest.raises(kb.KroQuantError):
        cal.run(0)
    cal.destroy()
