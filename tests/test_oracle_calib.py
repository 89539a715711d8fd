"""Pins for the calibration oracle (Section 3.3; Adam set-up of Appendix D).

Each test ties a part of oracle/calib_oracle.py to something outside it: a closed form, a
finite difference of the forward pass, an invariance the paper states, or a library
optimiser.
"""
import numpy as np
import pytest
import torch

from oracle import calib_oracle as co
from paper_2607_21446_b200 import workloads as wl


def _case(M=96, o=40, d=128, seed=11):
    A = wl.bf16_bits_to_f32(wl.gen_activations(wl.calib_spec(M, d, seed))).astype(np.float64)
    W = wl.bf16_bits_to_f32(wl.gen_weights(seed, o, d)).astype(np.float64)
    return A, W


def _theta(n_sets, seed=3):
    return wl.gen_lu_params(seed, n_sets).astype(np.float64)


def test_lu_form_and_unit_determinant():
    th = _theta(7)
    G = co.lu_factors(th)
    for s in range(7):
        for k in range(5):
            a, b, c = th[s, k]
            L = np.array([[1.0, 0.0], [c, 1.0]])
            U = np.array([[a, b], [0.0, -1.0 / a]])
            assert np.allclose(G[s, k], L @ U, rtol=1e-14, atol=0)
            assert abs(np.linalg.det(G[s, k]) + 1.0) < 1e-12
    K, P = co.blocks_of(th)
    for s in range(7):
        assert abs(abs(np.linalg.det(K[s])) - 1.0) < 1e-9
        assert np.allclose(K[s] @ P[s].T, np.eye(32), atol=1e-9)


def test_hadamard_initialisation_is_the_sylvester_matrix():
    K, P = co.blocks_of(co.hadamard_theta(1))
    r = np.arange(32)
    sign = np.array([[(-1.0) ** bin(i & j).count("1") for j in r] for i in r])
    assert np.allclose(K[0], sign / np.sqrt(32.0), atol=1e-14)
    assert np.allclose(P[0], K[0], atol=1e-13)           # orthogonal and symmetric


def test_inverse_transpose_closed_form_used_in_the_backward_pass():
    th = _theta(3)
    G = co.lu_factors(th)
    for s in range(3):
        H = np.stack([np.linalg.inv(G[s, k]).T for k in range(5)])
        assert np.allclose(co.kron5(H), np.linalg.inv(co.kron5(G[s])).T, rtol=1e-9, atol=1e-12)
        a, b, c = th[s, :, 0], th[s, :, 1], th[s, :, 2]
        closed = np.empty((5, 2, 2))
        closed[:, 0, 0], closed[:, 0, 1], closed[:, 1, 0], closed[:, 1, 1] = 1 / a - b * c, a * c, b, -a
        assert np.allclose(closed, H, rtol=1e-12, atol=1e-14)


def test_linear_map_is_invariant_without_quantisation(monkeypatch):
    """A T (W T^-1)^T = A W^T: with Q replaced by the identity all three terms vanish."""
    A, W = _case()
    monkeypatch.setattr(co, "fake_quant", lambda V: V.copy())
    for n_sets in (1, A.shape[1] // 32):
        l = co.losses(A, W, _theta(n_sets))
        ref = np.sum((A @ W.T) ** 2) / (A.shape[0] * W.shape[0])
        assert l[0] < 1e-22 * max(ref, 1.0) and l[1] == 0.0 and l[2] == 0.0


def test_fake_quant_is_idempotent_and_bounded():
    A, _ = _case()
    Aq = co.fake_quant(A)
    assert np.array_equal(co.fake_quant(Aq), Aq)
    blocks = A.reshape(A.shape[0], -1, 32)
    amax = np.abs(blocks).max(axis=2, keepdims=True)
    err = np.abs(Aq.reshape(blocks.shape) - blocks)
    # E2M1 with the floor scale rule: error at most amax/4 (saturation of (6,8) to 6), usually amax/8
    assert np.all(err <= amax / 4 + 1e-12)


def _surrogate(A, W, theta, frozen, lam_A, lam_W):
    """The function whose exact gradient the straight-through rule defines: the quantisation
    residuals and the regulariser targets are frozen at the expansion point."""
    M, d = A.shape
    o = W.shape[0]
    K, P = co.blocks_of(theta)
    Y = co.apply_blocks(A, K)
    Z = co.apply_blocks(W, P)
    E = (Y + frozen["cY"]) @ (Z + frozen["cZ"]).T - A @ W.T
    return (np.sum(E * E) / (M * o)
            + lam_A * np.sum((frozen["tY"] - Y) ** 2) / (M * d)
            + lam_W * np.sum((frozen["tZ"] - Z) ** 2) / (o * d))


@pytest.mark.parametrize("shared", [True, False])
@pytest.mark.parametrize("lams", [(0.0, 0.0), (3.0, 0.7)])
def test_gradient_matches_finite_differences_of_the_frozen_residual_function(shared, lams):
    A, W = _case(M=64, o=24, d=96)
    n_sets = 1 if shared else 3
    theta = _theta(n_sets, seed=5)
    lam_A, lam_W = lams
    f = co.forward(A, W, theta)
    frozen = dict(cY=f["Yq"] - f["Y"], cZ=f["Zq"] - f["Z"], tY=f["Yq"], tZ=f["Zq"])
    total, terms, g = co.loss_and_grad(A, W, theta, lam_A, lam_W)
    assert np.isclose(total, _surrogate(A, W, theta, frozen, lam_A, lam_W), rtol=1e-12)
    assert np.isclose(total, terms[0] + lam_A * terms[1] + lam_W * terms[2], rtol=1e-14)
    h = 1e-6
    fd = np.zeros_like(theta)
    for idx in np.ndindex(theta.shape):
        tp, tm = theta.copy(), theta.copy()
        tp[idx] += h
        tm[idx] -= h
        fd[idx] = (_surrogate(A, W, tp, frozen, lam_A, lam_W)
                   - _surrogate(A, W, tm, frozen, lam_A, lam_W)) / (2 * h)
    scale = np.abs(fd).max()
    assert scale > 0
    assert np.abs(g - fd).max() <= 1e-6 * scale


def test_regulariser_gradient_pulls_towards_the_grid():
    """With the output term removed (W = 0 makes E = 0) a small step against the gradient
    must not increase L_A measured against the frozen target."""
    A, W = _case(M=64, o=8, d=64)
    W0 = np.zeros_like(W)
    theta = _theta(1, seed=9)
    f = co.forward(A, W0, theta)
    _, _, g = co.loss_and_grad(A, W0, theta, 1.0, 0.0)
    frozen = dict(cY=f["Yq"] - f["Y"], cZ=f["Zq"] - f["Z"], tY=f["Yq"], tZ=f["Zq"])
    s0 = _surrogate(A, W0, theta, frozen, 1.0, 0.0)
    s1 = _surrogate(A, W0, theta - 1e-4 * g / np.abs(g).max(), frozen, 1.0, 0.0)
    assert s1 < s0


def test_auto_lambda_balances_the_terms_at_initialisation():
    A, W = _case()
    lam_A, lam_W, l0 = co.auto_lambda(A, W, 1)
    assert np.isclose(lam_A * l0[1], l0[0], rtol=1e-12)
    assert np.isclose(lam_W * l0[2], l0[0], rtol=1e-12)
    assert np.array_equal(l0, co.losses(A, W, co.hadamard_theta(1)))


def test_adam_matches_the_library_optimiser():
    rng = np.random.default_rng(0)
    shape = (4, 5, 3)
    th0 = rng.standard_normal(shape)
    grads = [rng.standard_normal(shape) * 10.0 ** rng.integers(-4, 2) for _ in range(25)]
    opt = co.Adam(shape, lr=1e-2)
    th = th0.copy()
    p = torch.tensor(th0, dtype=torch.float64, requires_grad=True)
    topt = torch.optim.Adam([p], lr=1e-2)
    for i, g in enumerate(grads):
        th = opt.step(th, g)
        p.grad = torch.tensor(g, dtype=torch.float64)
        topt.step()
        assert np.allclose(th, p.detach().numpy(), rtol=1e-12, atol=1e-14), i
    # first step in closed form: m_hat = g, v_hat = g^2
    opt1 = co.Adam(shape, lr=1e-2)
    g = grads[0]
    assert np.allclose(opt1.step(th0, g), th0 - 1e-2 * g / (np.abs(g) + 1e-8), rtol=1e-13)


@pytest.mark.parametrize("shared", [True, False])
def test_calibration_lowers_the_objective(shared):
    """Section 4.3's claim in miniature: starting from the Hadamard initialisation the learned
    parameters reach a lower objective on the calibration data."""
    A, W = _case(M=128, o=48, d=128, seed=21)
    n_sets = 1 if shared else 4
    theta, (lam_A, lam_W), hist = co.calibrate(A, W, n_sets, steps=40, lr=1e-2)
    total = hist[:, 0] + lam_A * hist[:, 1] + lam_W * hist[:, 2]
    assert np.isclose(total[0], 3.0 * hist[0, 0], rtol=1e-12)     # three balanced terms at T0
    assert total[1:].min() < total[0]
    assert total[-1] < total[0]
    assert np.all(np.isfinite(theta)) and np.all(np.abs(theta[..., 0]) > 1e-3)
