"""Layer-wise transform calibration, written out in float64 NumPy -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
module; the product path never does.

What it computes (Section 3.3 of the paper, with the set-up of Appendix D):

    theta = (a_k, b_k, c_k), k = 1..5, per factor set          (Section 3.2, LU form)
    G_k   = [[a, b], [a c, b c - 1/a]]                          (L_k U_k multiplied out)
    K     = G_1 (x) ... (x) G_5,  T = diag(K^(1), ..., K^(d/32))
    Y = A T,  Z = W T^{-T}                                      (Z block j = W block j times K_j^{-T})
    L_out = || Q(Y) Q(Z)^T - A W^T ||_F^2 / (M o)               (output error)
    L_A   = || Q(Y) - Y ||_F^2 / (M d),  L_W = || Q(Z) - Z ||_F^2 / (o d)
    L     = L_out + lambda_A L_A + lambda_W L_W                 (total objective)
    lambda_A = L_out(T0)/L_A(T0), lambda_W = L_out(T0)/L_W(T0), T0 = Hadamard initialisation
    Adam on theta, straight-through estimator for Q.

M = N m is the number of calibration rows (all samples stacked), o the number of output
features.  Q is the MXFP4 quantise-then-dequantise operator of Section 3.1 (the encoder of
the C oracle, fed with the float32 rounding of its argument, which is the precision the
quantizer decides in everywhere in this project).

Readings of points the paper leaves open:
  * Straight-through estimator: in the backward pass Q has the identity Jacobian (no
    clipping mask; the MX scale is not differentiated).
  * Under that rule the literal gradient of ||Q(Y) - Y||^2 is zero.  The paper says the two
    regularisers supply gradient signal, so in L_A and L_W the quantised tensor is a
    constant target: dL_A/dY = 2 (Y - Q(Y)) / (M d), and likewise for L_W.
  * Adam with the usual defaults (beta1 0.9, beta2 0.999, eps 1e-8, bias correction, no
    weight decay); the parameters after the last step are the result.
"""
from __future__ import annotations

import numpy as np

from . import c_oracle

BLOCK = 32


# ---------------------------------------------------------------- parametrisation (Section 3.2)

def lu_factors(theta: np.ndarray) -> np.ndarray:
    """theta [..., 3] = (a, b, c) -> G [..., 2, 2] = L(c) U(a, b), float64."""
    theta = np.asarray(theta, dtype=np.float64)
    a, b, c = theta[..., 0], theta[..., 1], theta[..., 2]
    G = np.empty(theta.shape[:-1] + (2, 2))
    G[..., 0, 0] = a
    G[..., 0, 1] = b
    G[..., 1, 0] = c * a
    G[..., 1, 1] = c * b - 1.0 / a
    return G


def kron5(F: np.ndarray) -> np.ndarray:
    """F [5, 2, 2] -> F[0] (x) F[1] (x) F[2] (x) F[3] (x) F[4], 32 x 32."""
    K = F[0]
    for k in range(1, 5):
        K = np.kron(K, F[k])
    return K


def hadamard_theta(n_sets: int) -> np.ndarray:
    """(a, b, c) = (cos(pi/4), sin(pi/4), 1) for every factor: T0 = block Hadamard."""
    th = np.empty((n_sets, 5, 3))
    th[..., 0] = np.cos(np.pi / 4)
    th[..., 1] = np.sin(np.pi / 4)
    th[..., 2] = 1.0
    return th


def blocks_of(theta: np.ndarray):
    """theta [n_sets, 5, 3] -> (K [n_sets, 32, 32], P [n_sets, 32, 32]) with P = K^{-T}."""
    G = lu_factors(theta)
    K = np.stack([kron5(G[s]) for s in range(G.shape[0])])
    P = np.stack([np.linalg.inv(K[s]).T for s in range(G.shape[0])])
    return K, P


def apply_blocks(X: np.ndarray, B: np.ndarray) -> np.ndarray:
    """Row-vector action: out[:, block j] = X[:, block j] @ B[j] (B[0] for every j if shared)."""
    rows, d = X.shape
    nb = d // BLOCK
    out = np.empty((rows, d))
    for j in range(nb):
        Bj = B[0] if B.shape[0] == 1 else B[j]
        out[:, j * BLOCK:(j + 1) * BLOCK] = X[:, j * BLOCK:(j + 1) * BLOCK] @ Bj
    return out


# ---------------------------------------------------------------- Q (Section 3.1)

def fake_quant(V: np.ndarray) -> np.ndarray:
    """MXFP4 quantise-then-dequantise of every 32-block of every row; float64 out (exact values)."""
    q, s = c_oracle.mx_encode(V.astype(np.float32))
    return c_oracle.dequantize(q, s).astype(np.float64)


# ---------------------------------------------------------------- objective (Section 3.3)

def forward(A: np.ndarray, W: np.ndarray, theta: np.ndarray):
    """-> dict with Y, Z, Yq, Zq, E = Yq Zq^T - A W^T and the three loss terms."""
    A = np.asarray(A, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    M, d = A.shape
    o = W.shape[0]
    K, P = blocks_of(theta)
    Y = apply_blocks(A, K)
    Z = apply_blocks(W, P)
    Yq = fake_quant(Y)
    Zq = fake_quant(Z)
    E = Yq @ Zq.T - A @ W.T
    return dict(
        K=K, P=P, Y=Y, Z=Z, Yq=Yq, Zq=Zq, E=E,
        L_out=float(np.sum(E * E) / (M * o)),
        L_A=float(np.sum((Yq - Y) ** 2) / (M * d)),
        L_W=float(np.sum((Zq - Z) ** 2) / (o * d)),
    )


def losses(A, W, theta) -> np.ndarray:
    f = forward(A, W, theta)
    return np.array([f["L_out"], f["L_A"], f["L_W"]])


def auto_lambda(A, W, n_sets: int):
    """lambda_A, lambda_W: each regulariser matches L_out at the Hadamard initialisation."""
    l0 = losses(A, W, hadamard_theta(n_sets))
    return l0[0] / l0[1], l0[0] / l0[2], l0


def _block_grads(X: np.ndarray, dV: np.ndarray, n_sets: int) -> np.ndarray:
    """dB[j] = X_j^T dV_j (summed over j when the set is shared)."""
    d = X.shape[1]
    nb = d // BLOCK
    out = np.zeros((n_sets, BLOCK, BLOCK))
    for j in range(nb):
        sl = slice(j * BLOCK, (j + 1) * BLOCK)
        out[0 if n_sets == 1 else j] += X[:, sl].T @ dV[:, sl]
    return out


def _factor_grads(F: np.ndarray, dB: np.ndarray) -> np.ndarray:
    """B = kron5(F).  dF[k][r][c] = <dB, dB/dF[k][r][c]>, and dB/dF[k][r][c] is the same
    Kronecker chain with factor k replaced by the unit matrix e_r e_c^T."""
    dF = np.zeros((5, 2, 2))
    for k in range(5):
        for r in range(2):
            for c in range(2):
                Fk = F.copy()
                Fk[k] = 0.0
                Fk[k, r, c] = 1.0
                dF[k, r, c] = np.sum(dB * kron5(Fk))
    return dF


def loss_and_grad(A, W, theta, lam_A: float, lam_W: float):
    """-> (L, [L_out, L_A, L_W], dL/dtheta [n_sets, 5, 3]) under the straight-through rule."""
    A = np.asarray(A, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    theta = np.asarray(theta, dtype=np.float64)
    n_sets = theta.shape[0]
    M, d = A.shape
    o = W.shape[0]
    f = forward(A, W, theta)
    dO = 2.0 * f["E"] / (M * o)
    dY = dO @ f["Zq"] + lam_A * 2.0 * (f["Y"] - f["Yq"]) / (M * d)
    dZ = dO.T @ f["Yq"] + lam_W * 2.0 * (f["Z"] - f["Zq"]) / (o * d)
    dK = _block_grads(A, dY, n_sets)
    dP = _block_grads(W, dZ, n_sets)

    G = lu_factors(theta)
    a, b, c = theta[..., 0], theta[..., 1], theta[..., 2]
    # H_k = G_k^{-T} in closed form (det G_k = -1), so that P = kron5(H)
    H = np.empty_like(G)
    H[..., 0, 0] = 1.0 / a - b * c
    H[..., 0, 1] = a * c
    H[..., 1, 0] = b
    H[..., 1, 1] = -a
    grad = np.zeros_like(theta)
    for s in range(n_sets):
        dG = _factor_grads(G[s], dK[s])
        dH = _factor_grads(H[s], dP[s])
        for k in range(5):
            ak, bk, ck = a[s, k], b[s, k], c[s, k]
            dG_da = np.array([[1.0, 0.0], [ck, 1.0 / ak ** 2]])
            dG_db = np.array([[0.0, 1.0], [0.0, ck]])
            dG_dc = np.array([[0.0, 0.0], [ak, bk]])
            dH_da = np.array([[-1.0 / ak ** 2, ck], [0.0, -1.0]])
            dH_db = np.array([[-ck, 0.0], [1.0, 0.0]])
            dH_dc = np.array([[-bk, ak], [0.0, 0.0]])
            grad[s, k, 0] = np.sum(dG[k] * dG_da) + np.sum(dH[k] * dH_da)
            grad[s, k, 1] = np.sum(dG[k] * dG_db) + np.sum(dH[k] * dH_db)
            grad[s, k, 2] = np.sum(dG[k] * dG_dc) + np.sum(dH[k] * dH_dc)
    terms = np.array([f["L_out"], f["L_A"], f["L_W"]])
    total = terms[0] + lam_A * terms[1] + lam_W * terms[2]
    return total, terms, grad


# ---------------------------------------------------------------- optimiser

class Adam:
    def __init__(self, shape, lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8):
        self.lr, self.b1, self.b2, self.eps = lr, beta1, beta2, eps
        self.m = np.zeros(shape)
        self.v = np.zeros(shape)
        self.t = 0

    def step(self, theta: np.ndarray, g: np.ndarray) -> np.ndarray:
        self.t += 1
        self.m = self.b1 * self.m + (1.0 - self.b1) * g
        self.v = self.b2 * self.v + (1.0 - self.b2) * g * g
        mhat = self.m / (1.0 - self.b1 ** self.t)
        vhat = self.v / (1.0 - self.b2 ** self.t)
        return theta - self.lr * mhat / (np.sqrt(vhat) + self.eps)


def calibrate(A, W, n_sets: int, steps: int = 100, lr: float = 1e-2):
    """Appendix D recipe: Hadamard initialisation, automatic lambdas, `steps` Adam steps.
    -> (theta, lambdas, history [steps + 1, 3] of (L_out, L_A, L_W); last row = final theta)."""
    theta = hadamard_theta(n_sets)
    lam_A, lam_W, l0 = auto_lambda(A, W, n_sets)
    opt = Adam(theta.shape, lr=lr)
    hist = []
    for _ in range(steps):
        _, terms, g = loss_and_grad(A, W, theta, lam_A, lam_W)
        hist.append(terms)
        theta = opt.step(theta, g)
    hist.append(losses(A, W, theta))
    return theta, (lam_A, lam_W), np.array(hist)
