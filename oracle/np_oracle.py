"""NumPy restatement of the KroQuant quantizer -- TEST INFRASTRUCTURE ONLY.

Independent of the C oracle in how it gets there: K is built with a chain of
``np.kron`` (the library's Kronecker product) instead of the bit formula, and the
E2M1 code is found by a nearest-grid-value search instead of interval tests.
The two must agree bit for bit; the tests check that.

Paper passages: blockwise quantizer Q_b (Section 3.1); K = G1 (x) ... (x) G5
(Section 3.2); y = x K on each 32-channel slice (Section 3.5); MXFP4 = E2M1 +
E8M0 per 32 block following OCP Microscaling (Section 4.1, Appendix D).

Parity pins (tests that fix each function to something other than itself):
  dense_k            np.kron chain vs the bit formula of the C twin; shear hand vectors; Hadamard closed form
  lu_to_factors      L U product written out, det = -1
  transform          exact Fraction sums on small blocks; the C twin bit for bit
  scale_transform    NumPy casts; the C twin
  mx_encode          hand-worked blocks (tests/golden/mxfp4_handworked.txt); brute force over every bf16
                     value in (-8, 8) with exact rationals; tie table
  decode             the E2M1 grid written out; np.linalg.inv round trip
  encode_with_scale  hand-worked blocks under imposed scale bytes (tests/golden/mxfp4_imposed_scale.txt);
                     brute force over every bf16 value in (-8, 8) at three scale bytes; equality with the
                     C encoder when the imposed byte is the block's own
Nothing here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

BLOCK = 32
E2M1_GRID = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0], dtype=np.float64)


def widen(X_bits: np.ndarray) -> np.ndarray:
    u = np.asarray(X_bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32)


def dense_k(G1: np.ndarray) -> np.ndarray:
    """K = G1 (x) G2 (x) G3 (x) G4 (x) G5 in float64 (Section 3.2)."""
    G1 = np.asarray(G1, dtype=np.float64).reshape(5, 2, 2)
    K = G1[0]
    for k in range(1, 5):
        K = np.kron(K, G1[k])
    return K


def lu_to_factors(abc: np.ndarray) -> np.ndarray:
    abc = np.asarray(abc, dtype=np.float64)
    a, b, c = abc[..., 0], abc[..., 1], abc[..., 2]
    L = np.zeros(abc.shape[:-1] + (2, 2))
    U = np.zeros_like(L)
    L[..., 0, 0] = 1.0
    L[..., 1, 0] = c
    L[..., 1, 1] = 1.0
    U[..., 0, 0] = a
    U[..., 0, 1] = b
    U[..., 1, 1] = -1.0 / a
    return (L @ U).astype(np.float32)


def transform(X_bits: np.ndarray, G: np.ndarray) -> np.ndarray:
    """float32( x K ) per 32-channel block; sums in float64."""
    x = widen(X_bits).astype(np.float64)
    t, d = x.shape
    nb = d // BLOCK
    G = np.asarray(G, dtype=np.float32)
    assert d % BLOCK == 0 and G.shape[0] in (1, nb)
    xb = x.reshape(t, nb, BLOCK)
    y = np.empty_like(xb)
    for j in range(nb):
        K = dense_k(G[0] if G.shape[0] == 1 else G[j])
        # explicit ascending-r accumulation, like the definition
        acc = np.zeros((t, BLOCK))
        for r in range(BLOCK):
            acc += xb[:, j, r:r + 1] * K[r:r + 1, :]
        y[:, j, :] = acc
    return y.reshape(t, d).astype(np.float32)


def scale_transform(X_bits: np.ndarray, s: np.ndarray) -> np.ndarray:
    x = widen(X_bits).astype(np.float64)
    return (x * np.asarray(s, dtype=np.float32).astype(np.float64)[None, :]).astype(np.float32)


def mx_encode(Y: np.ndarray):
    """float32 [t, d] -> (codes uint8 [t, d/2], scales uint8 [t, d/32])."""
    Y = np.asarray(Y, dtype=np.float32)
    t, d = Y.shape
    nb = d // BLOCK
    yb = Y.reshape(t, nb, BLOCK)
    amax = np.abs(yb).max(axis=2)
    # floor(log2 amax) via frexp: amax = m * 2^e, m in [0.5, 1) -> floor(log2) = e - 1
    _, e = np.frexp(amax.astype(np.float64))
    S = np.where(amax == 0, 0, np.clip(e - 1 - 2 + 127, 0, 254)).astype(np.int64)
    v = yb.astype(np.float64) * np.exp2((127 - S).astype(np.float64))[:, :, None]
    av = np.abs(v)
    # nearest grid value; ties -> even code; beyond 6 -> code 7
    dist = np.abs(av[..., None] - E2M1_GRID)            # [t, nb, 32, 8]
    best = dist.min(axis=-1, keepdims=True)
    is_best = dist == best
    codes_all = np.arange(8)
    even_pref = np.where(is_best & (codes_all % 2 == 0), codes_all, 99).min(axis=-1)
    any_pref = np.where(is_best, codes_all, 99).min(axis=-1)
    mag = np.where(even_pref != 99, even_pref, any_pref)
    code = (mag | (np.signbit(v).astype(np.int64) << 3)).astype(np.uint8)
    code = code.reshape(t, d)
    q = (code[:, 0::2] | (code[:, 1::2] << np.uint8(4))).astype(np.uint8)
    return q, S.astype(np.uint8)


def quantize(X_bits, G):
    Y = transform(X_bits, G)
    q, s = mx_encode(Y)
    return q, s, Y


def decode(q: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """codes + scales -> float64 transformed values (exact)."""
    q = np.asarray(q, dtype=np.uint8)
    t, half = q.shape
    d = half * 2
    code = np.empty((t, d), np.uint8)
    code[:, 0::2] = q & 15
    code[:, 1::2] = q >> 4
    mag = E2M1_GRID[code & 7]
    sign = np.where(code & 8, -1.0, 1.0)
    sc = np.exp2(np.asarray(scales, dtype=np.float64) - 127.0)
    return (mag * sign).reshape(t, d // BLOCK, BLOCK) * sc[:, :, None]


def encode_with_scale(Y: np.ndarray, S: np.ndarray) -> np.ndarray:
    """Codes (one per element, uint8 [t, d]) of float32 Y when the scale bytes S
    [t, d/32] are imposed instead of derived from the block amax.  Used by the
    parity rule that lets a block whose amax sits within rounding distance of a
    power of two take the neighbouring scale."""
    Y = np.asarray(Y, dtype=np.float32)
    t, d = Y.shape
    nb = d // BLOCK
    v = Y.reshape(t, nb, BLOCK).astype(np.float64) * np.exp2(127.0 - np.asarray(S, np.float64))[:, :, None]
    av = np.abs(v)
    bounds = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
    # ties to the even code: boundaries 0.25, 1.25, 2.5, 5.0 round down (<=), the others up
    mag = np.zeros(av.shape, np.int64)
    for i, b in enumerate(bounds):
        down = i % 2 == 0           # boundary between code i (even when i even) and i+1
        mag += (av > b) if down else (av >= b)
    code = mag | (np.signbit(v).astype(np.int64) << 3)
    return code.reshape(t, d).astype(np.uint8)
