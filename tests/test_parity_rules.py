"""The checker itself under test (CPU only): tests/parity.py decides which differences between the
CUDA quantizer and the oracle are allowed, so it is fed outputs that must be REJECTED and outputs
that must be ACCEPTED, all derived from the oracle's result on inputs built for the purpose.

Rules (stated in tests/parity.py): P0 exact kernels bit-identical; P1 values within 1e-5 relative
(floored at amax/32); P2 a code may differ by one step, same sign, only within 1e-5 relative of a
rounding boundary, at most 1e-4 of all codes; P3 a scale byte may differ by one only where the block
amax lies within 1e-5 relative of a power of two, its codes then follow the imposed scale, at most
1e-4 of all blocks; a zero's sign is free where the value is exactly zero (or, inexact kernels only,
within the value tolerance of zero).
"""
import numpy as np
import pytest

from oracle import c_oracle as co
from tests import parity as P

T, D = 64, 256          # 64 rows x 8 blocks = 512 blocks, 16384 codes


def base_case():
    """Blocks with amax exactly 4 (S = 127, scaled value = value) and well-separated small values,
    none of them near a rounding boundary."""
    rng = np.random.default_rng(7)
    grid = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
    Y = (grid[rng.integers(0, 7, size=(T, D))] * rng.choice([-1.0, 1.0], size=(T, D))).astype(np.float32)
    Y += (rng.uniform(-0.05, 0.05, size=(T, D))).astype(np.float32)      # stays >= 0.2 away from every boundary
    Y[:, 0::32] = 4.0                                                    # block amax = 4 exactly
    q, s = co.mx_encode(Y)
    assert (s == 127).all()
    return Y, q, s


def set_code(q, t, c, code):
    q = q.copy()
    b = q[t, c // 2]
    q[t, c // 2] = (b & 0xF0) | code if c % 2 == 0 else (b & 0x0F) | (code << 4)
    return q


def get_code(q, t, c):
    b = int(q[t, c // 2])
    return b & 15 if c % 2 == 0 else b >> 4


def test_identical_outputs_pass_both_modes():
    Y, q, s = base_case()
    for exact in (True, False):
        r = P.check_codes(q, s, q, s, Y, exact=exact)
        assert r == {"code_mismatches": 0, "scale_mismatches": 0, "zero_sign_only": 0}


# ---- P2 --------------------------------------------------------------------------------------
def near_boundary_case(n_near=1, rel=5e-6):
    """base case with n_near elements moved to a boundary * (1 + rel): the oracle rounds them up."""
    Y, _, _ = base_case()
    pos = [(3 + i % (T - 3), 5 + 32 * (i % 8) + (i // 8) % 20) for i in range(n_near)]
    for i, (t, c) in enumerate(pos):
        b = P.BOUNDS[i % 7]
        Y[t, c] = np.float32(b * (1.0 + rel))
    q, s = co.mx_encode(Y)
    return Y, q, s, pos


def test_p2_accepts_one_step_at_a_boundary():
    Y, q, s, pos = near_boundary_case(1)
    (t, c), = pos
    up = get_code(q, t, c)
    assert up == 1                                     # 0.25 (1 + 5e-6) -> 0.5
    r = P.check_codes(set_code(q, t, c, up - 1), s, q, s, Y, exact=False)
    assert r["code_mismatches"] == 1


def test_p2_rejects_the_same_difference_for_an_exact_kernel():
    Y, q, s, pos = near_boundary_case(1)
    (t, c), = pos
    with pytest.raises(AssertionError, match="P0"):
        P.check_codes(set_code(q, t, c, get_code(q, t, c) - 1), s, q, s, Y, exact=True)


def test_p2_rejects_one_step_far_from_any_boundary():
    Y, q, s = base_case()
    t, c = 5, 7
    code = get_code(q, t, c)
    other = (code & 8) | ((code & 7) + 1 if (code & 7) < 7 else 6)
    with pytest.raises(AssertionError, match="away from any rounding boundary"):
        P.check_codes(set_code(q, t, c, other), s, q, s, Y, exact=False)


def test_p2_rejects_one_step_just_outside_the_relative_window():
    Y, _, _ = base_case()
    Y[9, 9] = np.float32(2.5 * (1.0 + 3e-5))           # 3e-5 > 1e-5
    q, s = co.mx_encode(Y)
    assert get_code(q, 9, 9) == 5
    with pytest.raises(AssertionError, match="away from any rounding boundary"):
        P.check_codes(set_code(q, 9, 9, 4), s, q, s, Y, exact=False)


def test_p2_rejects_two_steps_at_a_boundary():
    Y, _, _ = base_case()
    Y[9, 9] = np.float32(2.5 * (1.0 + 5e-6))
    q, s = co.mx_encode(Y)
    assert get_code(q, 9, 9) == 5
    with pytest.raises(AssertionError, match="more than one step"):
        P.check_codes(set_code(q, 9, 9, 3), s, q, s, Y, exact=False)


def test_p2_rejects_a_sign_flip_on_a_nonzero_value():
    Y, _, _ = base_case()
    Y[9, 9] = np.float32(2.5 * (1.0 + 5e-6))
    q, s = co.mx_encode(Y)
    with pytest.raises(AssertionError, match="sign differs"):
        P.check_codes(set_code(q, 9, 9, 8 | 4), s, q, s, Y, exact=False)
    # and far from a boundary a flipped sign is an ordinary (forbidden) mismatch
    Y2, q2, s2 = base_case()
    code = get_code(q2, 5, 7)
    with pytest.raises(AssertionError):
        P.check_codes(set_code(q2, 5, 7, code ^ 8), s2, q2, s2, Y2, exact=False)


def test_p2_rejects_too_many_allowed_mismatches():
    n_codes = T * D
    limit = int(P.MAX_FRACTION * n_codes)              # 1 of 16384
    Y, q, s, pos = near_boundary_case(limit + 3)
    qg = q
    for t, c in pos:
        qg = set_code(qg, t, c, get_code(q, t, c) - 1)
    with pytest.raises(AssertionError, match="code mismatches"):
        P.check_codes(qg, s, q, s, Y, exact=False)
    # at the limit it passes
    qg = q
    for t, c in pos[:max(1, limit)]:
        qg = set_code(qg, t, c, get_code(q, t, c) - 1)
    assert P.check_codes(qg, s, q, s, Y, exact=False)["code_mismatches"] == max(1, limit)


# ---- zero sign ---------------------------------------------------------------------------------
def test_zero_sign_rules():
    Y, _, _ = base_case()
    Y[4, 3] = 0.0                                      # exactly zero
    Y[4, 4] = np.float32(4.0 * 1e-5 / 32 * 0.5)        # inside the value tolerance of zero
    Y[4, 6] = np.float32(0.1)                          # rounds to zero, but its sign is determined
    q, s = co.mx_encode(Y)
    assert get_code(q, 4, 3) == 0 and get_code(q, 4, 4) == 0 and get_code(q, 4, 6) == 0
    # exact zero: either sign, both modes
    for exact in (True, False):
        r = P.check_codes(set_code(q, 4, 3, 8), s, q, s, Y, exact=exact)
        assert r["zero_sign_only"] == 1 and r["code_mismatches"] == 0
    # undetermined zero: only the inexact kernels may differ
    assert P.check_codes(set_code(q, 4, 4, 8), s, q, s, Y, exact=False)["zero_sign_only"] == 1
    with pytest.raises(AssertionError, match="P0"):
        P.check_codes(set_code(q, 4, 4, 8), s, q, s, Y, exact=True)
    # a determined sign must be kept even though the magnitude code is 0
    with pytest.raises(AssertionError):
        P.check_codes(set_code(q, 4, 6, 8), s, q, s, Y, exact=False)


# ---- P3 --------------------------------------------------------------------------------------
def pow2_case(rel=3e-6):
    """One block whose amax sits just below 4: the oracle takes S = 126, the neighbouring S = 127 is allowed."""
    Y, _, _ = base_case()
    Y[10, 32:64] *= np.float32(0.5)                    # keep every other value of the block below the new amax
    Y[10, 32] = np.float32(4.0 * (1.0 - rel))
    q, s = co.mx_encode(Y)
    assert s[10, 1] == 126
    return Y, q, s


def reencode_block(Y, q, s, t, j, S):
    """The 'GPU' result of block (t, j) under scale byte S, worked here from first principles (nearest grid value)."""
    grid = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
    qg, sg = q.copy(), s.copy()
    sg[t, j] = S
    for c in range(32):
        v = float(Y[t, 32 * j + c]) * 2.0 ** (127 - S)
        dist = np.abs(abs(v) - grid)
        cands = np.flatnonzero(dist == dist.min())
        even = [int(i) for i in cands if i % 2 == 0]
        mag = even[0] if even else int(cands[0])
        if abs(v) > 6:
            mag = 7
        qg = set_code(qg, t, 32 * j + c, (8 if np.signbit(np.float32(v)) else 0) | mag)
    return qg, sg


def test_p3_accepts_the_neighbouring_scale_at_a_power_of_two():
    Y, q, s = pow2_case()
    qg, sg = reencode_block(Y, q, s, 10, 1, 127)
    assert not np.array_equal(qg, q)                   # the codes really change with the scale
    r = P.check_codes(qg, sg, q, s, Y, exact=False)
    assert r["scale_mismatches"] == 1 and r["code_mismatches"] == 0


def test_p3_rejects_neighbouring_scale_with_the_old_codes():
    Y, q, s = pow2_case()
    _, sg = reencode_block(Y, q, s, 10, 1, 127)
    with pytest.raises(AssertionError):
        P.check_codes(q, sg, q, s, Y, exact=False)     # scale changed, codes not re-encoded


def test_p3_rejects_for_an_exact_kernel():
    Y, q, s = pow2_case()
    qg, sg = reencode_block(Y, q, s, 10, 1, 127)
    with pytest.raises(AssertionError, match="P0"):
        P.check_codes(qg, sg, q, s, Y, exact=True)


def test_p3_rejects_a_scale_off_by_one_away_from_a_power_of_two():
    Y, q, s = base_case()
    Y = Y.copy()
    Y[10, 32] = np.float32(5.0)                        # amax 5: nowhere near a power of two
    q, s = co.mx_encode(Y)
    qg, sg = reencode_block(Y, q, s, 10, 1, int(s[10, 1]) + 1)
    with pytest.raises(AssertionError, match="not at a power of two"):
        P.check_codes(qg, sg, q, s, Y, exact=False)


def test_p3_rejects_a_scale_off_by_two():
    Y, q, s = pow2_case()
    qg, sg = reencode_block(Y, q, s, 10, 1, 128)
    with pytest.raises(AssertionError):
        P.check_codes(qg, sg, q, s, Y, exact=False)


def test_p3_rejects_too_many_scale_mismatches():
    Y, _, _ = base_case()
    blocks = [(t, 1) for t in range(10, 14)]           # 4 of 512 blocks > 1e-4 (limit: max(1, 0.05) = 1)
    for t, j in blocks:
        Y[t, 32 * j:32 * j + 32] *= np.float32(0.5)
        Y[t, 32 * j] = np.float32(4.0 * (1.0 - 3e-6))
    q, s = co.mx_encode(Y)
    qg, sg = q, s
    for t, j in blocks:
        qg, sg = reencode_block(Y, qg, sg, t, j, 127)
    with pytest.raises(AssertionError, match="scale mismatches"):
        P.check_codes(qg, sg, q, s, Y, exact=False)


# ---- P1 --------------------------------------------------------------------------------------
def test_p1_value_tolerance():
    Y, _, _ = base_case()
    big = np.abs(Y) >= 1.0
    ok = Y.astype(np.float64) * np.where(big, 1.0 + 5e-6, 1.0)
    assert P.check_values(ok.astype(np.float32), Y)["max_err_over_tol"] < 1.0
    bad = Y.astype(np.float64).copy()
    bad[7, 1] = Y[7, 1] * (1.0 + 2e-5) if abs(Y[7, 1]) >= 0.5 else Y[7, 1] + 4.0 * 2e-5
    with pytest.raises(AssertionError, match="P1"):
        P.check_values(bad, Y)
    # the floor: a small element may be off by 1e-5 * amax/32 but not by twice that
    small = Y.astype(np.float64).copy()
    t, c = 7, 2
    Yz = Y.copy()
    Yz[t, c] = 0.0
    small = Yz.astype(np.float64).copy()
    small[t, c] = 0.9e-5 * 4.0 / 32
    P.check_values(small, Yz)
    small[t, c] = 2e-5 * 4.0 / 32
    with pytest.raises(AssertionError, match="P1"):
        P.check_values(small, Yz)
