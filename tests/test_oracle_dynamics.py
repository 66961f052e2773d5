"""Pins for the oracle's cart-pole dynamics (CPU only).

The paper (Sec. IV) shows the update only as an image, so the dynamics are
pinned by what physics and arithmetic fix: the Lagrangian equations of motion
solved as a 2x2 linear system, exact rational closed forms at theta = 0, the
mirror antisymmetry of the system, the linearised solution, strict-threshold
termination and stored worked steps that predate the oracle.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from paper_2301_13062_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "dynamics_vectors.txt")

G, MC, MP, L, F, TAU = 9.8, 1.0, 0.1, 0.5, 10.0, 0.02
XT = 2.4
TT = 12 * 2 * np.pi / 360


def lagrange_accel(z, a):
    """Accelerations from the two coupled equations of motion of a uniform pole
    (half-length L, mass MP) hinged on a cart (mass MC) pushed by +-F:
        (MC+MP) x'' + MP L cos(th) th'' = F + MP L th'^2 sin(th)
        cos(th) x'' + (4/3) L th''     = G sin(th)
    solved as a linear system (no algebraic elimination)."""
    _, _, th, thd = (float(v) for v in z)
    f = F if a else -F
    s, c = np.sin(th), np.cos(th)
    A = np.array([[MC + MP, MP * L * c], [c, 4.0 / 3.0 * L]])
    b = np.array([f + MP * L * thd * thd * s, G * s])
    xacc, thacc = np.linalg.solve(A, b)
    return xacc, thacc


def lagrange_step(z, a):
    xacc, thacc = lagrange_accel(z, a)
    x, xd, th, thd = (float(v) for v in z)
    return np.array([x + TAU * xd, xd + TAU * xacc, th + TAU * thd, thd + TAU * thacc])


def _rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            kind, z0, acts, want = (p.strip() for p in line.split("|"))
            rows.append((kind, [float(v) for v in z0.split()], [int(v) for v in acts.split()], want.split()))
    return rows


def test_accelerations_solve_the_lagrangian_system(oracle):
    for spread in ("live", "wide", "start"):
        zs = inputs.random_states(300, seed=3, spread=spread).astype(np.float64)
        for i in range(zs.shape[1]):
            for a in (0, 1):
                xa, ta = oracle.accel_f64(zs[:, i], a)
                xr, tr = lagrange_accel(zs[:, i], a)
                assert abs(xa - xr) <= 1e-11 * max(1.0, abs(xr))
                assert abs(ta - tr) <= 1e-11 * max(1.0, abs(tr))


def test_f64_step_is_explicit_euler_of_the_lagrangian_system(oracle):
    zs = inputs.random_states(200, seed=4, spread="live").astype(np.float64)
    for i in range(zs.shape[1]):
        for a in (0, 1):
            got, done = oracle.dynamics_f64(zs[:, i], a)
            want = lagrange_step(zs[:, i], a)
            np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
            assert done == bool(abs(want[0]) > XT or abs(want[2]) > TT)


def test_f32_step_tracks_f64_step(oracle):
    # One step from the same float32 state: float32 chain vs float64 chain. The
    # float32 constants (9.8f, 0.1f, ...) differ from the decimal ones by < 1 ulp each,
    # so a dropped term or swapped operand (>= 1e-3) is caught, rounding (<= ~1e-6) is not.
    for spread in ("live", "edge", "start"):
        zs = inputs.random_states(2000, seed=8, spread=spread)
        for i in range(zs.shape[1]):
            a = i & 1
            z32, _ = oracle.dynamics_f32(zs[:, i], a)
            z64, _ = oracle.dynamics_f64(zs[:, i].astype(np.float64), a)
            xa, ta = oracle.accel_f64(zs[:, i].astype(np.float64), a)
            rate = np.array([zs[1, i], xa, zs[3, i], ta])
            tol = 2e-6 * np.maximum(np.maximum(np.abs(z64), np.abs(zs[:, i])), TAU * np.abs(rate))
            assert np.all(np.abs(z32 - z64) <= tol), (spread, i)


def test_exact_first_step_from_rest(oracle):
    # theta = 0: sin = 0, cos = 1 exactly, so the step is rational arithmetic.
    mt = Fraction(11, 10)
    temp = Fraction(10) / mt
    thacc = (0 - temp) / (Fraction(1, 2) * (Fraction(4, 3) - Fraction(1, 10) / mt))
    xacc = temp - Fraction(1, 20) * thacc / mt
    assert (temp, thacc, xacc) == (Fraction(100, 11), Fraction(-600, 41), Fraction(400, 41))
    want = [Fraction(0), Fraction(1, 50) * xacc, Fraction(0), Fraction(1, 50) * thacc]
    assert want[1] == Fraction(8, 41) and want[3] == Fraction(-12, 41)
    z64, d = oracle.dynamics_f64([0, 0, 0, 0], 1)
    assert not d
    for g, w in zip(z64, want):
        assert abs(g - float(w)) < 1e-15
    z32, d = oracle.dynamics_f32([0, 0, 0, 0], 1)
    assert z32[0] == 0 and z32[2] == 0
    for g, w in zip(z32, want):
        assert abs(float(g) - float(w)) <= 2 ** -24 * abs(float(w)) * 2
    xa, ta = oracle.accel_f64([0, 0, 0, 0], 0)
    assert abs(xa + 400 / 41) < 1e-13 and abs(ta - 600 / 41) < 1e-13


def test_golden_worked_steps(oracle):
    kinds = set()
    for kind, z0, acts, want in _rows():
        kinds.add(kind)
        if kind == "exact":
            z, _ = oracle.dynamics_f64(z0, acts[0])
            for g, w in zip(z, want):
                assert abs(g - float(Fraction(w))) < 1e-15
        elif kind == "f64":
            z = np.array(z0, np.float64)
            zl = z.copy()
            for a in acts:
                z, d = oracle.dynamics_f64(z, a)
                zl = lagrange_step(zl, a)
            np.testing.assert_allclose(z, [float(w) for w in want], rtol=0, atol=5e-16)
            np.testing.assert_allclose(zl, [float(w) for w in want], rtol=0, atol=1e-13)
        elif kind == "f32bits":
            z = np.array(z0, np.float32)
            for a in acts:
                z, d = oracle.dynamics_f32(z, a)
            assert [int(v) for v in z.view(np.uint32)] == [int(w, 16) for w in want]
    assert kinds == {"exact", "f64", "f32bits"}


def test_done_by_both_thresholds_example(oracle):
    z, d = oracle.dynamics_f64([2.39, 0.6, 0.2, 0.5], 1)
    assert d and z[0] > XT and z[2] > TT
    z, d = oracle.dynamics_f32([2.39, 0.6, 0.2, 0.5], 1)
    assert d


def test_mirror_antisymmetry_is_bit_exact(oracle):
    # Reflecting the track (z -> -z, push left <-> push right) negates the result
    # exactly: every float32 op in the chain is odd or even under the reflection.
    for spread, seed in (("live", 1), ("edge", 2), ("wide", 3), ("start", 4)):
        z = inputs.random_states(25000, seed=seed, spread=spread)
        a = inputs.random_actions(z.shape[1], seed)
        r1 = oracle.step(z, seed=0, t=0, action_u8=a, want_pre_reset=True)
        r2 = oracle.step(-z, seed=0, t=0, action_u8=1 - a, want_pre_reset=True)
        # value equality: an exact cancellation rounds to +0 on both sides of the mirror
        assert np.array_equal(-r1["pre_reset"], r2["pre_reset"])
        nz = r1["pre_reset"] != 0
        assert np.array_equal((-r1["pre_reset"]).view(np.uint32)[nz], r2["pre_reset"].view(np.uint32)[nz])
        assert np.array_equal(r1["done"], r2["done"])


def test_alternating_force_keeps_symmetry_and_termination_steps(oracle):
    # From rest, push right then left: both velocities return to exactly 0.
    z = np.zeros(4, np.float32)
    z, _ = oracle.dynamics_f32(z, 1)
    z, _ = oracle.dynamics_f32(z, 0)
    assert z[1] == 0.0 and z[3] == 0.0 and z[0] > 0 and z[2] < 0

    def run(pattern, sign, f32=True):
        z = np.zeros(4, np.float32 if f32 else np.float64)
        xmax = 0.0
        for k in range(200):
            a = pattern[k % len(pattern)]
            a = a if sign > 0 else 1 - a
            z, d = (oracle.dynamics_f32 if f32 else oracle.dynamics_f64)(z, a)
            if d:
                return k + 1, xmax, z
            xmax = max(xmax, abs(float(z[0])))
        return None, xmax, z

    def run_lagrange(pattern):
        z = np.zeros(4)
        for k in range(200):
            z = lagrange_step(z, pattern[k % len(pattern)])
            if abs(z[0]) > XT or abs(z[2]) > TT:
                return k + 1, z
        return None, z

    for pattern, step_done, xbound in (([1, 0], 33, 0.068), ([1, 0, 0, 1], 66, 0.0132)):
        k_ref, z_ref = run_lagrange(pattern)
        assert k_ref == step_done and z_ref[2] < -TT
        for f32 in (True, False):
            k, xmax, z = run(pattern, +1, f32)
            km, xmaxm, zm = run(pattern, -1, f32)
            assert k == km == step_done
            assert xmax <= xbound and xmax == xmaxm
            assert np.array_equal(z, -zm)
            assert z[2] < -TT  # falls to the negative side after starting with a push right


def test_linearised_closed_form(oracle):
    # Small angles, constant push right: theta obeys th'' = a (th - th*) with
    # a = g (MC+MP) / (L (4/3 (MC+MP) - MP)) and th* = F / ((MC+MP) g); explicit Euler
    # then has eigenvalues 1 +- tau sqrt(a).
    mt = MC + MP
    a_lin = G * mt / (L * (4.0 / 3.0 * mt - MP))
    assert abs(a_lin - 9.8 * 66 / 41) < 1e-12
    th_star = F / (mt * G)
    ra = np.sqrt(a_lin)
    lp, lm = 1 + TAU * ra, 1 - TAU * ra
    z = np.array([0.0, 0.0, 1e-3, -2e-3])
    u0, v0 = z[2] - th_star, z[3]
    for k in range(1, 4):
        z, _ = oracle.dynamics_f64(z, 1)
        cp, cm = u0 + v0 / ra, u0 - v0 / ra
        th_k = th_star + 0.5 * (cp * lp ** k + cm * lm ** k)
        thd_k = 0.5 * ra * (cp * lp ** k - cm * lm ** k)
        assert abs(z[2] - th_k) < 2e-8 * k ** 2
        assert abs(z[3] - thd_k) < 2e-5 * k ** 2
    # and the cart: x'' = (F - MP L th'') / mt to first order
    xa, ta = oracle.accel_f64([0, 0, 1e-4, 0], 1)
    assert abs(xa - (F - MP * L * ta) / mt) < 1e-6


def test_strict_thresholds(oracle):
    xt = np.float32(2.4)
    tt = np.float32(TT)
    assert tt.view(np.uint32) == 0x3E567750 and xt.view(np.uint32) == 0x4019999A
    up = lambda v: np.nextafter(v, np.float32(np.inf), dtype=np.float32)
    # velocities chosen so that x' == x and theta' == theta exactly (tau * 0 = 0)
    for sign in (1, -1):
        for a in (0, 1):
            z, d = oracle.dynamics_f32([sign * xt, 0, 0, 0], a)
            assert z[0] == sign * xt and not d
            z, d = oracle.dynamics_f32([sign * up(xt), 0, 0, 0], a)
            assert d
            z, d = oracle.dynamics_f32([0, 0, sign * tt, 0], a)
            assert z[2] == sign * tt and not d
            z, d = oracle.dynamics_f32([0, 0, sign * up(tt), 0], a)
            assert d


def test_euler_uses_old_velocities_bitwise(oracle):
    # Position and angle updates are fl(x + fl(tau*x_dot)) with the OLD rates.
    z = inputs.random_states(5000, seed=12, spread="live")
    r = oracle.step(z, seed=0, t=0, action_u8=inputs.random_actions(5000, 1), want_pre_reset=True)
    tau = np.float32(0.02)
    assert np.array_equal(r["pre_reset"][0], z[0] + tau * z[1])
    assert np.array_equal(r["pre_reset"][2], z[2] + tau * z[3])
    # velocity updates move by tau * acceleration of the OLD state
    for i in range(0, 5000, 97):
        xa, ta = oracle.accel_f32(z[:, i], int(r["action"][i]))
        assert r["pre_reset"][1, i] == z[1, i] + tau * xa
        assert r["pre_reset"][3, i] == z[3, i] + tau * ta


def test_nan_and_inf_states_do_not_terminate_or_crash(oracle):
    for bad in (np.nan, np.inf, -np.inf):
        z, d = oracle.dynamics_f32([bad, 0, 0, 0], 1)
        assert d == (np.isinf(bad))  # inf compares beyond the threshold, NaN never does
        z, d = oracle.dynamics_f32([0, 0, np.nan, 0], 0)
        assert not d and np.isnan(z[2])


@pytest.mark.parametrize("a", [0, 1])
def test_force_sign(oracle, a):
    xa, ta = oracle.accel_f32([0, 0, 0, 0], a)
    assert (xa > 0) == bool(a) and (ta < 0) == bool(a)
