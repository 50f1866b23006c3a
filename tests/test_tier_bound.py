"""The exit similarity of the locality-ordered search (host arithmetic of the library) against the geometry it rests
on: a closed form, the tight great-circle configuration on both sides of the bound, and random search for a violation."""
import math

import numpy as np
import pytest

siso = pytest.importorskip("paper_2508_18736_b200")

MARGIN = 1e-5          # what the library adds for the rounding of computed similarities


def exit_sim(sep, slack=0.0):
    return siso.tier_exit_sim(sep, slack)


@pytest.mark.parametrize("sep", [0.0, 0.3, 0.6, 0.86, 0.95, 0.999])
def test_unit_vectors_give_the_half_angle(sep):
    # without slack the condition is angle(q, h) < acos(sep) / 2, i.e. s > sqrt((1 + sep) / 2)
    assert exit_sim(sep) == pytest.approx(math.sqrt((1 + sep) / 2) + MARGIN, abs=1e-12)
    assert exit_sim(-0.5) == exit_sim(0.0)                     # negative bounds are treated as 0 (conservative)


def test_no_exit_when_entries_may_coincide_and_bad_arguments():
    assert math.isinf(exit_sim(1.0)) and math.isinf(exit_sim(1.2)) and math.isinf(exit_sim(float("nan")))
    assert math.isinf(exit_sim(0.999, 1e-3))                   # sep / (1 - d)^2 >= 1
    assert math.isinf(exit_sim(0.5, -1e-3)) and math.isinf(exit_sim(0.5, 0.3))
    seps = np.linspace(0, 0.99, 50)
    vals = [exit_sim(s, 1e-3) for s in seps]
    assert all(b > a for a, b in zip(vals, vals[1:]))          # a looser separation needs a higher similarity
    assert all(exit_sim(s, 1e-3) > exit_sim(s) for s in seps)  # and so do looser norms


@pytest.mark.parametrize("sep,slack", [(0.86, 0.0), (0.86, 2e-3), (0.4, 1e-3), (0.97, 1e-4)])
def test_great_circle_configuration_is_tight(sep, slack):
    """h, q, c on one great circle with c as close to h as allowed is the worst case.  Just above the exit similarity the
    cold entry loses; just below the slack-free half angle it wins, so the bound is not merely safe but sharp."""
    e = exit_sim(sep, slack) - MARGIN
    up, dn = 1 + slack, 1 - slack
    beta = math.acos(min(1.0, sep / (dn * dn)))                # smallest hot/cold angle the bound allows
    # worst norms for the exit: |q| |h| as large as allowed makes the angle to h as large as s permits
    alpha = math.acos(min(1.0, e * (1 + 1e-9) / (up * up)))
    h = np.array([up, 0.0])
    q = up * np.array([math.cos(alpha), math.sin(alpha)])
    c = up * np.array([math.cos(beta), math.sin(beta)])
    assert q @ h >= e and q @ c < q @ h
    if slack == 0.0:
        a2 = beta / 2 * (1 + 1e-6)                             # a hair past the half angle: the cold entry is nearer
        q2 = np.array([math.cos(a2), math.sin(a2)])
        assert q2 @ c > q2 @ h and q2 @ h < e


def test_random_search_finds_no_violation():
    rng = np.random.default_rng(5)
    worst, checked = -9.0, 0
    for trial in range(300):
        dim = int(rng.integers(2, 9))
        slack = float(rng.choice([0.0, 1e-4, 2e-3, 1e-2]))
        h = rng.standard_normal(dim)
        h /= np.linalg.norm(h)
        C = rng.standard_normal((400, dim))
        C /= np.linalg.norm(C, axis=1, keepdims=True)
        # pull half of the cold entries towards h: the dangerous ones are those right at the separation bound
        C[:200] = C[:200] * 0.3 + h * rng.uniform(0.5, 3.0, (200, 1))
        C /= np.linalg.norm(C, axis=1, keepdims=True)
        scale = lambda n: rng.uniform(1 - slack, 1 + slack, n)
        hs = h * scale(1)
        Cs = C * scale(400)[:, None]
        sep = float((Cs @ hs).max())
        e = exit_sim(sep, slack)
        if math.isinf(e):
            continue
        Q = h + rng.standard_normal((4000, dim)) * rng.uniform(0.01, 0.6)
        Q /= np.linalg.norm(Q, axis=1, keepdims=True)
        # and queries pushed from h towards the nearest cold entry, where a violation would show first
        near = Cs[np.argmax(Cs @ hs)]
        t = rng.uniform(0, 0.6, (2000, 1))
        Q2 = (1 - t) * h + t * near / np.linalg.norm(near)
        Q = np.concatenate([Q, Q2 / np.linalg.norm(Q2, axis=1, keepdims=True)]) * scale(6000)[:, None]
        s = Q @ hs
        done = s > e
        checked += int(done.sum())
        if done.any():
            worst = max(worst, float(((Q[done] @ Cs.T).max(axis=1) - s[done]).max()))
    # every query that may stop has all cold entries strictly below it, and queries right at the edge were among them
    assert checked > 100000 and -0.05 < worst < 0.0, (checked, worst)
