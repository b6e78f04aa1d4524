"""The scalar search logic of the product's conjugate-gradient module (Section 4.2: exponential step-size scheme that
brackets the minimum from the sign of the slope, then one quadratic interpolation), pinned on hand-worked cases.
Nothing here comes from the CPU checker's own copy of that logic: the expected brackets and vertices are worked out by
hand from the slope and error functions given."""
import math

from paper_1911_05181_b200.cg import ConjugateGradient as CG


def _counting(f):
    calls = []

    def g(a):
        calls.append(a)
        return f(a)
    return g, calls


def test_doubling_until_the_slope_turns_positive():
    # slope a - 5: negative at 1, 2, 4, positive at 8 -> bracket (4, 8) after four slope evaluations
    slope, calls = _counting(lambda a: a - 5.0)
    assert CG._bracket(slope, 1.0) == (4.0, 8.0, 4)
    assert calls == [1.0, 2.0, 4.0, 8.0]
    # already positive at the second step: (a0, 2 a0)
    assert CG._bracket(lambda a: a - 1.5, 1.0) == (1.0, 2.0, 2)


def test_halving_until_the_slope_turns_negative():
    # slope a - 0.3: non-negative at 1 and 0.5, negative at 0.25 -> bracket (0.25, 0.5) after three evaluations
    slope, calls = _counting(lambda a: a - 0.3)
    assert CG._bracket(slope, 1.0) == (0.25, 0.5, 3)
    assert calls == [1.0, 0.5, 0.25]
    # a slope that is exactly zero counts as "not negative"
    assert CG._bracket(lambda a: 0.0 if a == 1.0 else -1.0, 1.0) == (0.5, 1.0, 2)


def test_limits_of_the_two_schemes():
    # never negative: twelve halvings, lower end 0 (the caller then brackets again on all patterns)
    lo, hi, n = CG._bracket(lambda a: 1.0, 1.0)
    assert (lo, hi, n) == (0.0, 2.0 ** -12, 13)
    # always negative: thirty doublings; the bracket reported is the last two steps tried
    lo, hi, n = CG._bracket(lambda a: -1.0, 1.0)
    assert (lo, hi, n) == (2.0 ** 29, 2.0 ** 30, 31)
    lo, hi, n = CG._bracket(lambda a: -1.0, 1.0, max_doublings=1)
    assert (lo, hi, n) == (1.0, 2.0, 2)


def test_vertex_of_the_interpolating_parabola():
    f = lambda x: (x - 3.0) ** 2 + 1.0
    assert math.isclose(CG._vertex(1.0, f(1.0), 2.0, f(2.0), 4.0, f(4.0)), 3.0, rel_tol=1e-14)
    g = lambda x: 0.5 * (x + 2.0) ** 2 - 7.0          # vertex left of all three points
    assert math.isclose(CG._vertex(0.0, g(0.0), 1.0, g(1.0), 2.0, g(2.0)), -2.0, rel_tol=1e-13)
    # a parabola that opens downward, and three points on a line, have no minimum to interpolate
    assert CG._vertex(0.0, 0.0, 1.0, 1.0, 2.0, 0.0) is None
    assert CG._vertex(0.0, 0.0, 1.0, 1.0, 2.0, 2.0) is None
