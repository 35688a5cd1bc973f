"""Algorithm 1 of the paper's Appendix B (coordinate search of gamma, W, beta on wall-clock time), on closed-form clocks."""
import pytest

from paper_2402_13720_b200 import tune


def test_separable_clock_finds_the_minimum_of_every_coordinate():
    clock = lambda g, w, b, k: (g - 9) ** 2 + 2 * (w - 19) ** 2 + 3 * (b - 5) ** 2 + k
    g, w, b, k, hist = tune.heuristic_search(clock, "HH")
    assert (g, w, b, k) == (9, 19, 5, 3)
    # three one-dimensional sweeps, each setting measured once: 8 + 6 + 3 values minus the two revisited points
    assert len(hist) == 8 + 6 + 3 - 2 and len({h[:4] for h in hist}) == len(hist)


def test_order_of_the_sweeps_is_gamma_then_window_then_beta():
    """With a coupling between the coordinates the result depends on the order; worked by hand for this clock:
    start (4, 17, 6).  gamma sweep at W=17, beta=6: |g - 17/4| is smallest at g = 4.  Window sweep at gamma 4:
    (w - 4*4)^2 -> 16.  beta sweep: (b - 16/3)^2 over 5..7 -> 5."""
    clock = lambda g, w, b, k: abs(g - w / 4) + (w - 4 * g) ** 2 + (b - w / 3) ** 2
    g, w, b, k, hist = tune.heuristic_search(clock, "LH", start=(4, 17, 6))
    assert (g, w, b, k) == (4, 16, 5, 3)
    assert [h[:3] for h in hist[:5]] == [(2, 17, 6), (3, 17, 6), (4, 17, 6), (5, 17, 6), (6, 17, 6)]
    assert all(h[0] == 4 for h in hist[5:]) and all(h[1] == 16 for h in hist[-2:])


def test_ties_take_the_smallest_value_and_bad_starts_are_refused():
    g, w, b, k, _ = tune.heuristic_search(lambda *a: 1.0, "LH", k0=4)
    assert (g, w, b, k) == (2, 15, 5, 4)
    with pytest.raises(ValueError):
        tune.heuristic_search(lambda *a: 1.0, "LH", start=(9, 17, 6))
