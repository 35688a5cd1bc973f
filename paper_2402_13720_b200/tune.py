"""Hyper-parameter search of the paper's Appendix B (Algorithm 1): a coordinate search on wall-clock time.

K is fixed (3 in the paper).  Starting from a point inside the recipe's ranges (Table "empirical recipe": gamma 7-14
for tasks where draft and target agree often, 2-6 where they do not; window W 15-20; phrase length beta 5-7), the
draft length is set to the value that minimises the measured time with the other two held at their starting values,
then the window with the new draft length, then the phrase length with both.  Three one-dimensional sweeps, not a
grid: the paper's observation is that the coordinates are stable enough for that.

`clock_time(gamma, window, beta, K)` is whatever the caller measures (bench.py --generate .. --tune times a generation
on the GPU); this module holds only the search, so it runs anywhere.
"""
from __future__ import annotations

RANGES = {"HH": {"gamma": (7, 14), "window": (15, 20), "beta": (5, 7)},
          "LH": {"gamma": (2, 6), "window": (15, 20), "beta": (5, 7)}}


def heuristic_search(clock_time, task_type="HH", k0=3, start=None, ranges=None):
    """Returns (gamma, window, beta, K, history).  `start` = (gamma, window, beta) inside the ranges (the paper draws it
    from them; default: the middle of each range).  Ties go to the smallest value.  `history` lists every evaluation
    (gamma, window, beta, K, time) in the order it was made; a setting is measured once."""
    r = dict(RANGES[task_type] if ranges is None else ranges)
    mid = lambda lo_hi: (lo_hi[0] + lo_hi[1]) // 2
    g_hat, w_hat, b_hat = start if start is not None else (mid(r["gamma"]), mid(r["window"]), mid(r["beta"]))
    for name, v in (("gamma", g_hat), ("window", w_hat), ("beta", b_hat)):
        if not r[name][0] <= v <= r[name][1]:
            raise ValueError(f"start value of {name} outside its range")
    seen, history = {}, []

    def t(g, w, b):
        key = (g, w, b, k0)
        if key not in seen:
            seen[key] = float(clock_time(g, w, b, k0))
            history.append(key + (seen[key],))
        return seen[key]

    def argmin(values, f):
        best = None
        for v in values:
            tv = f(v)
            if best is None or tv < best[1]:
                best = (v, tv)
        return best[0]

    span = lambda name: range(r[name][0], r[name][1] + 1)
    g0 = argmin(span("gamma"), lambda g: t(g, w_hat, b_hat))
    w0 = argmin(span("window"), lambda w: t(g0, w, b_hat))
    b0 = argmin(span("beta"), lambda b: t(g0, w0, b))
    return g0, w0, b0, k0, history
