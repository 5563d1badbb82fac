"""Exact minimiser of ||x - alpha*[x/alpha]_Zp||^2 over alpha, by breakpoint enumeration.

A checker for tiny inputs, independent of the oracle: for fixed codes q the objective is the
quadratic sum(x^2) - 2*alpha*<x,q> + alpha^2*<q,q>, and the codes change only where some
x_i/alpha crosses a half-integer k+1/2 with lo <= k < hi, i.e. at alpha = x_i/(k+1/2).
Between consecutive breakpoints the codes are constant, so the minimum over an interval is
at the clipped vertex or at an end.  Everything in float64.
"""
import numpy as np


def exact_optimum(x, lo, hi, a_max=None):
    """Return (sse, alpha, codes) minimising over 0 < alpha <= a_max (default: everywhere)."""
    x = np.asarray(x, dtype=np.float64)
    top = 2.0 * np.max(np.abs(x)) * 1.0000001 + 1e-300   # above this every code is 0
    if a_max is None:
        a_max = top
    bps = set()
    for xi in x:
        if xi == 0.0:
            continue
        for k in range(lo, hi):
            b = xi / (k + 0.5)
            if 0.0 < b < a_max:
                bps.add(b)
    edges = [0.0] + sorted(bps) + [a_max]
    best = (np.inf, None, None)
    for left, right in zip(edges[:-1], edges[1:]):
        if not right > left:
            continue
        mid = 0.5 * (left + right)
        q = np.clip(np.rint(x / mid), lo, hi)
        sqq, sxq = float(q @ q), float(x @ q)
        trial = [right]
        if left > 0.0:
            trial.append(left)
        if sqq > 0.0 and left <= sxq / sqq <= right:
            trial.append(sxq / sqq)
        for a in trial:
            d = x - a * q
            s = float(d @ d)
            if s < best[0]:
                best = (s, a, q.copy())
    return best
