"""The selection rule as the paper defines it.  TEST INFRASTRUCTURE ONLY.

Section 3.3 defines max-variance down-sampling as the m-subset S of the n
rollouts that maximises Var({r_i : i in S}); the proof of Lemma 3.1 writes the
variance as (1/m) sum r^2 - ((1/m) sum r)^2.  This module evaluates exactly that
over every subset, in rational arithmetic (every finite float is a rational), so
it is usable only for tiny n.  It knows nothing of sorting or of Algorithm 2.
"""
from fractions import Fraction
from itertools import combinations


def variance_exact(values):
    """Population variance (1/m) sum x^2 - ((1/m) sum x)^2 as a Fraction."""
    xs = [Fraction(float(v)) for v in values]
    m = len(xs)
    mean = sum(xs) / m
    return sum(x * x for x in xs) / m - mean * mean


def max_variance_subsets(rewards, m):
    """Return (max variance as a Fraction, list of every m-subset attaining it)."""
    n = len(rewards)
    best, argbest = None, []
    for S in combinations(range(n), m):
        v = variance_exact([rewards[i] for i in S])
        if best is None or v > best:
            best, argbest = v, [S]
        elif v == best:
            argbest.append(S)
    return best, argbest
