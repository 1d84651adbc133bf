"""Exhaustive, exact-rational restatement of the paper's definitions for tiny
inputs.  It is deliberately a different program from the oracle: scores come
from enumerating every neighbour subset (Eq. 4: the sum over the k-f-2 closest
gradients is the minimum of that sum over all (k-f-2)-subsets of the others),
selections from enumerating every m-subset of the remaining gradients, the
median from its rank definition and the kept values from enumerating every
beta-subset.  Only usable for n up to about 11."""
from fractions import Fraction
from itertools import combinations


def F(x):
    return Fraction(x)


def sqdist(u, v):
    return sum((F(a) - F(b)) ** 2 for a, b in zip(u, v))


def score(rows, alive, i, q):
    others = [j for j in alive if j != i]
    return min(sum(sqdist(rows[i], rows[j]) for j in sub)
               for sub in combinations(others, q))


def multi_krum_round(rows, alive, f, clamp=False, m=None):
    k = len(alive)
    q = k - f - 2
    if clamp:
        q = max(q, 1)
    sc = {i: score(rows, alive, i, q) for i in alive}
    best = min(sc.values())
    winner = min(i for i in alive if sc[i] == best)
    if m is None:
        m = q
    # (m)argmin: the m-subset with the smallest total score; among equal
    # totals the lexicographically smallest index tuple (lowest-index ties).
    best_sub = min(combinations(sorted(alive), m),
                   key=lambda sub: (sum(sc[i] for i in sub), sub))
    return winner, sorted(best_sub), sc


def rounds(rows, f, theta, clamp=False):
    alive = list(range(len(rows)))
    out = []
    for _ in range(theta):
        w, S, sc = multi_krum_round(rows, alive, f, clamp)
        out.append((w, S, sc))
        alive.remove(w)
    return out


def score_gaps(sc, m):
    """Exact relative gaps of one round: between the two smallest scores, and
    between the m-th and the (m+1)-th smallest (None where there is no such pair)."""
    s = sorted(sc.values())
    gap_w = (s[1] - s[0]) / s[1] if len(s) > 1 and s[1] > 0 else None
    gap_s = (s[m] - s[m - 1]) / s[m] if m < len(s) and s[m] > 0 else None
    return gap_w, gap_s


def multi_krum(rows, f, m=None):
    """Average of the m best-scored gradients (Eq. 4's (m)arg-min), any 1 <= m <= n-f-2."""
    _, S, _ = multi_krum_round(rows, list(range(len(rows))), f, m=m)
    return mean_rows(rows, S)


def lower_median(vals):
    vals = list(vals)
    cnt = len(vals)
    target = (cnt - 1) // 2
    for v in vals:
        less = sum(1 for u in vals if u < v)
        leq = sum(1 for u in vals if u <= v)
        if less <= target < leq:
            return v
    raise AssertionError


def closest_average(ext, agr, beta):
    """Per coordinate, by enumeration of every beta-subset of the rounds."""
    theta = len(agr)
    d = len(agr[0])
    out = []
    for t in range(d):
        M = lower_median([ext[r][t] for r in range(theta)])
        key = [abs(agr[r][t] - M) for r in range(theta)]
        sub = min(combinations(range(theta), beta),
                  key=lambda s: (sorted((key[r] for r in s), reverse=True), s))
        out.append(sum(agr[r][t] for r in sub) / beta)
    return out


def mean_rows(rows, idx):
    d = len(rows[0])
    return [sum(F(rows[i][t]) for i in idx) / len(idx) for t in range(d)]


def multi_bulyan(rows, f, theta=None, median_of_agr=False):
    n = len(rows)
    if theta is None:
        theta = n - 2 * f - 2
    rs = rounds(rows, f, theta)
    ext = [[F(x) for x in rows[w]] for w, _, _ in rs]
    agr = [mean_rows(rows, S) for _, S, _ in rs]
    return closest_average(agr if median_of_agr else ext, agr, theta - 2 * f)


def bulyan(rows, f):
    n = len(rows)
    theta = n - 2 * f
    rs = rounds(rows, f, theta, clamp=True)
    ext = [[F(x) for x in rows[w]] for w, _, _ in rs]
    return closest_average(ext, ext, theta - 2 * f)
