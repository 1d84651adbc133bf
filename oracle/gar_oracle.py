"""Slow, plain fp64 CPU statement of the gradient aggregation rules (GARs) of
"Fast and Robust Distributed Learning in High Dimension" (multi-Bulyan paper).

THIS IS TEST INFRASTRUCTURE.  It is the oracle the CUDA path is compared with.
It shares no code with the CUDA path, imports nothing from the product package
and must never be called from it.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it.

Everything is written in the paper's order and notation:

* Eq. 4 and Algorithm 1 (function multi-Krum): for every remaining gradient
  G_i the score is the sum of the squared l2 distances to its k-f-2 closest
  other gradients; the winner has the smallest score; the output is the
  average of the m = k-f-2 gradients with the smallest scores.
* Algorithm 1 (function multi-Bulyan): theta = n-2f-2 rounds of multi-Krum on
  the gradients not yet extracted; each round stores its winner in G^ext and
  its average in G^agr and removes the winner; M = coordinate-wise median of
  G^ext; per coordinate the beta = theta-2f entries of G^agr closest to M are
  averaged.
* Section 2.2 (one-sentence Bulyan): coordinate-wise median of the selected
  vectors, then the average of the (count-2f) values closest to that median.

Readings taken where the text is silent (also listed in the design notes):
a gradient is not its own neighbour; f stays fixed while k shrinks; the loop of
multi-Bulyan runs theta times; ties are broken by the lowest index (lowest
round in the coordinate phase); the median of an even count is the lower
middle value; a non-finite distance counts as +infinity.

Parity pins live in tests/test_oracle_*.py (brute force over subsets on tiny
inputs, hand-worked traces under tests/golden/, closed forms, invariances and
degenerate reductions).  Unpinned: which of the two theta conventions
(n-2f-2 in Algorithm 1, n-2f in the proof of Theorem 2) the authors ran; both
are implemented ("multi_bulyan" and "bulyan").
"""
from __future__ import annotations

import itertools
from dataclasses import dataclass, field

import numpy as np

RULES = ("average", "median", "krum", "multi_krum", "bulyan", "multi_bulyan")


class PreconditionError(ValueError):
    """n, f violate the rule's requirement (Section 2.2: n >= 2f+3, n >= 4f+3)."""


def check_preconditions(rule: str, n: int, f: int) -> None:
    """Section 2.2: multi-Krum needs n >= 2f+3, (multi-)Bulyan n >= 4f+3."""
    if rule not in RULES:
        raise ValueError(f"unknown rule {rule!r}")
    if n < 1 or f < 0:
        raise ValueError("need n >= 1 and f >= 0")
    if rule in ("krum", "multi_krum") and n < 2 * f + 3:
        raise PreconditionError(f"{rule}: need n >= 2f+3, got n={n}, f={f}")
    if rule in ("bulyan", "multi_bulyan") and n < 4 * f + 3:
        raise PreconditionError(f"{rule}: need n >= 4f+3, got n={n}, f={f}")


# --------------------------------------------------------------------------
# Distances (Algorithm 1, multi-Krum: "k-f-2 closest (l2 norm) vectors",
# "sum of ||G_i - G||^2"): D_ij = sum_t (G_i[t] - G_j[t])^2.
# --------------------------------------------------------------------------
def pairwise_sq_distances(G, block: int = 4096) -> np.ndarray:
    """n x n matrix of squared l2 distances, fp64, symmetric, zero diagonal.

    The input values (whatever their dtype) are promoted to fp64 first.  The
    sum over coordinates is taken block by block (numpy's pairwise summation
    inside a block, sequential over blocks); its own rounding error is far
    below 1e-12 relative.  Non-finite results are replaced by +inf.
    """
    G = np.asarray(G)
    n, d = G.shape
    D = np.zeros((n, n), dtype=np.float64)
    with np.errstate(invalid="ignore", over="ignore"):
        for t0 in range(0, d, block):
            X = G[:, t0:t0 + block].astype(np.float64)
            for i in range(n - 1):
                diff = X[i + 1:] - X[i]
                D[i, i + 1:] += np.sum(diff * diff, axis=1)
    D = D + D.T
    D[~np.isfinite(D)] = np.inf
    np.fill_diagonal(D, 0.0)
    return D


# --------------------------------------------------------------------------
# Scores and one multi-Krum call (Eq. 4; Algorithm 1, function multi-Krum)
# --------------------------------------------------------------------------
def krum_scores(D: np.ndarray, alive, f: int, clamp: bool = False) -> dict:
    """score[i] = sum of the q = k-f-2 smallest D[i][j], j alive, j != i.

    k = number of alive gradients.  `clamp` (only for the n-2f-round variant,
    whose last rounds have k < 2f+3) uses q = max(k-f-2, 1).  The q values are
    added in ascending order, one by one.
    """
    alive = list(alive)
    k = len(alive)
    q = k - f - 2
    if clamp:
        q = max(q, 1)
    if q < 1:
        raise PreconditionError(f"k-f-2 = {q} < 1 neighbours (k={k}, f={f})")
    scores = {}
    for i in alive:
        vals = sorted(float(D[i, j]) for j in alive if j != i)
        s = 0.0
        for v in vals[:q]:
            s += v
        scores[i] = s
    return scores


@dataclass
class Round:
    alive: list          # indices still present when the round starts
    scores: dict         # index -> score
    order: list          # alive indices by (score, index) ascending
    winner: int          # order[0]
    m: int               # k - f - 2 (clamped to >= 1 when `clamp`)
    selected: list       # order[:m]  (the gradients multi-Krum averages)
    gap_winner: float    # relative gap between the two smallest scores
    gap_set: float       # relative gap between the m-th and (m+1)-th scores


def _rel_gap(lo: float, hi: float) -> float:
    if not np.isfinite(hi):
        return np.inf if np.isfinite(lo) else 0.0
    if hi <= 0.0:
        return 0.0
    return (hi - lo) / hi


def multi_krum_round(D: np.ndarray, alive, f: int, clamp: bool = False,
                     m: int | None = None) -> Round:
    """One call of multi-Krum on the alive gradients (Algorithm 1)."""
    alive = list(alive)
    k = len(alive)
    scores = krum_scores(D, alive, f, clamp=clamp)
    order = sorted(alive, key=lambda i: (scores[i], i))
    m_default = k - f - 2
    if clamp:
        m_default = max(m_default, 1)
    if m is None:
        m = m_default
    if not (1 <= m <= m_default):
        raise ValueError(f"m={m} outside [1, {m_default}]")
    s = [scores[i] for i in order]
    gap_w = _rel_gap(s[0], s[1]) if k > 1 else np.inf
    gap_s = _rel_gap(s[m - 1], s[m]) if m < k else np.inf
    return Round(alive=alive, scores=scores, order=order, winner=order[0], m=m,
                 selected=order[:m], gap_winner=gap_w, gap_set=gap_s)


@dataclass
class Selection:
    theta: int
    beta: int
    rounds: list = field(default_factory=list)

    @property
    def winners(self):
        return [r.winner for r in self.rounds]

    @property
    def sets(self):
        return [sorted(r.selected) for r in self.rounds]

    @property
    def min_gap(self):
        return min(min(r.gap_winner, r.gap_set) for r in self.rounds)


def select_rounds(D: np.ndarray, n: int, f: int, theta: int,
                  clamp: bool = False) -> Selection:
    """theta successive multi-Krum calls; each removes its winner
    (Algorithm 1, multi-Bulyan loop: [G_1..G_n] minus G^ext)."""
    sel = Selection(theta=theta, beta=theta - 2 * f)
    alive = list(range(n))
    for _ in range(theta):
        rnd = multi_krum_round(D, alive, f, clamp=clamp)
        sel.rounds.append(rnd)
        alive = [i for i in alive if i != rnd.winner]
    return sel


def theta_of(rule: str, n: int, f: int) -> int:
    """Number of extraction rounds: n-2f-2 (Algorithm 1) for multi_bulyan,
    n-2f (proof of Theorem 2 (i)) for bulyan."""
    if rule == "multi_bulyan":
        return n - 2 * f - 2
    if rule == "bulyan":
        return n - 2 * f
    raise ValueError(rule)


# --------------------------------------------------------------------------
# Coordinate phase (Algorithm 1, multi-Bulyan: Median(G^ext), Argpartition of
# |G^agr - M| with beta, Average)
# --------------------------------------------------------------------------
def median_rows(V: np.ndarray, even: str = "lower") -> np.ndarray:
    """Coordinate-wise median over axis 0 of a (count x c) fp64 array."""
    count = V.shape[0]
    Vs = np.sort(V, axis=0)
    if count % 2 == 1 or even == "lower":
        return Vs[(count - 1) // 2]
    if even == "mean":
        return 0.5 * (Vs[count // 2 - 1] + Vs[count // 2])
    raise ValueError(even)


def extracted_and_aggregated(G, winners, sets):
    """G^ext[r] = G[winner_r]; G^agr[r] = average of G[i], i in set_r, added in
    ascending index order (sets=None: G^agr = G^ext).  fp64, shape theta x c."""
    G = np.asarray(G)
    ext = G[list(winners)].astype(np.float64)
    if sets is None:
        return ext, ext.copy()
    agr = np.zeros_like(ext)
    for r, S in enumerate(sets):
        acc = np.zeros(G.shape[1], dtype=np.float64)
        for i in sorted(S):
            acc = acc + G[i].astype(np.float64)
        agr[r] = acc / float(len(S))
    return ext, agr


def closest_to_median_average(ext: np.ndarray, agr: np.ndarray, beta: int,
                              median_source: str = "ext", even: str = "lower"):
    """Per coordinate: M = median of ext (or of agr), keep the beta entries of
    agr with the smallest |agr - M| (ties: lowest round first), average them.

    Returns (out, M, gap) where gap[t] is the difference between the
    (beta+1)-th and the beta-th smallest |agr - M| (inf when beta == theta).
    """
    theta = agr.shape[0]
    if not (1 <= beta <= theta):
        raise ValueError(f"beta={beta} outside [1, {theta}]")
    M = median_rows(ext if median_source == "ext" else agr, even=even)
    key = np.abs(agr - M[None, :])
    order = np.argsort(key, axis=0, kind="stable")
    acc = np.zeros(agr.shape[1], dtype=np.float64)
    for b in range(beta):
        acc = acc + np.take_along_axis(agr, order[b:b + 1], axis=0)[0]
    out = acc / float(beta)
    if beta < theta:
        ks = np.take_along_axis(key, order, axis=0)
        gap = ks[beta] - ks[beta - 1]
    else:
        gap = np.full(agr.shape[1], np.inf)
    return out, M, gap


def coordinate_phase(G, winners, sets, beta: int, median_source: str = "ext",
                     even: str = "lower", block: int = 1 << 16):
    """Whole coordinate phase over all columns of G, block by block."""
    G = np.asarray(G)
    d = G.shape[1]
    out = np.empty(d, dtype=np.float64)
    gap = np.empty(d, dtype=np.float64)
    for t0 in range(0, d, block):
        ext, agr = extracted_and_aggregated(G[:, t0:t0 + block], winners, sets)
        o, _, g = closest_to_median_average(ext, agr, beta, median_source, even)
        out[t0:t0 + block] = o
        gap[t0:t0 + block] = g
    return out, gap


def admissible_outputs(ext_col, agr_col, beta: int, band: float,
                       median_source: str = "ext", even: str = "lower"):
    """All outputs one coordinate may take when |agr - M| values closer than
    `band` to the beta-th smallest are treated as tied (the paper fixes no
    tie-break, and a rounding of agr at fp32 level may reorder such keys).
    Returns a list of candidate averages (at least the oracle's own)."""
    ext_col = np.asarray(ext_col, dtype=np.float64)
    agr_col = np.asarray(agr_col, dtype=np.float64)
    theta = agr_col.shape[0]
    M = median_rows((ext_col if median_source == "ext" else agr_col)[:, None], even)[0]
    key = np.abs(agr_col - M)
    kb = np.sort(key)[beta - 1]
    must = [r for r in range(theta) if key[r] < kb - band]
    free = [r for r in range(theta) if kb - band <= key[r] <= kb + band]
    need = beta - len(must)
    outs = []
    for combo in itertools.combinations(free, need):
        kept = must + list(combo)
        outs.append(float(np.sum(agr_col[kept]) / beta))
    return outs


# --------------------------------------------------------------------------
# The six rules
# --------------------------------------------------------------------------
def average(G):
    """Averaging GAR (Introduction): (1/n) sum_i G_i, rows added in index order."""
    G = np.asarray(G)
    acc = np.zeros(G.shape[1], dtype=np.float64)
    for i in range(G.shape[0]):
        acc = acc + G[i].astype(np.float64)
    return acc / float(G.shape[0])


def coordinate_median(G, even: str = "lower"):
    """Coordinate-wise Median GAR (Section 5)."""
    return median_rows(np.asarray(G).astype(np.float64), even=even)


def krum(G, f: int, D=None):
    """Krum: the single gradient with the smallest score (multi-Krum, m = 1)."""
    G = np.asarray(G)
    n = G.shape[0]
    check_preconditions("krum", n, f)
    if D is None:
        D = pairwise_sq_distances(G)
    rnd = multi_krum_round(D, range(n), f)
    return G[rnd.winner].astype(np.float64), rnd


def multi_krum(G, f: int, m: int | None = None, D=None):
    """multi-Krum: average of the m (default n-f-2) smallest-score gradients."""
    G = np.asarray(G)
    n = G.shape[0]
    check_preconditions("multi_krum", n, f)
    if D is None:
        D = pairwise_sq_distances(G)
    rnd = multi_krum_round(D, range(n), f, m=m)
    _, agr = extracted_and_aggregated(G, [rnd.winner], [rnd.selected])
    return agr[0], rnd


def multi_bulyan(G, f: int, D=None, theta: int | None = None,
                 median_source: str = "ext", even: str = "lower"):
    """Algorithm 1: theta = n-2f-2 rounds, pre-aggregated G^agr, beta = theta-2f."""
    G = np.asarray(G)
    n = G.shape[0]
    check_preconditions("multi_bulyan", n, f)
    if D is None:
        D = pairwise_sq_distances(G)
    if theta is None:
        theta = theta_of("multi_bulyan", n, f)
    sel = select_rounds(D, n, f, theta)
    out, gap = coordinate_phase(G, sel.winners, sel.sets, sel.beta,
                                median_source=median_source, even=even)
    return out, sel, gap


def bulyan(G, f: int, D=None, even: str = "lower"):
    """Bulyan over iterated Krum winners: theta = n-2f winners (scores
    recomputed on the remaining set, neighbour count clamped to >= 1), their
    coordinate-wise median, average of the beta = theta-2f selected values
    closest to it (Section 2.2; proof of Theorem 2 (i))."""
    G = np.asarray(G)
    n = G.shape[0]
    check_preconditions("bulyan", n, f)
    if D is None:
        D = pairwise_sq_distances(G)
    theta = theta_of("bulyan", n, f)
    sel = select_rounds(D, n, f, theta, clamp=True)
    out, gap = coordinate_phase(G, sel.winners, None, sel.beta, even=even)
    return out, sel, gap


# --------------------------------------------------------------------------
# The update the aggregate feeds (Eq. 2: x_{k+1} = x_k - gamma_k * GAR(...);
# Section 5.1 trains with a momentum of 0.9)
# --------------------------------------------------------------------------
def sgd_step(x, g, lr: float, momentum_buf=None, momentum: float = 0.0):
    """One SGD step with the aggregated gradient g.  Without a momentum buffer:
    x - lr * g (Eq. 2).  With one: v <- momentum * v + g, x <- x - lr * v (the
    heavy-ball form PyTorch's SGD uses, the optimiser of Section 5.1).  fp64;
    returns (x_new, v_new or None)."""
    x = np.asarray(x, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    if momentum_buf is None:
        return x - lr * g, None
    v = momentum * np.asarray(momentum_buf, dtype=np.float64) + g
    return x - lr * v, v


def aggregate(rule: str, G, f: int):
    """GAR(f, [G_1..G_n]) -> fp64 vector of dimension d."""
    G = np.asarray(G)
    check_preconditions(rule, G.shape[0], f)
    if rule == "average":
        return average(G)
    if rule == "median":
        return coordinate_median(G)
    if rule == "krum":
        return krum(G, f)[0]
    if rule == "multi_krum":
        return multi_krum(G, f)[0]
    if rule == "bulyan":
        return bulyan(G, f)[0]
    return multi_bulyan(G, f)[0]
