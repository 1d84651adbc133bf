"""Pins of the CPU oracle against things other than itself: exhaustive
rational enumeration (tests/_brute.py), hand-worked traces
(tests/golden/worked_examples.txt), closed forms, library routines on the
special cases that reduce to them, and the invariances the paper's
definitions imply."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import gar_oracle as O
from tests import _brute as B

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_examples.txt")


def _load_examples():
    examples, cur = [], None
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            tok = line.split()
            if tok[0] == "example":
                cur = {"name": tok[1], "n": int(tok[2]), "f": int(tok[3]),
                       "x": [int(v) for v in tok[4:]], "rounds": [], "expect": {}}
                examples.append(cur)
            elif tok[0] == "round":
                cur["rounds"].append({
                    "winner": int(tok[3]),
                    "set": [int(v) for v in tok[5].split(",")],
                    "scores": {int(p.split(":")[0]): int(p.split(":")[1])
                               for p in tok[7].split(",")},
                    "gaps": tuple(Fraction(v) for v in tok[9].split(","))})
            elif tok[0] == "expect":
                cur["expect"][tok[1]] = Fraction(tok[2])
    return examples


EXAMPLES = _load_examples()


# ---------------------------------------------------------------- distances
def test_distances_closed_forms():
    n, d = 6, 10007
    c = np.array([0.5, -1.0, 2.0, 2.0, 7.0, -3.5])
    G = np.repeat(c[:, None], d, axis=1).astype(np.float32)
    D = O.pairwise_sq_distances(G)
    want = d * (c[:, None] - c[None, :]) ** 2
    np.testing.assert_allclose(D, want, rtol=1e-13)
    assert np.all(np.diag(D) == 0) and np.array_equal(D, D.T)
    # one-hot rows: every pair at squared distance 2
    E = np.eye(5, 9000, dtype=np.float32)
    D = O.pairwise_sq_distances(E)
    assert np.array_equal(D, 2.0 * (1 - np.eye(5)))


def test_distances_integer_rows_exact_and_library():
    rng = np.random.default_rng(1)
    G = rng.integers(-50, 50, size=(7, 12345)).astype(np.float32)
    D = O.pairwise_sq_distances(G)
    Gi = G.astype(np.int64)
    for i in range(7):
        for j in range(7):
            assert D[i, j] == float(np.sum((Gi[i] - Gi[j]) ** 2))
    # library routine on a generic input
    X = rng.standard_normal((5, 7001)).astype(np.float32)
    D = O.pairwise_sq_distances(X)
    for i in range(5):
        for j in range(5):
            ref = np.linalg.norm(X[i].astype(np.float64) - X[j].astype(np.float64)) ** 2
            assert abs(D[i, j] - ref) <= 1e-12 * max(ref, 1.0)


def test_distances_not_gram_transposed():
    # A transposed operand or a dropped cross term would break asymmetric data.
    G = np.array([[1, 2, 3, 4], [0, 0, 0, 0], [4, 3, 2, 1]], dtype=np.float32)
    D = O.pairwise_sq_distances(G)
    assert D[0, 1] == 30 and D[1, 2] == 30 and D[0, 2] == 9 + 1 + 1 + 9


def test_nonfinite_distance_is_infinite():
    G = np.ones((4, 10), dtype=np.float32)
    G[2, 3] = np.nan
    G[3, 1] = np.inf
    D = O.pairwise_sq_distances(G)
    assert np.isinf(D[2, 0]) and np.isinf(D[3, 1]) and np.isinf(D[2, 3])
    assert D[0, 1] == 0 and D[2, 2] == 0


# ------------------------------------------------------------------- scores
@pytest.mark.parametrize("n,f", [(5, 1), (7, 1), (7, 2), (9, 2), (9, 3)])
def test_scores_match_subset_enumeration(n, f):
    rng = np.random.default_rng(100 * n + f)
    rows = rng.integers(-20, 20, size=(n, 3))
    D = O.pairwise_sq_distances(rows.astype(np.float32))
    sc = O.krum_scores(D, range(n), f)
    q = n - f - 2
    for i in range(n):
        assert Fraction(sc[i]) == B.score(rows.tolist(), list(range(n)), i, q)


def test_self_is_not_a_neighbour():
    # Counting G_i itself (distance 0) among its k-f-2 closest would leave only
    # k-f-3 real neighbours; on example A that changes the order of the scores.
    ex = EXAMPLES[0]
    rows = [[v] for v in ex["x"]]
    n, f = ex["n"], ex["f"]
    alive = list(range(n))
    with_self = {i: B.score(rows, alive, i, n - f - 3) for i in alive}
    correct = {i: B.score(rows, alive, i, n - f - 2) for i in alive}
    D = O.pairwise_sq_distances(np.array(rows, dtype=np.float32))
    sc = O.krum_scores(D, alive, f)
    assert {i: Fraction(sc[i]) for i in alive} == correct
    assert sorted(alive, key=lambda i: (with_self[i], i)) != \
        sorted(alive, key=lambda i: (correct[i], i))


# ------------------------------------------------------------ golden traces
@pytest.mark.parametrize("ex", EXAMPLES, ids=lambda e: e["name"])
def test_worked_examples_rounds(ex):
    n, f = ex["n"], ex["f"]
    rows = [[v] for v in ex["x"]]
    G = np.array(rows, dtype=np.float32)
    D = O.pairwise_sq_distances(G)
    sel = O.select_rounds(D, n, f, n - 2 * f - 2)
    brute = B.rounds(rows, f, n - 2 * f - 2)
    assert len(sel.rounds) == len(ex["rounds"]) == n - 2 * f - 2
    for rnd, gold, (bw, bS, bsc) in zip(sel.rounds, ex["rounds"], brute):
        # golden file == exhaustive enumeration == oracle
        assert gold["winner"] == bw == rnd.winner
        assert gold["set"] == bS == sorted(rnd.selected)
        assert {i: Fraction(s) for i, s in gold["scores"].items()} == bsc
        assert {i: Fraction(s) for i, s in rnd.scores.items()} == bsc
        assert rnd.m == len(rnd.alive) - f - 2
    assert len(set(sel.winners)) == len(sel.winners)


@pytest.mark.parametrize("ex", EXAMPLES, ids=lambda e: e["name"])
def test_worked_examples_gaps(ex):
    """The relative score gaps of every round: hand values of the golden file ==
    exact fractions recomputed from the enumeration's scores == the oracle's."""
    n, f = ex["n"], ex["f"]
    rows = [[v] for v in ex["x"]]
    D = O.pairwise_sq_distances(np.array(rows, dtype=np.float32))
    sel = O.select_rounds(D, n, f, n - 2 * f - 2)
    brute = B.rounds(rows, f, n - 2 * f - 2)
    for rnd, gold, (_, bS, bsc) in zip(sel.rounds, ex["rounds"], brute):
        gw, gs = B.score_gaps(bsc, len(bS))
        assert (gw, gs) == gold["gaps"]
        assert abs(rnd.gap_winner - float(gw)) <= 1e-15
        assert abs(rnd.gap_set - float(gs)) <= 1e-15
    # what a plausible mistake would give on example A, round 0 (scores 30, 31 | 63, 102):
    # relative to the smaller score, absolute, or zero -- none equals the pinned 1/31 and 13/34
    if ex["name"] == "A":
        r0 = sel.rounds[0]
        for wrong in (1 / 30, 1.0, 0.0):
            assert abs(r0.gap_winner - wrong) > 1e-3
        for wrong in (39 / 63, 39.0, 0.0, 21 / 63):
            assert abs(r0.gap_set - wrong) > 1e-3
    assert sel.min_gap == min(min(float(a), float(b)) for a, b in (g["gaps"] for g in ex["rounds"]))


def test_gap_special_cases():
    """Exact ties give gap 0 (both sides then break them by index); non-finite scores."""
    # five identical rows and two far ones, f = 1: q = m = 4, the identical rows all score 0
    x = np.array([[1.0]] * 5 + [[50.0], [-70.0]], dtype=np.float32)
    rnd = O.multi_krum_round(O.pairwise_sq_distances(x), range(7), 1)
    assert [rnd.scores[i] for i in range(5)] == [0.0] * 5 and rnd.scores[5] > 0
    assert rnd.gap_winner == 0.0 and rnd.winner == 0              # s(1) = s(2) = 0: exact tie, lowest index
    assert rnd.selected == [0, 1, 2, 3] and rnd.gap_set == 0.0     # s(4) = s(5) = 0: exact tie again
    # equal positive scores: two mirrored pairs around a centre row
    y = np.array([[-2.0], [-1.0], [0.0], [1.0], [2.0]], dtype=np.float32)
    rnd = O.multi_krum_round(O.pairwise_sq_distances(y), range(5), 0)   # q = m = 3
    assert rnd.scores[1] == rnd.scores[3] == 1 + 1 + 4 and rnd.scores[2] == 1 + 1 + 4
    assert rnd.scores[0] == rnd.scores[4] == 1 + 4 + 9
    assert rnd.gap_winner == 0.0 and rnd.winner == 1 and rnd.gap_set == (14.0 - 6.0) / 14.0
    # rows with NaN / Inf are at infinite distance from everybody.  n = 6, f = 1: q = m = 3 of 5
    # others, the four finite rows keep finite scores, the two others score +inf and stay out
    w = np.array([[0.0], [1.0], [3.0], [6.0], [np.nan], [np.inf]], dtype=np.float32)
    D = O.pairwise_sq_distances(w)
    rnd = O.multi_krum_round(D, range(6), 1)
    assert [rnd.scores[i] for i in range(4)] == [46.0, 30.0, 22.0, 70.0]
    assert np.isinf(rnd.scores[4]) and np.isinf(rnd.scores[5])
    assert rnd.order[:4] == [2, 1, 0, 3] and rnd.gap_winner == 8.0 / 30.0 and rnd.gap_set == 24.0 / 70.0
    # too many non-finite rows for anybody to avoid them: every score is +inf, every gap a tie
    rnd = O.multi_krum_round(D, [0, 1, 4, 5], 0)                   # k = 4, q = 2 of 3 others
    assert all(np.isinf(v) for v in rnd.scores.values())
    assert rnd.gap_winner == 0.0 and rnd.gap_set == 0.0 and rnd.winner == 0
    # a finite score next to an infinite one cannot decide a round (a finite score needs
    # more finite rows than m); the gap function still orders it as "clear"
    assert O._rel_gap(3.0, np.inf) == np.inf and O._rel_gap(np.inf, np.inf) == 0.0
    assert O._rel_gap(0.0, 0.0) == 0.0 and O._rel_gap(0.0, 5.0) == 1.0 and O._rel_gap(2.0, 8.0) == 0.75


@pytest.mark.parametrize("n,f,m,seed", [(7, 1, 2, 0), (7, 1, 3, 1), (9, 2, 2, 2), (9, 2, 4, 3), (11, 2, 3, 4),
                                        (11, 2, 6, 5), (10, 1, 5, 6)])
def test_multi_krum_intermediate_m_matches_enumeration(n, f, m, seed):
    """Section 3 allows any m <= n-f-2: the average of the m best-scored gradients."""
    rng = np.random.default_rng(seed)
    d = 3
    rows = rng.integers(-30, 30, size=(n, d))
    rows[rng.choice(n, f, replace=False)] *= 7
    _, _, sc = B.multi_krum_round(rows.tolist(), list(range(n)), f)
    if len(set(sc.values())) != len(sc):
        pytest.skip("tied scores")
    assert 1 < m < n - f - 2
    want = B.multi_krum(rows.tolist(), f, m=m)
    got, rnd = O.multi_krum(rows.astype(np.float32), f, m=m)
    assert rnd.m == m and len(rnd.selected) == m
    for t in range(d):
        assert abs(got[t] - float(want[t])) <= 1e-12 * (1 + abs(float(want[t])))
    gw, gs = B.score_gaps(sc, m)
    assert abs(rnd.gap_set - float(gs)) <= 1e-15 and abs(rnd.gap_winner - float(gw)) <= 1e-15


@pytest.mark.parametrize("n,f,theta,seed", [(9, 1, 3, 0), (9, 1, 4, 1), (10, 1, 5, 2), (11, 1, 6, 3), (11, 1, 3, 4),
                                            (11, 2, 5, 5)])
def test_multi_bulyan_theta_option_matches_enumeration(n, f, theta, seed):
    """A shorter extraction loop (2f+1 <= theta <= n-2f-2 rounds): beta = theta-2f follows it."""
    rng = np.random.default_rng(50 + seed)
    d = 4
    rows = rng.integers(-30, 30, size=(n, d))
    rows[rng.choice(n, f, replace=False)] *= 9
    for _, _, sc in B.rounds(rows.tolist(), f, theta):
        if len(set(sc.values())) != len(sc):
            pytest.skip("tied scores")
    assert 2 * f + 1 <= theta <= n - 2 * f - 2
    want = B.multi_bulyan(rows.tolist(), f, theta=theta)
    got, sel, _ = O.multi_bulyan(rows.astype(np.float32), f, theta=theta)
    assert sel.theta == theta and sel.beta == theta - 2 * f and len(sel.rounds) == theta
    for t in range(d):
        assert abs(got[t] - float(want[t])) <= 1e-12 * (1 + abs(float(want[t])))


@pytest.mark.parametrize("ex", EXAMPLES, ids=lambda e: e["name"])
def test_worked_examples_outputs(ex):
    n, f = ex["n"], ex["f"]
    rows = [[v] for v in ex["x"]]
    G = np.array(rows, dtype=np.float32)
    exp = ex["expect"]
    tol = 1e-14

    def close(val, frac):
        return abs(float(val) - float(frac)) <= tol * max(1.0, abs(float(frac)))

    assert B.multi_bulyan(rows, f)[0] == exp["multi_bulyan"]
    assert close(O.aggregate("multi_bulyan", G, f)[0], exp["multi_bulyan"])
    assert B.multi_bulyan(rows, f, median_of_agr=True)[0] == exp["multi_bulyan_median_of_agr"]
    assert close(O.multi_bulyan(G, f, median_source="agr")[0][0],
                 exp["multi_bulyan_median_of_agr"])
    assert close(O.aggregate("krum", G, f)[0], exp["krum"])
    assert close(O.aggregate("multi_krum", G, f)[0], exp["multi_krum"])
    assert close(O.aggregate("average", G, f)[0], exp["average"])
    assert close(O.aggregate("median", G, f)[0], exp["median"])
    if "bulyan" in exp:
        assert B.bulyan(rows, f)[0] == exp["bulyan"]
        assert close(O.aggregate("bulyan", G, f)[0], exp["bulyan"])


# ------------------------------------------- whole rules vs the enumeration
@pytest.mark.parametrize("n,f,seed", [(7, 1, 0), (7, 1, 1), (8, 1, 2), (9, 1, 3),
                                      (11, 2, 4), (11, 2, 5), (10, 1, 6)])
def test_multi_bulyan_matches_enumeration(n, f, seed):
    rng = np.random.default_rng(seed)
    d = 4
    rows = rng.integers(-30, 30, size=(n, d))
    rows[rng.choice(n, f, replace=False)] *= 9          # far-away rows
    # distinct scores are needed for a unique answer; skip seeds with ties
    brute_rounds = B.rounds(rows.tolist(), f, n - 2 * f - 2)
    for _, _, sc in brute_rounds:
        if len(set(sc.values())) != len(sc):
            pytest.skip("tied scores")
    want = B.multi_bulyan(rows.tolist(), f)
    got = O.aggregate("multi_bulyan", rows.astype(np.float32), f)
    for t in range(d):
        assert abs(got[t] - float(want[t])) <= 1e-12 * (1 + abs(float(want[t])))


@pytest.mark.parametrize("n,f,seed", [(7, 1, 10), (8, 1, 11), (11, 2, 12), (9, 1, 13)])
def test_bulyan_matches_enumeration(n, f, seed):
    rng = np.random.default_rng(seed)
    d = 5
    rows = rng.integers(-30, 30, size=(n, d))
    want = B.bulyan(rows.tolist(), f)
    got = O.aggregate("bulyan", rows.astype(np.float32), f)
    for t in range(d):
        assert abs(got[t] - float(want[t])) <= 1e-12 * (1 + abs(float(want[t])))


# ------------------------------------------------------------ preconditions
def test_preconditions():
    for f in range(0, 6):
        with pytest.raises(O.PreconditionError):
            O.check_preconditions("multi_bulyan", 4 * f + 2, f)
        with pytest.raises(O.PreconditionError):
            O.check_preconditions("bulyan", 4 * f + 2, f)
        O.check_preconditions("multi_bulyan", 4 * f + 3, f)
        O.check_preconditions("bulyan", 4 * f + 3, f)
        with pytest.raises(O.PreconditionError):
            O.check_preconditions("multi_krum", 2 * f + 2, f)
        O.check_preconditions("krum", 2 * f + 3, f)
    O.check_preconditions("average", 1, 0)
    with pytest.raises(ValueError):
        O.check_preconditions("nope", 5, 1)


def test_every_round_meets_multi_krum_precondition():
    # With theta = n-2f-2 the last round still has k = 2f+3 gradients.
    for n, f in [(7, 1), (11, 2), (23, 5), (39, 9), (51, 12), (15, 3), (20, 3)]:
        rng = np.random.default_rng(n)
        G = rng.standard_normal((n, 50)).astype(np.float32)
        sel = O.select_rounds(O.pairwise_sq_distances(G), n, f, n - 2 * f - 2)
        ks = [len(r.alive) for r in sel.rounds]
        assert ks == list(range(n, 2 * f + 2, -1)) and ks[-1] == 2 * f + 3
        assert sel.beta == n - 4 * f - 2 >= 1


# ------------------------------------------------------- degenerate reductions
def test_median_rule_matches_libraries():
    rng = np.random.default_rng(3)
    G = rng.standard_normal((9, 501)).astype(np.float32)
    np.testing.assert_array_equal(O.coordinate_median(G), np.median(G.astype(np.float64), axis=0))
    G = rng.standard_normal((10, 501)).astype(np.float32)      # even count: lower middle
    want = torch.median(torch.from_numpy(G), dim=0).values.numpy().astype(np.float64)
    np.testing.assert_array_equal(O.coordinate_median(G), want)
    np.testing.assert_allclose(O.coordinate_median(G, even="mean"),
                               np.median(G.astype(np.float64), axis=0), rtol=1e-15)


def test_average_rule_matches_library():
    rng = np.random.default_rng(4)
    G = rng.standard_normal((13, 777)).astype(np.float32)
    np.testing.assert_allclose(O.average(G), G.astype(np.float64).mean(axis=0), rtol=1e-14, atol=1e-16)


def test_krum_is_an_input_row_and_multi_krum_m1():
    rng = np.random.default_rng(5)
    G = rng.standard_normal((9, 300)).astype(np.float32)
    out, rnd = O.krum(G, 2)
    assert np.array_equal(out, G[rnd.winner].astype(np.float64))
    out1, _ = O.multi_krum(G, 2, m=1)
    assert np.array_equal(out1, out)
    outm, rndm = O.multi_krum(G, 2)
    assert rndm.m == 9 - 2 - 2
    np.testing.assert_allclose(outm, G[sorted(rndm.selected)].astype(np.float64).mean(axis=0),
                               rtol=1e-14, atol=1e-16)


def test_bulyan_f0_is_averaging():
    rng = np.random.default_rng(6)
    G = rng.standard_normal((6, 400)).astype(np.float32)
    np.testing.assert_allclose(O.aggregate("bulyan", G, 0), G.astype(np.float64).mean(axis=0),
                               rtol=1e-13, atol=1e-15)


def test_coordinate_phase_beta_extremes():
    rng = np.random.default_rng(7)
    theta = 7
    ext = rng.standard_normal((theta, 1000))
    agr = rng.standard_normal((theta, 1000))
    out, M, gap = O.closest_to_median_average(ext, agr, theta)
    np.testing.assert_allclose(out, agr.mean(axis=0), rtol=1e-14, atol=1e-16)
    assert np.all(np.isinf(gap))
    # beta = 1 with agr = ext and an odd count is the coordinate-wise median
    out, M, _ = O.closest_to_median_average(ext, ext, 1)
    np.testing.assert_array_equal(out, np.median(ext, axis=0))
    np.testing.assert_array_equal(M, np.median(ext, axis=0))
    # the output always lies between the smallest and largest aggregated value
    out, _, _ = O.closest_to_median_average(ext, agr, 3)
    assert np.all(out >= agr.min(axis=0) - 1e-15) and np.all(out <= agr.max(axis=0) + 1e-15)


def test_coordinate_phase_keeps_the_closest():
    ext = np.array([[0.0], [10.0], [4.0], [5.0], [100.0]])        # median 5
    agr = np.array([[4.0], [7.0], [5.5], [-50.0], [6.9]])         # |a-M| = 1, 2, .5, 55, 1.9
    out, M, gap = O.closest_to_median_average(ext, agr, 3)
    assert M[0] == 5.0
    assert out[0] == pytest.approx((5.5 + 4.0 + 6.9) / 3)
    assert gap[0] == pytest.approx(2.0 - 1.9)
    # a tie is broken towards the lowest round
    agr2 = np.array([[6.0], [4.0], [5.0], [9.0], [9.0]])
    out, _, gap = O.closest_to_median_average(ext, agr2, 2)
    assert out[0] == 5.5 and gap[0] == 0.0
    cands = O.admissible_outputs(ext[:, 0], agr2[:, 0], 2, band=1e-9)
    assert sorted(cands) == [4.5, 5.5]


# ----------------------------------------------------------------- invariances
def _cluster(n, f, d, seed):
    rng = np.random.default_rng(seed)
    mu = rng.standard_normal(d)
    G = mu + 0.3 * rng.standard_normal((n, d))
    byz = rng.choice(n, f, replace=False)
    G[byz] = 20.0 * rng.standard_normal((f, d))
    return G.astype(np.float32), byz


@pytest.mark.parametrize("rule", ["krum", "multi_krum", "bulyan", "multi_bulyan", "median", "average"])
def test_row_permutation_invariance(rule):
    n, f, d = 11, 2, 200
    G, _ = _cluster(n, f, d, 21)
    perm = np.random.default_rng(22).permutation(n)
    a = O.aggregate(rule, G, f)
    b = O.aggregate(rule, G[perm], f)
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("rule", ["multi_krum", "bulyan", "multi_bulyan"])
def test_translation_scaling_coordinate_permutation(rule):
    n, f, d = 11, 2, 128
    G, _ = _cluster(n, f, d, 31)
    G = np.round(G * 64) / 64                      # keep shifts/scales exact in fp32
    base = O.aggregate(rule, G, f)
    shift = np.round(np.random.default_rng(32).standard_normal(d) * 8) / 8
    np.testing.assert_allclose(O.aggregate(rule, (G + shift).astype(np.float32), f),
                               base + shift, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(O.aggregate(rule, (G * 4).astype(np.float32), f),
                               base * 4, rtol=1e-12, atol=1e-12)
    cp = np.random.default_rng(33).permutation(d)
    np.testing.assert_allclose(O.aggregate(rule, G[:, cp], f), base[cp], rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("rule", ["krum", "multi_krum", "bulyan", "multi_bulyan"])
@pytest.mark.parametrize("n,f", [(7, 1), (11, 2), (15, 3), (23, 5)])
def test_equal_honest_rows_give_that_row(rule, n, f):
    # All n-f honest gradients equal v: whatever the f others are, every
    # honest score is 0 and the output is v.
    d = 64
    rng = np.random.default_rng(n * 10 + f)
    v = rng.standard_normal(d).astype(np.float32)
    G = np.repeat(v[None, :], n, axis=0)
    byz = rng.choice(n, f, replace=False)
    G[byz] = (rng.standard_normal((f, d)) * rng.choice([1e-3, 1.0, 1e4], size=(f, 1))).astype(np.float32)
    out = O.aggregate(rule, G, f)
    np.testing.assert_array_equal(out, v.astype(np.float64))


def test_identical_byzantine_rows_and_selection_is_honest():
    # f identical far-away rows (the shape of several workloads): never selected.
    n, f, d = 15, 3, 500
    G, _ = _cluster(n, 0, d, 41)
    byz = [2, 7, 11]
    G[byz] = -10.0 * G[[i for i in range(n) if i not in byz]].mean(axis=0)
    out, sel, _ = O.multi_bulyan(G, f)
    assert not (set(sel.winners) & set(byz))
    for S in sel.sets:
        assert not (set(S) & set(byz))
    D = O.pairwise_sq_distances(G)
    assert D[2, 7] == 0 and D[7, 11] == 0


# ------------------------------------------------------------------ the SGD step (Eq. 2)
def test_sgd_step_closed_form_and_library():
    rng = np.random.default_rng(3)
    x0 = rng.standard_normal(50)
    gs = [rng.standard_normal(50) for _ in range(4)]
    lr, mu = 0.1, 0.9
    # plain SGD: x_k = x_0 - lr * sum of the gradients
    x = x0.copy()
    for g in gs:
        x, v = O.sgd_step(x, g, lr)
        assert v is None
    np.testing.assert_allclose(x, x0 - lr * np.sum(gs, axis=0), rtol=0, atol=1e-14)
    # momentum: v_k = sum_i mu^(k-i) g_i (closed form), and PyTorch's SGD on the same numbers
    x, v = x0.copy(), np.zeros(50)
    px = torch.tensor(x0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([px], lr=lr, momentum=mu)
    for k, g in enumerate(gs):
        x, v = O.sgd_step(x, g, lr, momentum_buf=v, momentum=mu)
        want_v = sum(mu ** (k - i) * gs[i] for i in range(k + 1))
        np.testing.assert_allclose(v, want_v, rtol=0, atol=1e-13)
        px.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        np.testing.assert_allclose(x, px.detach().numpy(), rtol=0, atol=1e-13)
    # a sign or operand mix-up shows on a one-coordinate example: x = 1, g = 2, lr = 0.5 -> 0
    assert O.sgd_step([1.0], [2.0], 0.5)[0][0] == 0.0
    xn, vn = O.sgd_step([1.0], [2.0], 0.5, momentum_buf=[4.0], momentum=0.5)
    assert vn[0] == 4.0 and xn[0] == -1.0
