"""Comparison helpers for the parity tests (CUDA path vs CPU oracle)."""
import numpy as np

from oracle import gar_oracle as O

TOL = 1e-5            # max |delta| <= TOL * (1 + |oracle|), fp32 outputs
GAP_REL = 1e-6        # selections must agree where the oracle's relative score gap exceeds this


def rule_tables(rule, G, f, D=None, **kw):
    """Oracle output + (winners, sets or None, beta, gap, selection) for a rule."""
    G = np.asarray(G)
    n = G.shape[0]
    if rule == "average":
        return O.average(G), None
    even = kw.get("even", "lower")
    if rule == "median":
        return O.coordinate_median(G, even=even), None
    if D is None:
        D = O.pairwise_sq_distances(G)
    if rule == "krum":
        out, rnd = O.krum(G, f, D=D)
        return out, dict(winners=[rnd.winner], sets=None, beta=1, gap=None, rounds=[rnd])
    if rule == "multi_krum":
        out, rnd = O.multi_krum(G, f, D=D, m=kw.get("m"))
        return out, dict(winners=[rnd.winner], sets=[sorted(rnd.selected)], beta=1, gap=None, rounds=[rnd])
    if rule == "bulyan":
        out, sel, gap = O.bulyan(G, f, D=D, even=even)
        return out, dict(winners=sel.winners, sets=None, beta=sel.beta, gap=gap, rounds=sel.rounds)
    out, sel, gap = O.multi_bulyan(G, f, D=D, theta=kw.get("theta"),
                                   median_source="agr" if kw.get("median_of_agr") else "ext", even=even)
    return out, dict(winners=sel.winners, sets=sel.sets, beta=sel.beta, gap=gap, rounds=sel.rounds)


def assert_outputs_match(got, want, G=None, tables=None, median_source="ext", tol=TOL, cols=None, even="lower",
                         max_tie_frac=2e-4):
    """Element-wise bar max|delta| <= tol*(1+|oracle|).  A coordinate outside the
    bar is accepted only if the oracle's gap between the beta-th and (beta+1)-th
    closest value is within a rounding band AND the value equals one of the
    averages obtainable by breaking that near-tie differently.  Returns the
    number of such coordinates (must stay a tiny fraction)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape
    err = np.abs(got - want)
    bad = np.nonzero(~(err <= tol * (1.0 + np.abs(want))))[0]
    if bad.size == 0:
        return 0
    assert tables is not None and tables.get("gap") is not None and G is not None, \
        f"{bad.size} coordinates outside the bar, max err {err[bad].max():.3e} at {bad[:5]}"
    assert bad.size <= max(3, int(max_tie_frac * got.size)), f"{bad.size} of {got.size} coordinates outside the bar"
    G = np.asarray(G)
    for t in bad:
        col = t if cols is None else cols[t]
        ext, agr = O.extracted_and_aggregated(G[:, col:col + 1], tables["winners"], tables["sets"])
        band = 1e-5 * (1.0 + np.abs(agr[:, 0]).max())
        assert tables["gap"][t] <= band, f"coordinate {col}: err {err[t]:.3e} with a clear gap {tables['gap'][t]:.3e}"
        cands = O.admissible_outputs(ext[:, 0], agr[:, 0], tables["beta"], band, median_source=median_source, even=even)
        assert any(abs(got[t] - c) <= tol * (1.0 + abs(c)) for c in cands), \
            f"coordinate {col}: {got[t]} matches no admissible average {cands}"
    return int(bad.size)


def assert_selection_match(sel_host, rounds, preagg):
    """Winners (and sets when pre-aggregating) identical in every round whose
    oracle gap exceeds GAP_REL; stops comparing after the first ambiguous round
    (later rounds depend on it).  Returns the number of rounds compared."""
    compared = 0
    for r, rnd in enumerate(rounds):
        gap = min(rnd.gap_winner, rnd.gap_set) if preagg else rnd.gap_winner
        if 0.0 < gap <= GAP_REL:      # near-tie: either order is a correct result
            return compared           # (an exact tie, gap == 0, is broken by index on both sides)
        assert sel_host.winners[r] == rnd.winner, f"round {r}: winner {sel_host.winners[r]} != {rnd.winner}"
        if preagg:
            mask = 0
            for i in rnd.selected:
                mask |= 1 << i
            assert sel_host.sets[r] == mask, f"round {r}: set {sel_host.sets[r]:x} != {mask:x}"
            assert sel_host.m[r] == rnd.m
        compared += 1
    return compared
