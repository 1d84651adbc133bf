"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same
seeded inputs: each kernel alone (distances, selection, coordinate phase) and
every rule end to end, at sizes that span several tiles and a ragged tail."""
import numpy as np
import pytest
import torch

from oracle import gar_oracle as O
from tests._compare import GAP_REL, assert_outputs_match, assert_selection_match, rule_tables

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
# (config, n, f) of the five workloads (all sit at n = 4f+3)
CONFIGS = [(1, 11, 2), (2, 23, 5), (3, 39, 9), (4, 51, 12), (5, 15, 3)]


@pytest.fixture(scope="module")
def pkg():
    import __graft_entry__ as entry
    entry.build()
    import paper_1905_04374_b200 as p
    return p


def draw(pkg, cfg, d, **kw):
    G, byz = pkg.workloads.make_gradients(cfg, d=d, device=DEV, **kw)
    return G, G.cpu().numpy(), byz


# ---------------------------------------------------------------- distances
@pytest.mark.parametrize("cfg,n,f", CONFIGS)
@pytest.mark.parametrize("d", [1, 3, 127, 4099, 4100, 262_148])
def test_distances(pkg, cfg, n, f, d):
    G, Gh, _ = draw(pkg, cfg, d)
    D = pkg.gar_pairwise_distances(G).cpu().numpy()
    want = O.pairwise_sq_distances(Gh)
    assert np.array_equal(D, D.T) and np.all(np.diag(D) == 0)
    rel = np.abs(D - want) / np.maximum(want, 1e-300)
    rel[want == 0] = np.abs(D[want == 0])
    assert rel.max() <= 1e-6, f"max relative distance error {rel.max():.3e}"
    # identical rows (several workloads have f identical Byzantine rows) give exactly 0
    assert np.all(D[want == 0] == 0)


@pytest.mark.parametrize("n", [1, 2, 7, 8, 9, 16, 17, 24, 25, 32, 33, 40, 41, 48, 49, 56, 57, 63, 64])
def test_distances_every_row_block_count(pkg, n):
    d = 5000 + n
    G = pkg.workloads.make_uniform(n, d, device=DEV, seed=n)
    D = pkg.gar_pairwise_distances(G).cpu().numpy()
    want = O.pairwise_sq_distances(G.cpu().numpy())
    np.testing.assert_allclose(D, want, rtol=1e-6, atol=0)
    assert np.array_equal(D, D.T)


def test_distances_strided_and_unaligned(pkg):
    n, d = 23, 10_001
    big = pkg.workloads.make_uniform(n, d + 7, device=DEV, seed=5)
    for view in (big[:, :d], big[:, 1:d + 1], big[:, 3:d - 2], big[:, 4:d]):
        D = pkg.gar_pairwise_distances(view).cpu().numpy()
        want = O.pairwise_sq_distances(view.cpu().numpy())
        np.testing.assert_allclose(D, want, rtol=1e-6, atol=0)


def test_distances_bit_reproducible(pkg):
    G, _, _ = draw(pkg, 3, 300_001)
    a = pkg.gar_pairwise_distances(G).clone()
    b = pkg.gar_pairwise_distances(G).clone()
    assert torch.equal(a, b)


def test_distances_nonfinite_rows(pkg):
    G, Gh, _ = draw(pkg, 1, 5000)
    G[3, 17] = float("nan")
    G[5, 4000] = float("inf")
    Gh = G.cpu().numpy()
    out = pkg.gar_aggregate("multi_bulyan", G, 2).cpu().numpy()
    want, sel, gap = O.multi_bulyan(Gh, 2)
    assert 3 not in sel.winners and 5 not in sel.winners
    assert np.all(np.isfinite(out))
    assert_outputs_match(out, want)


# The distance kernel for 16 < n <= 64, 16-byte-aligned rows and d >= 32768 forms the Gram matrix
# from exact integer limbs; the cases below reach it (the ones above mostly stop short of it).
@pytest.mark.parametrize("n", [17, 24, 25, 31, 32, 33, 40, 41, 47, 48, 49, 56, 57, 63, 64])
def test_distances_large_d_every_row_count(pkg, n):
    d = 33_000 + 4 * n
    G = pkg.workloads.make_uniform(n, d, device=DEV, seed=100 + n)
    G -= 0.5
    D = pkg.gar_pairwise_distances(G).cpu().numpy()
    want = O.pairwise_sq_distances(G.cpu().numpy())
    np.testing.assert_allclose(D, want, rtol=1e-6, atol=0)
    assert np.array_equal(D, D.T) and np.all(np.diag(D) == 0)


@pytest.mark.parametrize("n", [23, 39, 51])
@pytest.mark.parametrize("where", ["first", "middle", "late", "everywhere"])
def test_distances_exact_on_small_integers(pkg, n, where):
    """Rows of small integers, non-zero only in one band of columns: the squared distances are
    integers below 2^53 and every summation order gives them exactly, so any contribution that is
    dropped, doubled or filed under the wrong pair shows."""
    d = 148 * 128 * 70 + 8
    cols = torch.arange(d, device=DEV)
    band = {"first": cols < 148 * 128, "middle": (cols >= 148 * 128 * 20) & (cols < 148 * 128 * 21),
            "late": cols >= 148 * 128 * 69, "everywhere": cols >= 0}[where]
    c = torch.arange(1, n + 1, dtype=torch.float32, device=DEV)[:, None]
    sign = torch.where(cols % 3 == 0, -1.0, 1.0)[None, :]
    G = (c * sign) * band[None, :].to(torch.float32)
    G[n // 2] *= -1.0
    D = pkg.gar_pairwise_distances(G).cpu().numpy()
    want = O.pairwise_sq_distances(G.cpu().numpy())
    assert want.max() < 2.0 ** 53
    assert np.array_equal(D, want)


@pytest.mark.parametrize("n", [23, 39, 51])
def test_distances_growing_magnitudes(pkg, n):
    """The magnitude of every row doubles a dozen times along the columns, at a different place
    for every row: running sums are rescaled again and again while they are non-zero."""
    d = 1_200_004
    G = pkg.workloads.make_uniform(n, d, device=DEV, seed=7 * n) - 0.5
    cols = torch.arange(d, device=DEV)
    for i in range(n):
        G[i] *= torch.exp2(torch.floor(cols * (12.0 + (i % 5)) / d) - 6.0)
    G[3] = G[n - 1]                                    # two identical rows: exactly 0 between them
    D = pkg.gar_pairwise_distances(G).cpu().numpy()
    want = O.pairwise_sq_distances(G.cpu().numpy())
    np.testing.assert_allclose(D, want, rtol=1e-6, atol=0)
    assert D[3, n - 1] == 0 and np.array_equal(D, D.T)


def test_distances_large_d_strided_nonfinite_reproducible(pkg):
    n, d = 39, 50_000
    big = pkg.workloads.make_uniform(n, d + 12, device=DEV, seed=9) - 0.5
    for view in (big[:, :d], big[:, 4:d + 4], big[:, 8:d]):          # 16-byte-aligned starts, ld != d
        D = pkg.gar_pairwise_distances(view).cpu().numpy()
        want = O.pairwise_sq_distances(view.cpu().numpy())
        np.testing.assert_allclose(D, want, rtol=1e-6, atol=0)
    G = big[:, :d].contiguous()
    assert torch.equal(pkg.gar_pairwise_distances(G).clone(), pkg.gar_pairwise_distances(G).clone())
    G[5, 17] = float("nan")
    G[20, d - 1] = float("inf")
    G[38, 40_000] = float("-inf")
    D = pkg.gar_pairwise_distances(G).cpu().numpy()
    want = O.pairwise_sq_distances(G.cpu().numpy())
    bad = np.isinf(want)
    assert bad[5].sum() == n - 1 and bad[20].sum() == n - 1 and bad[38].sum() == n - 1
    assert np.array_equal(np.isinf(D), bad)
    np.testing.assert_allclose(D[~bad], want[~bad], rtol=1e-6, atol=0)


# ------------------------------------------------ selection from the oracle's D
@pytest.mark.parametrize("rule", ["krum", "multi_krum", "bulyan", "multi_bulyan"])
@pytest.mark.parametrize("cfg,n,f", CONFIGS)
def test_selection_given_oracle_distances(pkg, rule, cfg, n, f):
    _, Gh, _ = draw(pkg, cfg, 2000)
    D = O.pairwise_sq_distances(Gh)
    sel = pkg.read_selection(pkg.gar_select(rule, torch.from_numpy(D).to(DEV), n, f))
    _, tab = rule_tables(rule, Gh, f, D=D)
    preagg = rule in ("multi_krum", "multi_bulyan")
    assert sel.theta == len(tab["rounds"]) and sel.beta == tab["beta"] and sel.preagg == int(preagg)
    # same D on both sides: every round must agree, scores to fp64 rounding
    for r, rnd in enumerate(tab["rounds"]):
        assert sel.winners[r] == rnd.winner
        for i in rnd.alive:
            assert abs(sel.scores[r][i] - rnd.scores[i]) <= 1e-12 * max(rnd.scores[i], 1e-300)
        if preagg:
            assert sel.sets[r] == sum(1 << i for i in rnd.selected)
        if np.isfinite(rnd.gap_winner):
            assert abs(sel.gap_winner[r] - rnd.gap_winner) <= 1e-9
    assert 1 <= sel.nu <= n


def test_selection_integer_ties(pkg):
    # d = 1 integer inputs: exact score ties, broken towards the lowest index on both sides
    x = np.array([[5], [-40], [9], [2], [14], [0], [60], [7], [3], [11], [20]], dtype=np.float32)
    D = O.pairwise_sq_distances(x)
    sel = pkg.read_selection(pkg.gar_select("bulyan", torch.from_numpy(D).to(DEV), 11, 2))
    _, tab = rule_tables("bulyan", x, 2, D=D)
    assert [sel.winners[r] for r in range(7)] == tab["winners"] == [7, 0, 2, 8, 9, 3, 4]
    G = torch.from_numpy(x).to(DEV)
    assert pkg.gar_aggregate("bulyan", G, 2).item() == 7.0
    assert abs(pkg.gar_aggregate("multi_bulyan", G, 2).item() - 51 / 7) < 1e-6
    assert pkg.gar_aggregate("krum", G, 2).item() == 7.0


# ------------------------------------ coordinate phase from the oracle's tables
def _upload_tables(pkg, n, f, rule_id, winners, sets, beta, preagg, median_of_agr=0):
    h = pkg.GarSelection()
    h.n, h.f, h.rule, h.theta, h.beta = n, f, rule_id, len(winners), beta
    h.preagg, h.median_of_agr = preagg, median_of_agr
    for r, w in enumerate(winners):
        h.winners[r] = w
        S = sets[r] if sets is not None else [w]
        h.sets[r] = sum(1 << i for i in S)
    dev = pkg.write_selection(h, DEV)
    pkg.gar_schedule_from_tables(dev)
    return dev


@pytest.mark.parametrize("cfg,n,f", CONFIGS)
@pytest.mark.parametrize("rule", ["bulyan", "multi_bulyan"])
@pytest.mark.parametrize("d", [1, 5, 1023, 70_001, 70_004])
def test_coordinate_phase_given_oracle_tables(pkg, cfg, n, f, rule, d):
    G, Gh, _ = draw(pkg, cfg, d)
    want, tab = rule_tables(rule, Gh, f)
    preagg = int(rule == "multi_bulyan")
    dev = _upload_tables(pkg, n, f, pkg.RULES[rule], tab["winners"], tab["sets"], tab["beta"], preagg)
    out = pkg.gar_coordinate_phase(G, dev, len(tab["winners"]), preagg).cpu().numpy()
    assert_outputs_match(out, want, G=Gh, tables=tab)


@pytest.mark.parametrize("d", [30_011, 412_347])        # register kernel; kernel staged by bulk copies (+ tail)
def test_coordinate_phase_general_schedule(pkg, d):
    # sets that are NOT nested (a later round holds a row the earlier one lacks):
    # the summation plan must restart or reuse a saved sum
    n, f = 15, 3
    G, Gh, _ = draw(pkg, 5, d)
    winners = [4, 9, 1, 12, 6, 0, 7]
    sets = [[0, 1, 4, 6, 7, 9, 12, 13], [0, 1, 6, 9, 12, 13, 14], [1, 6, 7, 12, 13, 14],
            [0, 6, 12, 13, 14], [6, 7, 13, 14], [0, 7, 13], [7, 13]]
    beta = 3
    ext, agr = O.extracted_and_aggregated(Gh, winners, sets)
    want, _, gap = O.closest_to_median_average(ext, agr, beta)
    dev = _upload_tables(pkg, n, f, 5, winners, sets, beta, 1)
    plan = pkg.read_selection(dev)
    assert plan.nu == 9 and any(plan.slot_src[s] != 254 for s in range(1, 7))   # some slot cannot just continue
    out = pkg.gar_coordinate_phase(G, dev, len(winners), 1).cpu().numpy()
    assert_outputs_match(out, want, G=Gh, tables=dict(winners=winners, sets=sets, beta=beta, gap=gap))


@pytest.mark.parametrize("theta", list(range(1, 33)) + [35, 40, 47, 52, 59, 63, 64])
def test_median_rule_every_slot_count(pkg, theta):
    # the Median rule exercises the median network at every row count (odd and even)
    d = 3001
    G = pkg.workloads.make_uniform(theta, d, device=DEV, seed=100 + theta)
    out = pkg.gar_aggregate("median", G, 0).cpu().numpy()
    want = O.coordinate_median(G.cpu().numpy())
    np.testing.assert_array_equal(out.astype(np.float64), want)


# ------------------------------------------------------------ rules end to end
@pytest.mark.parametrize("rule", ["average", "median", "krum", "multi_krum", "bulyan", "multi_bulyan"])
@pytest.mark.parametrize("cfg,n,f", CONFIGS)
@pytest.mark.parametrize("d", [4099, 65_540, 1_048_584])
def test_rules_end_to_end(pkg, rule, cfg, n, f, d):
    if d > 1_000_000 and rule in ("average", "median", "krum"):
        pytest.skip("covered at the small size")
    G, Gh, byz = draw(pkg, cfg, d)
    sel_dev = pkg.new_selection(DEV)
    dist = torch.empty(n, n, dtype=torch.float64, device=DEV)
    out = pkg.gar_aggregate_ex(rule, G, f, dist_out=dist, selection_out=sel_dev).cpu().numpy()
    want, tab = rule_tables(rule, Gh, f)
    if tab is None:
        assert_outputs_match(out, want)
        return
    sel = pkg.read_selection(sel_dev)
    preagg = rule in ("multi_krum", "multi_bulyan")
    compared = assert_selection_match(sel, tab["rounds"], preagg)
    # how much of the selection was really compared: all rounds at the two small sizes (their
    # score gaps are far above 1e-6), at least the first one at the large size, where the honest
    # scores of the later rounds come within 1e-6 of each other
    print(f"{rule} workload {cfg} d={d}: {compared} of {len(tab['rounds'])} rounds compared exactly")
    assert compared >= (len(tab["rounds"]) if d <= 65_540 else 1)
    if compared == len(tab["rounds"]):
        assert_outputs_match(out, want, G=Gh, tables=tab)
    else:
        # a score gap below 1e-6 relative: compare against the oracle's coordinate
        # phase run on the selection the GPU made (any order is a correct result)
        winners = [sel.winners[r] for r in range(sel.theta)]
        sets = [[i for i in range(n) if (sel.sets[r] >> i) & 1] for r in range(sel.theta)] if preagg else None
        want2, gap2 = O.coordinate_phase(Gh, winners, sets, sel.beta)
        assert_outputs_match(out, want2, G=Gh, tables=dict(winners=winners, sets=sets, beta=sel.beta, gap=gap2))
    if rule in ("multi_bulyan", "multi_krum") and cfg in (1, 3, 5):
        # far-away Byzantine rows are never averaged (the small-perturbation rows of
        # workloads 2 and 4 are built to blend in and may be)
        for r in range(sel.theta):
            assert not any((sel.sets[r] >> b) & 1 for b in byz), "a Byzantine row was averaged"


def test_gar_aggregate_plain_call_and_determinism(pkg):
    G, Gh, _ = draw(pkg, 2, 200_003)
    a = pkg.gar_aggregate("multi_bulyan", G, 5).clone()
    b = pkg.gar_aggregate("multi_bulyan", G, 5).clone()
    assert torch.equal(a, b)
    want, tab = rule_tables("multi_bulyan", Gh, 5)
    assert_outputs_match(a.cpu().numpy(), want, G=Gh, tables=tab)


def test_options_m_theta_median_of_agr(pkg):
    G, Gh, _ = draw(pkg, 5, 50_001)
    n, f = 15, 3
    out = pkg.gar_aggregate_ex("multi_krum", G, f, m=4).cpu().numpy()
    want, _ = rule_tables("multi_krum", Gh, f, m=4)
    assert_outputs_match(out, want)
    out = pkg.gar_aggregate_ex("multi_bulyan", G, f, median_of_agr=1).cpu().numpy()
    want, tab = rule_tables("multi_bulyan", Gh, f, median_of_agr=True)
    assert_outputs_match(out, want, G=Gh, tables=tab, median_source="agr")
    G2, G2h, _ = draw(pkg, 1, 20_001, n=20, f=3)
    out = pkg.gar_aggregate_ex("multi_bulyan", G2, 3, theta=9).cpu().numpy()
    want, tab = rule_tables("multi_bulyan", G2h, 3, theta=9)
    assert_outputs_match(out, want, G=G2h, tables=tab)


def test_strided_rows_and_caller_workspace(pkg):
    n, f, d = 23, 5, 33_333
    big, _ = pkg.workloads.make_gradients(2, d=d + 11, device=DEV)
    ws = torch.zeros(pkg.gar_workspace_bytes("multi_bulyan", n, f, d), dtype=torch.uint8, device=DEV)
    for view in (big[:, :d], big[:, 1:d + 1], big[:, 2:d + 2], big[:, 4:d + 4]):
        out = pkg.gar_aggregate_ex("multi_bulyan", view, f, workspace=ws).cpu().numpy()
        vh = view.cpu().numpy()
        want, tab = rule_tables("multi_bulyan", vh, f)
        assert_outputs_match(out, want, G=vh, tables=tab)


def test_staged_kernels_strided_rows_and_options(pkg):
    # sizes at which the kernels that stage tiles through shared memory by bulk copies run
    # (16-byte aligned rows, several tiles per SM), with a row stride larger than d, a ragged
    # tail, and the multi-Bulyan options; the unaligned view takes the register kernels
    n, f, d = 15, 3, 450_003
    big, _ = pkg.workloads.make_gradients(5, d=d + 9, device=DEV)      # row stride 450,012: a multiple of 4
    for view in (big[:, :d], big[:, 4:d + 4], big[:, 1:d + 1]):
        vh = view.cpu().numpy()
        for kw in (dict(), dict(median_of_agr=1), dict(theta=7)):
            out = pkg.gar_aggregate_ex("multi_bulyan", view, f, **kw).cpu().numpy()
            want, tab = rule_tables("multi_bulyan", vh, f, theta=kw.get("theta"), median_of_agr=bool(kw.get("median_of_agr")))
            assert_outputs_match(out, want, G=vh, tables=tab, median_source="agr" if kw.get("median_of_agr") else "ext")
        D = pkg.gar_pairwise_distances(view).cpu().numpy()
        Dh = O.pairwise_sq_distances(vh)
        assert np.max(np.abs(D - Dh) / np.maximum(Dh, 1e-300)) <= 1e-6
        assert np.array_equal(D, D.T) and np.all(np.diag(D) == 0.0)


def test_equal_honest_rows_give_that_row(pkg):
    n, f, d = 15, 3, 9001
    v = torch.randn(d, device=DEV)
    G = v.repeat(n, 1).contiguous()
    G[[2, 8, 13]] = torch.randn(3, d, device=DEV) * 1e3
    assert torch.equal(pkg.gar_aggregate("krum", G, f), v)
    for rule in ("bulyan", "multi_krum", "multi_bulyan"):      # fp32 mean of equal values: a rounding or two
        out = pkg.gar_aggregate(rule, G, f)
        assert torch.all((out - v).abs() <= 4e-7 * v.abs())


def test_host_entry_point(pkg):
    n, f, d = 11, 2, 123_457
    G, Gh, _ = draw(pkg, 1, d)
    host = G.cpu().pin_memory()
    out = pkg.gar_aggregate_host("multi_bulyan", host, f)
    dev = pkg.gar_aggregate("multi_bulyan", G, f).cpu()
    assert torch.equal(out, dev)


# --------------------------------------------------- the paper's own timing inputs (Section 5.1)
@pytest.mark.parametrize("n", list(range(7, 40, 4)) + [39])
@pytest.mark.parametrize("rule", ["multi_bulyan", "multi_krum", "median"])
def test_paper_grid_input_family(pkg, n, rule):
    """n gradients i.i.d. U(0,1)^d with f = floor((n-3)/4): the inputs of the paper's timing grid."""
    f = (n - 3) // 4
    d = 100_000
    G = pkg.workloads.make_uniform(n, d, device=DEV, seed=1905 + n)
    Gh = G.cpu().numpy()
    sel_dev = pkg.new_selection(DEV)
    out = pkg.gar_aggregate_ex(rule, G, f, selection_out=sel_dev).cpu().numpy()
    want, tab = rule_tables(rule, Gh, f)
    if tab is None:
        assert_outputs_match(out, want)
        return
    sel = pkg.read_selection(sel_dev)
    compared = assert_selection_match(sel, tab["rounds"], True)
    if compared == len(tab["rounds"]):
        assert_outputs_match(out, want, G=Gh, tables=tab)
    else:
        winners = [sel.winners[r] for r in range(sel.theta)]
        sets = [[i for i in range(n) if (sel.sets[r] >> i) & 1] for r in range(sel.theta)]
        want2, gap2 = O.coordinate_phase(Gh, winners, sets, sel.beta)
        assert_outputs_match(out, want2, G=Gh, tables=dict(winners=winners, sets=sets, beta=sel.beta, gap=gap2))


@pytest.mark.parametrize("cfg,n,f", [(5, 15, 3), (2, 23, 5), (4, 51, 12)])
def test_multi_krum_every_kind_of_m(pkg, cfg, n, f):
    """Section 3: Theorem 1 holds for any m <= n-f-2; m = 1 is Krum."""
    d = 50_001
    G, Gh, _ = draw(pkg, cfg, d)
    D = O.pairwise_sq_distances(Gh)
    for m in sorted({1, 2, (n - f - 2) // 2, n - f - 3, n - f - 2}):
        sel_dev = pkg.new_selection(DEV)
        out = pkg.gar_aggregate_ex("multi_krum", G, f, m=m, selection_out=sel_dev).cpu().numpy()
        want, tab = rule_tables("multi_krum", Gh, f, D=D, m=m)
        sel = pkg.read_selection(sel_dev)
        rnd = tab["rounds"][0]
        assert sel.m[0] == m and sel.winners[0] == rnd.winner
        if rnd.gap_set > 1e-6:
            assert sel.sets[0] == sum(1 << i for i in rnd.selected)
            assert_outputs_match(out, want)
    krum = pkg.gar_aggregate("krum", G, f).cpu().numpy()
    one = pkg.gar_aggregate_ex("multi_krum", G, f, m=1).cpu().numpy()
    assert np.array_equal(krum, one)
