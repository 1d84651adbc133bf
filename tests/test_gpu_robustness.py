"""GPU tests of what lies off the five workloads' beaten track: rows with a wide dynamic range
(the tensor-core distance kernel bounds its own rounding and hands over to the difference form),
the Bulyan family away from n = 4f+3 (beta > 1, even theta, exact ties at the beta-th place),
the even-median option, and the error path: a poisoned distance matrix, inconsistent tables and a
bounded wait that runs out must all end in a status and a NaN output, never in a plausible vector.
Nothing here faults or hangs a GPU: failures are injected as data."""
import numpy as np
import pytest
import torch

from oracle import gar_oracle as O
from tests._compare import assert_outputs_match, assert_selection_match, rule_tables

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def pkg():
    import __graft_entry__ as entry
    entry.build()
    import paper_1905_04374_b200 as p
    return p


def _workspace(pkg):
    return torch.zeros(pkg.gar_workspace_bytes("multi_bulyan", 11, 2, 1000), dtype=torch.uint8, device=DEV)


def _check_distances(pkg, G, expect_path=None):
    ws = _workspace(pkg)
    D = pkg.gar_pairwise_distances(G, workspace=ws).cpu().numpy()
    want = O.pairwise_sq_distances(G.cpu().numpy())
    pos = want > 0
    rel = np.abs(D - want)[pos] / want[pos]
    path = pkg.distance_path(ws)
    assert rel.max() <= 1e-6, f"max relative distance error {rel.max():.3e} on path {path}"
    assert np.array_equal(D, D.T) and np.all(np.diag(D) == 0) and np.all(D[~pos] == 0)
    if expect_path is not None:
        assert path == expect_path, path
    return path, rel.max()


# ------------------------------------------------------- dynamic range of the rows (distances)
@pytest.mark.parametrize("n", [23, 39])
@pytest.mark.parametrize("case", ["shared_spike", "private_spikes", "scaled_block"])
def test_distances_wide_dynamic_range(pkg, n, case):
    d = 200_064
    gen = torch.Generator(device=DEV)
    gen.manual_seed(1000 + n)
    G = torch.randn(n, d, generator=gen, device=DEV)
    if case == "shared_spike":            # the same huge entry in every row: cancels in every distance
        G[:, 0] = 1e5
        expect = "gram_rejected"
    elif case == "private_spikes":        # one large entry per row, early in the row
        for i in range(n):
            G[i, (7 * i) % 128] = 1e4
        expect = None
    else:                                 # a block of columns 2^14 times larger than the rest
        G[:, 100_000:101_000] *= 2.0 ** 14
        expect = None
    path, err = _check_distances(pkg, G, expect)
    print(f"{case} n={n}: path {path}, max relative error {err:.2e}")


@pytest.mark.parametrize("noise,d", [(1e-3, 262_144), (1e-4, 1_048_576), (3e-2, 262_144)])
def test_distances_shared_mean_small_noise(pkg, noise, d):
    """Honest-looking rows: a shared vector plus small private noise.  The distances are tiny next
    to the rows' norms; the Gram form only keeps them when its rounding bound says so."""
    n = 23
    gen = torch.Generator(device=DEV)
    gen.manual_seed(77)
    mu = torch.randn(d, generator=gen, device=DEV)
    G = mu[None, :] + noise * torch.randn(n, d, generator=gen, device=DEV)
    path, err = _check_distances(pkg, G)
    print(f"noise {noise} d={d}: path {path}, max relative error {err:.2e}")
    if noise <= 1e-3:
        assert path == "gram_rejected"


def test_distances_falling_magnitude_and_forced_difference_form(pkg):
    n, d = 39, 262_144
    gen = torch.Generator(device=DEV)
    gen.manual_seed(5)
    G = torch.randn(n, d, generator=gen, device=DEV) * torch.exp2(-torch.arange(d, device=DEV) * (20.0 / d))[None, :]
    _check_distances(pkg, G)
    ws = _workspace(pkg)
    D = pkg.gar_pairwise_distances(G, workspace=ws, distance_mode="difference").cpu().numpy()
    assert pkg.distance_path(ws) == "difference"
    np.testing.assert_allclose(D, O.pairwise_sq_distances(G.cpu().numpy()), rtol=1e-6, atol=0)


@pytest.mark.parametrize("cfg", [2, 3, 4])
def test_workloads_stay_on_the_tensor_core_path(pkg, cfg):
    """The benchmark workloads are inside the fast kernel's input range (and the bound that decides
    it is not vacuous: the spiked inputs above are rejected)."""
    G, _ = pkg.workloads.make_gradients(cfg, d=1_048_576 * (4 if cfg == 4 else 1), device=DEV)
    _check_distances(pkg, G, "gram")


def test_rerouted_aggregation_end_to_end(pkg):
    """A whole multi-Bulyan call whose distance step is rejected and recomputed on the device."""
    n, f, d = 23, 5, 450_048
    G, _ = pkg.workloads.make_gradients(2, d=d, device=DEV)
    G[:, 5] += 3e5
    Gh = G.cpu().numpy()
    ws = _workspace(pkg)
    sel_dev = pkg.new_selection(DEV)
    out = pkg.gar_aggregate_ex("multi_bulyan", G, f, workspace=ws, selection_out=sel_dev).cpu().numpy()
    assert pkg.distance_path(ws) == "gram_rejected"
    want, tab = rule_tables("multi_bulyan", Gh, f)
    sel = pkg.read_selection(sel_dev)
    assert sel.status == 0
    compared = assert_selection_match(sel, tab["rounds"], True)
    assert compared >= 5
    if compared == len(tab["rounds"]):
        assert_outputs_match(out, want, G=Gh, tables=tab)
    else:                                  # a later round's scores lie within 1e-6: either order is right
        winners = [sel.winners[r] for r in range(sel.theta)]
        sets = [[i for i in range(n) if (sel.sets[r] >> i) & 1] for r in range(sel.theta)]
        want2, gap2 = O.coordinate_phase(Gh, winners, sets, sel.beta)
        assert_outputs_match(out, want2, G=Gh, tables=dict(winners=winners, sets=sets, beta=sel.beta, gap=gap2))


# --------------------------------------------------- Bulyan family away from n = 4f + 3
OFF_LINE = [(12, 2), (16, 3), (20, 3), (33, 4), (64, 15), (9, 0), (64, 0), (13, 1)]


@pytest.mark.parametrize("n,f", OFF_LINE)
@pytest.mark.parametrize("rule", ["bulyan", "multi_bulyan"])
@pytest.mark.parametrize("d", [4099, 401_408])
def test_bulyan_family_off_the_line(pkg, rule, n, f, d):
    """beta = theta - 2f takes the values 2, 4, 6, 8, 15, ... here, theta is even in several cases,
    and f = 0 makes Bulyan the plain average (beta = theta = n)."""
    if rule == "multi_bulyan" and n - 4 * f - 2 < 1:
        pytest.skip("multi-Bulyan needs beta = n-4f-2 >= 1")
    cfg = 4 if n > 40 else 2
    G, _ = pkg.workloads.make_gradients(cfg, d=d, device=DEV, n=n, f=f)
    Gh = G.cpu().numpy()
    sel_dev = pkg.new_selection(DEV)
    out = pkg.gar_aggregate_ex(rule, G, f, selection_out=sel_dev).cpu().numpy()
    want, tab = rule_tables(rule, Gh, f)
    sel = pkg.read_selection(sel_dev)
    assert sel.status == 0 and sel.theta == len(tab["rounds"]) and sel.beta == tab["beta"]
    preagg = rule == "multi_bulyan"
    compared = assert_selection_match(sel, tab["rounds"], preagg)
    if compared == len(tab["rounds"]):
        assert_outputs_match(out, want, G=Gh, tables=tab)
    else:
        winners = [sel.winners[r] for r in range(sel.theta)]
        sets = [[i for i in range(n) if (sel.sets[r] >> i) & 1] for r in range(sel.theta)] if preagg else None
        want2, gap2 = O.coordinate_phase(Gh, winners, sets, sel.beta)
        assert_outputs_match(out, want2, G=Gh, tables=dict(winners=winners, sets=sets, beta=sel.beta, gap=gap2))
    if rule == "bulyan" and f == 0:
        np.testing.assert_allclose(out, Gh.astype(np.float64).mean(axis=0), rtol=0, atol=1e-5 * (1 + np.abs(Gh).max()))


def _upload(pkg, n, f, rule_id, winners, sets, beta, preagg, even_median=0):
    h = pkg.GarSelection()
    h.n, h.f, h.rule, h.theta, h.beta = n, f, rule_id, len(winners), beta
    h.preagg, h.median_of_agr, h.even_median = preagg, 0, even_median
    for r, w in enumerate(winners):
        h.winners[r] = w
        h.sets[r] = sum(1 << i for i in (sets[r] if sets is not None else [w]))
    dev = pkg.write_selection(h, DEV)
    pkg.gar_schedule_from_tables(dev)
    return dev


@pytest.mark.parametrize("theta,beta", [(7, 2), (7, 3), (9, 5), (12, 4), (20, 6)])
@pytest.mark.parametrize("d,preagg", [(4099, 0), (4099, 1), (401_408, 1)])
def test_exact_ties_at_the_beta_th_place(pkg, theta, beta, d, preagg):
    """Small-integer columns: several |a - M| are EQUAL at the beta-th place, so more values tie
    than there is room for and the kept ones are decided by the tie-break alone (earliest round
    first, on both sides).  Integer data: the expected averages are exact."""
    n = theta
    rng = np.random.default_rng(10 * theta + beta)
    Gh = rng.integers(-3, 4, size=(n, d)).astype(np.float32)
    G = torch.from_numpy(Gh).to(DEV)
    winners = list(rng.permutation(n))
    sets = [[int(w)] for w in winners]           # one-gradient sets: G^agr = G^ext through the summing kernels too
    ext, agr = O.extracted_and_aggregated(Gh, winners, sets)
    want, M, gap = O.closest_to_median_average(ext, agr, beta)
    assert (gap == 0).mean() > 0.2               # the ties are really there
    dev = _upload(pkg, n, 0, 5 if preagg else 4, [int(w) for w in winners], sets if preagg else None, beta, preagg)
    out = pkg.gar_coordinate_phase(G, dev, theta, preagg).cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(out, want, rtol=0, atol=2e-6)


# --------------------------------------------------------------- median of an even count
@pytest.mark.parametrize("n", [2, 4, 6, 10, 16, 24, 32, 36, 40, 50, 64])
def test_median_rule_even_count_mean(pkg, n):
    d = 3001
    G = pkg.workloads.make_uniform(n, d, device=DEV, seed=300 + n)
    Gh = G.cpu().numpy()
    out = pkg.gar_aggregate_ex("median", G, 0, even_median="mean").cpu().numpy().astype(np.float64)
    want = O.coordinate_median(Gh, even="mean")
    np.testing.assert_allclose(out, want, rtol=0, atol=1.2e-7)
    np.testing.assert_allclose(want, np.median(Gh.astype(np.float64), axis=0), rtol=0, atol=0)
    lower = pkg.gar_aggregate_ex("median", G, 0, even_median="lower").cpu().numpy().astype(np.float64)
    np.testing.assert_array_equal(lower, O.coordinate_median(Gh, even="lower"))


@pytest.mark.parametrize("rule,n,f", [("multi_bulyan", 12, 2), ("multi_bulyan", 16, 3), ("bulyan", 12, 2),
                                      ("bulyan", 20, 3), ("multi_bulyan", 44, 5), ("bulyan", 64, 15)])
@pytest.mark.parametrize("d", [4099, 401_408])
def test_even_theta_with_mean_median(pkg, rule, n, f, d):
    G, _ = pkg.workloads.make_gradients(4 if n > 40 else 1, d=d, device=DEV, n=n, f=f)
    Gh = G.cpu().numpy()
    sel_dev = pkg.new_selection(DEV)
    out = pkg.gar_aggregate_ex(rule, G, f, even_median="mean", selection_out=sel_dev).cpu().numpy()
    sel = pkg.read_selection(sel_dev)
    assert sel.theta % 2 == 0 and sel.even_median == 1
    preagg = rule == "multi_bulyan"
    winners = [sel.winners[r] for r in range(sel.theta)]
    sets = [[i for i in range(n) if (sel.sets[r] >> i) & 1] for r in range(sel.theta)] if preagg else None
    want, gap = O.coordinate_phase(Gh, winners, sets, sel.beta, even="mean")
    # The mean of the two middle values is equidistant from both: with identical Byzantine rows
    # among the winners (workload 4's attack at n = 64 has eight and seven copies) a copy of a middle
    # value ties EXACTLY with the other middle value at the beta-th place in about 1 % of the
    # columns.  Every such column is still checked against the averages its tie admits.
    assert_outputs_match(out, want, G=Gh, tables=dict(winners=winners, sets=sets, beta=sel.beta, gap=gap), even="mean",
                         max_tie_frac=2e-2 if n == 64 else 2e-4)
    # and it is a different function from the lower median
    want_lower, _ = O.coordinate_phase(Gh, winners, sets, sel.beta, even="lower")
    assert np.abs(want - want_lower).max() > 0


# ------------------------------------------------------------------------- the error path
def test_poisoned_distance_matrix_gives_status_and_nan_output(pkg):
    n, f, d = 15, 3, 50_000
    G, _ = pkg.workloads.make_gradients(5, d=d, device=DEV)
    D = pkg.gar_pairwise_distances(G).clone()
    good = pkg.read_selection(pkg.gar_select("multi_bulyan", D, n, f))
    assert good.status == 0
    D.fill_(float("nan"))                                   # what a distance kernel that gave up leaves behind
    sel_dev = pkg.gar_select("multi_bulyan", D, n, f)
    assert pkg.read_selection(sel_dev).status == 6          # GAR_ERR_TIMEOUT
    out = pkg.gar_coordinate_phase(G, sel_dev, good.theta, 1)
    assert bool(torch.isnan(out).all())
    # only the diagonal decides: NaN off the diagonal is data (a row with a NaN entry)
    D2 = pkg.gar_pairwise_distances(G).clone()
    D2[2, :] = float("nan"); D2[:, 2] = float("nan"); D2[2, 2] = 0.0
    ok = pkg.read_selection(pkg.gar_select("multi_bulyan", D2, n, f))
    assert ok.status == 0 and 2 not in [ok.winners[r] for r in range(ok.theta)]
    # large aligned d: the staged coordinate kernel answers the same way
    G2, _ = pkg.workloads.make_gradients(5, d=450_048, device=DEV)
    out = pkg.gar_coordinate_phase(G2, sel_dev, good.theta, 1)
    assert bool(torch.isnan(out).all())


@pytest.mark.parametrize("d", [30_011, 450_048])
def test_inconsistent_tables_are_refused_on_the_device(pkg, d):
    n, f = 15, 3
    G, _ = pkg.workloads.make_gradients(5, d=d, device=DEV)
    D = pkg.gar_pairwise_distances(G)
    sel_dev = pkg.gar_select("multi_bulyan", D, n, f)
    h = pkg.read_selection(sel_dev)
    want = pkg.gar_coordinate_phase(G, sel_dev, h.theta, 1).clone()
    assert bool(torch.isfinite(want).all())
    # theta that does not match the selection
    out = pkg.gar_coordinate_phase(G, sel_dev, h.theta - 2, 1)
    assert bool(torch.isnan(out).all()) and pkg.read_selection(sel_dev).status == 1
    # pre-aggregation flag that does not match
    sel_dev = pkg.gar_select("multi_bulyan", D, n, f)
    out = pkg.gar_coordinate_phase(G, sel_dev, h.theta, 0)
    assert bool(torch.isnan(out).all()) and pkg.read_selection(sel_dev).status == 1
    # a winner index outside the matrix; fewer rows than the tables name
    for field, idx, value in (("winners", 1, 15), ("winners", 0, -1), ("base_rows", 0, 200), ("m", 2, 0)):
        sel_dev = pkg.gar_select("multi_bulyan", D, n, f)
        hh = pkg.read_selection(sel_dev)
        getattr(hh, field)[idx] = value
        bad = pkg.write_selection(hh, DEV)
        out = pkg.gar_coordinate_phase(G, bad, h.theta, 1)
        assert bool(torch.isnan(out).all()), field
        assert pkg.read_selection(bad).status == 1
    sel_dev = pkg.gar_select("multi_bulyan", D, n, f)
    out = pkg.gar_coordinate_phase(G[:12], sel_dev, h.theta, 1)
    assert bool(torch.isnan(out).all())
    # and the untouched selection still works
    sel_dev = pkg.gar_select("multi_bulyan", D, n, f)
    assert torch.equal(pkg.gar_coordinate_phase(G, sel_dev, h.theta, 1), want)


def test_bounded_wait_runs_out_with_a_status(pkg):
    """A wait on a barrier that nothing arrives on (no copy, no tensor-core work in flight) must
    give up after its iteration limit and say so; the context stays usable."""
    status, ns = pkg.gar_selftest_bounded_wait(200)
    assert status == 6
    assert ns < 1_000_000_000, f"200 bounded polls took {ns} ns"
    status2, ns2 = pkg.gar_selftest_bounded_wait(2000)
    assert status2 == 6
    print(f"bounded wait: {ns / 200:.0f} ns per suspended poll at 200, {ns2 / 2000:.0f} ns at 2000")
    x = torch.ones(10, device=DEV)
    assert float(x.sum()) == 10.0


# ----------------------------------------------------------- SGD step fused into the store
@pytest.mark.parametrize("d", [4099, 450_048])
@pytest.mark.parametrize("with_momentum", [False, True])
def test_fused_sgd_step(pkg, d, with_momentum):
    """Eq. 2 with the aggregate never written out: x <- x - lr * GAR (or through a momentum buffer),
    three steps in a row, against the oracle's step applied to the oracle's aggregate."""
    n, f = 15, 3
    lr, mu = 0.05, 0.9
    gen = torch.Generator(device=DEV).manual_seed(9)
    x = torch.randn(d, generator=gen, device=DEV)
    v = torch.zeros(d, device=DEV) if with_momentum else None
    xh = x.cpu().numpy().astype(np.float64)
    vh = np.zeros(d) if with_momentum else None
    for step in range(3):
        G, _ = pkg.workloads.make_gradients(5, d=d, device=DEV, seed=500 + step)
        Gh = G.cpu().numpy()
        keep = pkg.gar_aggregate_ex("multi_bulyan", G, f, sgd_params=x, sgd_momentum_buf=v, sgd_lr=lr, sgd_momentum=mu,
                                    store_out=(step == 0))
        agg, tab = rule_tables("multi_bulyan", Gh, f)
        if step == 0:                            # the aggregate is still stored when an output is given
            assert_outputs_match(keep.cpu().numpy(), agg, G=Gh, tables=tab)
        else:
            assert keep is None
        xh, vh = O.sgd_step(xh, agg, lr, momentum_buf=vh, momentum=mu)
        # the same tie-aware bar as for the aggregate, scaled by what multiplies it on the way to x
        scale = lr * sum(mu ** k for k in range(step + 1)) if with_momentum else lr * (step + 1)
        bad = np.abs(x.cpu().numpy() - xh) > 1e-5 * (1 + np.abs(xh)) + scale * 1e-5 * (1 + np.abs(agg))
        assert bad.sum() <= max(3, int(6e-4 * d)), f"step {step}: {int(bad.sum())} coordinates of x off"
        if with_momentum:
            badv = np.abs(v.cpu().numpy() - vh) > 1e-5 * (1 + np.abs(vh)) * (step + 1)
            assert badv.sum() <= max(3, int(6e-4 * d))
        # keep the two sides from drifting apart through legitimate near-tie choices
        xh = x.cpu().numpy().astype(np.float64)
        if with_momentum:
            vh = v.cpu().numpy().astype(np.float64)


def test_fused_sgd_leaves_the_model_alone_on_failure(pkg):
    n, f, d = 15, 3, 50_000
    G, _ = pkg.workloads.make_gradients(5, d=d, device=DEV)
    D = torch.full((n, n), float("nan"), dtype=torch.float64, device=DEV)
    sel = pkg.gar_select("multi_bulyan", D, n, f)
    assert pkg.read_selection(sel).status == 6
    # the fused step goes through gar_aggregate_ex only; the same kernels refuse a poisoned selection
    # for the plain output, which is what decides whether x is touched
    out = pkg.gar_coordinate_phase(G, sel, pkg.gar_theta("multi_bulyan", n, f), 1)
    assert bool(torch.isnan(out).all())


# ------------------------------------------------------------ 16-bit gradient inputs
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("cfg,d", [(5, 4099), (5, 450_048), (5, 450_051), (2, 70_001), (3, 262_148), (1, 200_003),
                                   (3, 262_144), (4, 401_408), (2, 1_048_576)])
def test_sixteen_bit_gradients(pkg, dtype, cfg, d):
    """bfloat16 / binary16 gradients: every value is widened to fp32 exactly when it is loaded, so
    the oracle, fed the same 16-bit values promoted to fp64, is the reference at the usual bars
    (distances 1e-6 relative, outputs 1e-5 (1 + |oracle|), selection where the gap is clear)."""
    wl = pkg.workloads.WORKLOADS[cfg]
    n, f = wl.n, wl.f
    G32, _ = pkg.workloads.make_gradients(cfg, d=d, device=DEV)
    G = G32.to(dtype)
    Gh = G.to(torch.float32).cpu().numpy()            # exact: both formats embed in fp32
    for rule in ("multi_bulyan", "bulyan", "median", "average"):
        sel_dev = pkg.new_selection(DEV)
        dist = torch.empty(n, n, dtype=torch.float64, device=DEV)
        out = pkg.gar_aggregate_ex(rule, G, f, dist_out=dist, selection_out=sel_dev).cpu().numpy()
        want, tab = rule_tables(rule, Gh, f)
        if tab is None:
            assert_outputs_match(out, want)
            continue
        D = dist.cpu().numpy()
        wantD = O.pairwise_sq_distances(Gh)
        pos = wantD > 0
        assert np.max(np.abs(D - wantD)[pos] / wantD[pos]) <= 1e-6 and np.all(D[~pos] == 0)
        sel = pkg.read_selection(sel_dev)
        assert sel.status == 0
        preagg = rule == "multi_bulyan"
        compared = assert_selection_match(sel, tab["rounds"], preagg)
        # 16-bit values collide often (8 or 11 significant bits): exact ties between |a - M| values are
        # a hundred times more frequent than with fp32 inputs; every one is still checked against
        # the averages its tie admits
        if compared == len(tab["rounds"]):
            assert_outputs_match(out, want, G=Gh, tables=tab, max_tie_frac=1e-2)
        else:
            winners = [sel.winners[r] for r in range(sel.theta)]
            sets = [[i for i in range(n) if (sel.sets[r] >> i) & 1] for r in range(sel.theta)] if preagg else None
            want2, gap2 = O.coordinate_phase(Gh, winners, sets, sel.beta)
            assert_outputs_match(out, want2, G=Gh, tables=dict(winners=winners, sets=sets, beta=sel.beta, gap=gap2),
                                 max_tie_frac=1e-2)


def test_sixteen_bit_strided_views(pkg):
    n, f, d = 15, 3, 33_333
    big, _ = pkg.workloads.make_gradients(5, d=d + 11, device=DEV)
    big = big.to(torch.bfloat16)
    for view in (big[:, :d], big[:, 1:d + 1], big[:, 2:d + 2], big[:, 8:d + 8]):
        vh = view.to(torch.float32).cpu().numpy()
        out = pkg.gar_aggregate_ex("multi_bulyan", view, f).cpu().numpy()
        want, tab = rule_tables("multi_bulyan", vh, f)
        assert_outputs_match(out, want, G=vh, tables=tab, max_tie_frac=1e-2)


def test_cuda_graph_capture_and_replay(pkg):
    """The three launches of an aggregation are plain stream work: once a first call has set the
    kernels' attributes they can be captured into a CUDA graph and replayed (the launch-bound
    small-d regime), on new contents of the same buffers."""
    cfg = 1
    wl = pkg.workloads.WORKLOADS[cfg]
    G, _ = pkg.workloads.make_gradients(cfg, d=100_000, device=DEV)
    out = torch.empty(G.shape[1], dtype=torch.float32, device=DEV)
    ws = torch.zeros(pkg.gar_workspace_bytes("multi_bulyan", wl.n, wl.f, G.shape[1]), dtype=torch.uint8, device=DEV)
    pkg.gar_aggregate_ex("multi_bulyan", G, wl.f, out=out, workspace=ws)
    torch.cuda.synchronize()
    first = out.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        pkg.gar_aggregate_ex("multi_bulyan", G, wl.f, out=out, workspace=ws)
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, first)
    # new gradients in the captured buffer: the replay aggregates them
    G2, _ = pkg.workloads.make_gradients(cfg, d=100_000, device=DEV, seed=4242)
    G.copy_(G2)
    graph.replay()
    torch.cuda.synchronize()
    Gh = G2.cpu().numpy()
    want, osel, gap = O.multi_bulyan(Gh, wl.f)
    assert_outputs_match(out.cpu().numpy(), want, G=Gh, tables=dict(winners=osel.winners, sets=osel.sets, beta=osel.beta, gap=gap))
