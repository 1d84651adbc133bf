"""Parity at the benchmark's full size (workload 3: n=39, f=9, d=25.6e6) in the
launch configuration bench.py times.  The oracle cannot redo 4 GB in seconds, so
each stage is checked where it can be: sampled pairs of the distance matrix over
the full d, the selection exactly from the GPU's matrix, the coordinate phase on
sampled column blocks (start, tile boundaries, ragged end)."""
import numpy as np
import pytest
import torch

from oracle import gar_oracle as O
from tests._compare import assert_outputs_match

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def pkg():
    import __graft_entry__ as entry
    entry.build()
    import paper_1905_04374_b200 as p
    return p


@pytest.mark.parametrize("rule", ["multi_bulyan", "bulyan"])
def test_workload3_full_size(pkg, rule):
    wl = pkg.workloads.WORKLOADS[3]
    n, f, d = wl.n, wl.f, wl.d
    G, byz = pkg.workloads.make_gradients(3, device=DEV)
    dist = torch.empty(n, n, dtype=torch.float64, device=DEV)
    sel_dev = pkg.new_selection(DEV)
    out = pkg.gar_aggregate_ex(rule, G, f, dist_out=dist, selection_out=sel_dev)
    torch.cuda.synchronize()
    D = dist.cpu().numpy()
    # (1) sampled pairs over the full dimension: honest-honest, honest-Byzantine, Byzantine-Byzantine
    honest = [i for i in range(n) if i not in byz]
    pairs = [(honest[0], honest[1]), (honest[2], honest[-1]), (honest[3], byz[0]), (byz[0], byz[1]), (0, n - 1)]
    for i, j in pairs:
        gi, gj = G[i].cpu().numpy(), G[j].cpu().numpy()
        want = O.pairwise_sq_distances(np.stack([gi, gj]))[0, 1]
        assert abs(D[i, j] - want) <= 1e-6 * want, (i, j, D[i, j], want)
        assert D[i, j] == D[j, i]
    # (2) the selection, exactly, from the same matrix
    sel = pkg.read_selection(sel_dev)
    if rule == "multi_bulyan":
        osel = O.select_rounds(D, n, f, O.theta_of(rule, n, f))
        sets = osel.sets
    else:
        osel = O.select_rounds(D, n, f, O.theta_of(rule, n, f), clamp=True)
        sets = None
    assert [sel.winners[r] for r in range(sel.theta)] == osel.winners
    if sets is not None:
        for r, S in enumerate(sets):
            assert sel.sets[r] == sum(1 << i for i in S)
            assert not (set(S) & set(byz))
    # (3) the coordinate phase on sampled column blocks
    blocks = [(0, 4096), (65_536 - 100, 65_536 + 100), (d // 2 - 1000, d // 2 + 1000), (d - 5000, d)]
    for c0, c1 in blocks:
        Gb = G[:, c0:c1].cpu().numpy()
        want, gap = O.coordinate_phase(Gb, osel.winners, sets, osel.beta)
        got = out[c0:c1].cpu().numpy()
        assert_outputs_match(got, want, G=Gb, tables=dict(winners=osel.winners, sets=sets, beta=osel.beta, gap=gap))
    # (4) properties that hold at any size: the output is finite and inside the honest range
    assert bool(torch.isfinite(out).all())
    Gh = G[honest]
    assert bool((out <= Gh.max(dim=0).values).all()) and bool((out >= Gh.min(dim=0).values).all())
