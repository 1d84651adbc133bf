"""Parity at the full size of the three large workloads (3: n=39, d=25.6e6; 4: n=51, d=1e8, 5.1e9
elements; 5: n=15, d=1e9, 1.5e10 elements) in the launch configuration bench.py times.  The oracle
cannot redo 4 to 60 GB in seconds, so each stage is checked where it can be: sampled pairs of the
distance matrix over the full d (two rows pulled to the host at a time), the selection exactly from
the GPU's matrix, the coordinate phase on sampled column blocks -- the start, tile boundaries, the
columns where the element offset row * ld + column crosses 2^31 and 2^32 (the 64-bit offset
arithmetic has nothing to hide behind there), and the ragged end -- and properties that hold at
any size."""
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


def _crossing_columns(n, ld, d, offset):
    """Column at which some row's element offset equals `offset` (None if no row reaches it)."""
    row = offset // ld
    col = offset - row * ld
    return int(col) if row < n and col < d else None


@pytest.mark.parametrize("cfg", [3, 4, 5])
def test_workload_full_size(pkg, cfg):
    wl = pkg.workloads.WORKLOADS[cfg]
    n, f, d = wl.n, wl.f, wl.d
    G, byz = pkg.workloads.make_gradients(cfg, device=DEV)
    honest = [i for i in range(n) if i not in byz]
    # (1) sampled pairs over the full dimension: honest-honest, honest-Byzantine, Byzantine-Byzantine
    pairs = [(honest[0], honest[1]), (honest[2], honest[-1]), (honest[3], byz[0])]
    if cfg != 5:
        pairs += [(byz[0], byz[1]), (0, n - 1)]
    want_pairs = {}
    for i, j in pairs:
        gi, gj = G[i].cpu().numpy(), G[j].cpu().numpy()
        want_pairs[(i, j)] = O.pairwise_sq_distances(np.stack([gi, gj]), block=1 << 22)[0, 1]
        del gi, gj
    for rule in ("multi_bulyan", "bulyan"):
        dist = torch.empty(n, n, dtype=torch.float64, device=DEV)
        sel_dev = pkg.new_selection(DEV)
        ws = torch.zeros(pkg.gar_workspace_bytes(rule, n, f, d), dtype=torch.uint8, device=DEV)
        out = pkg.gar_aggregate_ex(rule, G, f, dist_out=dist, selection_out=sel_dev, workspace=ws)
        torch.cuda.synchronize()
        D = dist.cpu().numpy()
        assert pkg.distance_path(ws) == ("gram" if n > 16 else "difference")
        for (i, j), want in want_pairs.items():
            assert abs(D[i, j] - want) <= 1e-6 * want, (i, j, D[i, j], want)
            assert D[i, j] == D[j, i]
        assert np.all(np.diag(D) == 0) and np.all(np.isfinite(D))
        # (2) the selection, exactly, from the same matrix
        sel = pkg.read_selection(sel_dev)
        assert sel.status == 0
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
                if cfg in (3, 5):               # far-away Byzantine rows are never averaged
                    assert not (set(S) & set(byz))
        # (3) the coordinate phase on sampled column blocks
        blocks = [(0, 4096), (65_536 - 100, 65_536 + 100), (d // 2 - 1000, d // 2 + 1000), (d - 5000, d)]
        for offset in (1 << 31, 1 << 32, 1 << 33):
            col = _crossing_columns(n, d, d, offset)
            if col is not None:
                blocks.append((max(col - 1500, 0), min(col + 1500, d)))
        for c0, c1 in blocks:
            Gb = G[:, c0:c1].cpu().numpy()
            want, gap = O.coordinate_phase(Gb, osel.winners, sets, osel.beta)
            got = out[c0:c1].cpu().numpy()
            assert_outputs_match(got, want, G=Gb, tables=dict(winners=osel.winners, sets=sets, beta=osel.beta, gap=gap))
        # (4) properties that hold at any size: the output is finite and inside the honest range
        assert bool(torch.isfinite(out).all())
        if cfg in (3, 5):
            step = 1 << 25
            for c0 in range(0, d, step):
                c1 = min(c0 + step, d)
                hi = G[honest[0], c0:c1].clone()
                lo = hi.clone()
                for i in honest[1:]:
                    hi = torch.maximum(hi, G[i, c0:c1])
                    lo = torch.minimum(lo, G[i, c0:c1])
                assert bool((out[c0:c1] <= hi).all()) and bool((out[c0:c1] >= lo).all())
        del out, dist
    del G
    torch.cuda.empty_cache()
