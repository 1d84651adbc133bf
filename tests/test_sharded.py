"""Aggregation sharded over the coordinates.

CPU part (gloo, world size 2, runs anywhere): the orchestration of
paper_1905_04374_b200.sharded -- local partial matrices, all-gather, sum in rank order,
replicated selection, local coordinate phase -- with the oracle's functions standing in for the
kernels: both ranks must end with the bit-identical matrix, the same winners, and slices that
concatenate to the single-process result.

GPU part (one GPU): the same path through the real kernels, the "ranks" being two column
slices processed one after the other (nothing waits on anything), against the single-device call
and the oracle; and gar_reduce_partials against a left-to-right sum."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from oracle import gar_oracle as O
from tests._compare import assert_outputs_match, rule_tables

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["GAR_ROOT"])
import numpy as np, torch, torch.distributed as dist
from oracle import gar_oracle as O
from paper_1905_04374_b200 import sharded, workloads

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
n, f, d = 11, 2, 5_000_003
rule = "multi_bulyan"

class Sel:                                     # what the stand-in selection hands to the coordinate stage
    def __init__(self, s): self.s = s

def distances(G):
    return torch.from_numpy(O.pairwise_sq_distances(G.numpy(), block=1 << 20))

def reduce(parts):                             # left to right, as gar_reduce_partials does
    acc = parts[0].clone()
    for r in range(1, parts.shape[0]):
        acc = acc + parts[r]
    return acc

def select(rule, D, n, f, **kw):
    return Sel(O.select_rounds(D.numpy(), n, f, O.theta_of(rule, n, f)))

def coordinate(G, sel, theta, preagg):
    out, _ = O.coordinate_phase(G.numpy(), sel.s.winners, sel.s.sets if preagg else None, sel.s.beta)
    return torch.from_numpy(out)

stages = sharded.Stages(distances=distances, reduce=reduce, select=select, coordinate=coordinate,
                        theta=lambda rule, n, f: O.theta_of(rule, n, f))
# integer-valued gradients: every partial sum is exact, so any order of adding the slices gives the
# same bits -- and the rank-order sum must reproduce the single-process matrix exactly
gen = torch.Generator().manual_seed(1234)
full = torch.randint(-8, 9, (n, d), generator=gen).to(torch.float32)
full[3] *= 50.0; full[7] = full[3]
c0, c1 = workloads.shard_columns(d, world, rank)
out, sel, D = sharded.sharded_aggregate(rule, full[:, c0:c1].contiguous(), f, stages=stages)
D_single = torch.from_numpy(O.pairwise_sq_distances(full.numpy(), block=1 << 20))
assert torch.equal(D, D_single), "rank-order sum of the slices' matrices differs from the single-process matrix"
# every rank holds the same matrix and makes the same selection
gathered = [torch.empty_like(D) for _ in range(world)]
dist.all_gather(gathered, D)
assert all(torch.equal(g, D) for g in gathered)
w = torch.tensor(sel.s.winners)
ws = [torch.empty_like(w) for _ in range(world)]
dist.all_gather(ws, w)
assert all(torch.equal(x, w) for x in ws)
# the slices concatenate to the single-process aggregate
want, _, _ = O.multi_bulyan(full.numpy(), f, D=D_single.numpy())
assert np.array_equal(out.numpy(), want[c0:c1])
# a rank without columns takes part in the exchange and returns an empty slice
out0, _, D0 = sharded.sharded_aggregate(rule, full[:, :0] if rank == 1 else full, f, stages=stages)
assert torch.equal(D0, D_single) and out0.numel() == (0 if rank == 1 else d)
dist.barrier()
sys.stdout.write("rank %d sharded ok\n" % rank); sys.stdout.flush()
dist.destroy_process_group()
"""


def test_sharded_orchestration_gloo_world2(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, GAR_ROOT=ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29741", str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, env=env, cwd=ROOT, timeout=900)
    assert res.returncode == 0, res.stdout + res.stderr
    assert res.stdout.count("sharded ok") == 2


def test_shard_columns_cover_the_dimension():
    from paper_1905_04374_b200 import workloads as W
    for d in (1, W.CHUNK, W.CHUNK + 1, 5 * W.CHUNK + 17, 1_000_000_000):
        for world in (1, 2, 3, 8):
            edges = [W.shard_columns(d, world, r) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == d
            assert all(a[1] == b[0] for a, b in zip(edges, edges[1:]))
            assert all(c0 % W.CHUNK == 0 or c0 == d for c0, _ in edges)


def test_sliced_draw_equals_the_full_draw():
    from paper_1905_04374_b200 import workloads as W
    d = 2 * W.CHUNK + 12_345
    G, byz = W.make_gradients(4, d=d, n=9, f=1)
    for world in (2, 3):
        parts = [W.make_gradients(4, d=d, n=9, f=1, columns=W.shard_columns(d, world, r))[0] for r in range(world)]
        assert torch.equal(torch.cat(parts, dim=1), G)


# ------------------------------------------------------------------ GPU: the real kernels
@pytest.fixture(scope="module")
def pkg():
    import __graft_entry__ as entry
    entry.build()
    import paper_1905_04374_b200 as p
    return p


@pytest.mark.gpu
def test_reduce_partials_is_a_left_to_right_sum(pkg):
    gen = torch.Generator(device="cuda:0").manual_seed(3)
    for count, n in ((1, 5), (2, 15), (8, 39), (5, 64)):
        parts = torch.randn(count, n, n, generator=gen, device="cuda:0", dtype=torch.float64) * 1e6
        want = parts[0].clone()
        for r in range(1, count):
            want = want + parts[r]
        assert torch.equal(pkg.gar_reduce_partials(parts), want)
    nan = torch.zeros(2, 4, 4, dtype=torch.float64, device="cuda:0")
    nan[1].fill_diagonal_(float("nan"))
    assert bool(torch.isnan(torch.diagonal(pkg.gar_reduce_partials(nan))).all())


@pytest.mark.gpu
@pytest.mark.parametrize("cfg,rule", [(5, "multi_bulyan"), (2, "multi_bulyan"), (3, "bulyan"), (1, "multi_krum")])
def test_sharded_path_on_one_gpu_matches_single_device_and_oracle(pkg, cfg, rule):
    from paper_1905_04374_b200 import workloads as W
    wl = W.WORKLOADS[cfg]
    n, f = wl.n, wl.f
    d = W.CHUNK + 450_048                      # two slices: one whole chunk and a ragged, staged-size rest
    G, _ = W.make_gradients(cfg, d=d, device="cuda:0")
    Gh = G.cpu().numpy()
    slices = [W.make_gradients(cfg, d=d, device="cuda:0", columns=W.shard_columns(d, 2, r))[0] for r in range(2)]
    assert torch.equal(torch.cat(slices, dim=1), G)
    parts = torch.stack([pkg.gar_pairwise_distances(S).clone() for S in slices])
    D = pkg.gar_reduce_partials(parts)
    want_D = O.pairwise_sq_distances(Gh)
    pos = want_D > 0
    assert np.max(np.abs(D.cpu().numpy() - want_D)[pos] / want_D[pos]) <= 1e-6
    sel = pkg.gar_select(rule, D, n, f)
    theta = pkg.gar_theta(rule, n, f)
    preagg = int(rule in ("multi_bulyan", "multi_krum"))
    out = torch.cat([pkg.gar_coordinate_phase(S, sel, theta, preagg) for S in slices]).cpu().numpy()
    # against the oracle's coordinate phase on the selection the sharded path made from its matrix
    h = pkg.read_selection(sel)
    winners = [h.winners[r] for r in range(h.theta)]
    sets = [[i for i in range(n) if (h.sets[r] >> i) & 1] for r in range(h.theta)] if preagg else None
    osel = O.select_rounds(D.cpu().numpy(), n, f, theta, clamp=(rule == "bulyan")) if rule != "multi_krum" else None
    if osel is not None:
        assert winners == osel.winners
    want, gap = O.coordinate_phase(Gh, winners, sets, h.beta)
    assert_outputs_match(out, want, G=Gh, tables=dict(winners=winners, sets=sets, beta=h.beta, gap=gap))
