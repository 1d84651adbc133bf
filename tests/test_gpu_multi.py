"""gar_aggregate_multi against the oracle: many small tensors in one launch sequence.
joint=False: every tensor is a problem of its own and is compared with the oracle run on that
tensor.  joint=True: the tensors are the pieces of one gradient (Section 2.1: the rule acts on the
whole gradient), compared with the oracle run on the concatenation."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import gar_oracle as O
from tests._compare import assert_outputs_match, assert_selection_match, rule_tables

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# lengths of the "layers": single coordinates, odd lengths (rows then start unaligned), lengths
# around the kernels' slab and vector widths, and one that takes a few hundred CTAs
DIMS = [1, 3, 64, 10, 1000, 4099, 512, 2, 65_536, 30_001, 262_148, 7, 1728, 36_864]


@pytest.fixture(scope="module")
def pkg():
    import __graft_entry__ as entry
    entry.build()
    import paper_1905_04374_b200 as p
    return p


def layers(pkg, cfg, dims, strided=False):
    """One draw of the workload's recipe at d = sum(dims), cut into tensors of their own.  Every
    tensor is a fresh allocation (so its rows start wherever its length puts them); `strided`
    makes every third one a view into a wider buffer (ld > d, a misaligned first row)."""
    total = sum(dims)
    G, byz = pkg.workloads.make_gradients(cfg, d=total, device=DEV)
    parts, c0 = [], 0
    for k, d in enumerate(dims):
        piece = G[:, c0:c0 + d]
        if strided and k % 3 == 1:
            wide = torch.zeros(G.shape[0], d + 5, dtype=torch.float32, device=DEV)
            wide[:, 3:3 + d] = piece
            parts.append(wide[:, 3:3 + d])
        else:
            parts.append(piece.contiguous())
        c0 += d
    return G, parts, byz


def read_selections(pkg, buf, count):
    size = C.sizeof(pkg.GarSelection)
    raw = buf.cpu().numpy().tobytes()
    return [pkg.GarSelection.from_buffer_copy(raw[t * size:(t + 1) * size]) for t in range(count)]


def check_tensor(pkg, rule, Gh, f, got, sel, D_gpu=None):
    """One problem against the oracle: the distances, the selection where the oracle's score gap is
    clear, the output (on the GPU's own selection where a near-tie let the two differ)."""
    n = Gh.shape[0]
    want, tab = rule_tables(rule, Gh, f)
    if tab is None:
        assert_outputs_match(got, want)
        return 0
    if D_gpu is not None:
        D = O.pairwise_sq_distances(Gh)
        assert np.all(np.abs(D_gpu - D) <= 1e-6 * D + 1e-30), np.abs(D_gpu - D).max()
        assert np.array_equal(D_gpu, D_gpu.T) and np.all(np.diag(D_gpu) == 0)
    assert sel.status == 0
    preagg = rule in ("multi_krum", "multi_bulyan")
    compared = assert_selection_match(sel, tab["rounds"], preagg)
    if compared == len(tab["rounds"]):
        assert_outputs_match(got, want, G=Gh, tables=tab)
    else:
        winners = [sel.winners[r] for r in range(sel.theta)]
        sets = [[i for i in range(n) if (sel.sets[r] >> i) & 1] for r in range(sel.theta)] if preagg else None
        want2, gap2 = O.coordinate_phase(Gh, winners, sets, sel.beta)
        assert_outputs_match(got, want2, G=Gh, tables=dict(winners=winners, sets=sets, beta=sel.beta, gap=gap2))
    return compared


@pytest.mark.parametrize("rule", ["multi_bulyan", "bulyan", "multi_krum", "krum", "median", "average"])
@pytest.mark.parametrize("cfg", [1, 2, 3])
def test_independent_problems(pkg, rule, cfg):
    wl = pkg.workloads.WORKLOADS[cfg]
    n, f = wl.n, wl.f
    _, parts, _ = layers(pkg, cfg, DIMS, strided=True)
    count = len(parts)
    dist = torch.full((count, n, n), -1.0, dtype=torch.float64, device=DEV)
    sels = torch.zeros(count * C.sizeof(pkg.GarSelection), dtype=torch.uint8, device=DEV)
    outs = pkg.gar_aggregate_multi(rule, parts, f, dist_out=dist, selection_out=sels)
    torch.cuda.synchronize()
    sel_host = read_selections(pkg, sels, count)
    D = dist.cpu().numpy()
    needs_dist = rule not in ("median", "average")
    total = 0
    for t, (g, o) in enumerate(zip(parts, outs)):
        assert o.shape == (g.shape[1],)
        total += check_tensor(pkg, rule, g.cpu().numpy(), f, o.cpu().numpy(), sel_host[t], D[t] if needs_dist else None)
    if needs_dist:
        print(f"{rule} workload {cfg}: {total} rounds compared exactly over {count} tensors")
        assert total >= count // 2     # the first round at least, nearly everywhere


@pytest.mark.parametrize("rule", ["multi_bulyan", "bulyan", "multi_krum"])
@pytest.mark.parametrize("cfg", [1, 2, 3])
def test_joint_is_the_rule_on_the_concatenation(pkg, rule, cfg):
    wl = pkg.workloads.WORKLOADS[cfg]
    n, f = wl.n, wl.f
    G, parts, byz = layers(pkg, cfg, DIMS, strided=True)
    dist = torch.empty(n, n, dtype=torch.float64, device=DEV)
    sel = pkg.new_selection(DEV)
    outs = pkg.gar_aggregate_multi(rule, parts, f, joint=True, dist_out=dist, selection_out=sel)
    torch.cuda.synchronize()
    got = torch.cat(outs).cpu().numpy()
    compared = check_tensor(pkg, rule, G.cpu().numpy(), f, got, pkg.read_selection(sel), dist.cpu().numpy())
    assert compared >= 1
    # the same call through gar_aggregate_ex on the concatenation selects the same gradients
    sel2 = pkg.new_selection(DEV)
    pkg.gar_aggregate_ex(rule, G, f, selection_out=sel2)
    a, b = pkg.read_selection(sel), pkg.read_selection(sel2)
    assert a.winners[0] == b.winners[0]
    if rule != "bulyan" and cfg in (1, 3):
        for r in range(a.theta):
            assert not any((a.sets[r] >> i) & 1 for i in byz), "a Byzantine row was averaged"


@pytest.mark.parametrize("n,f", [(7, 1), (16, 3), (17, 3), (33, 4), (64, 15)])
def test_row_counts_and_one_long_tensor_among_short_ones(pkg, n, f):
    dims = [5, 1_200_004, 33, 4096, 3]
    gen = torch.Generator(device=DEV)
    gen.manual_seed(1000 + n)
    parts = [torch.randn(n, d, generator=gen, device=DEV, dtype=torch.float32) for d in dims]
    for g in parts:
        g[-f:] += 50.0                       # f far-away rows
    count = len(parts)
    sels = torch.zeros(count * C.sizeof(pkg.GarSelection), dtype=torch.uint8, device=DEV)
    dist = torch.empty(count, n, n, dtype=torch.float64, device=DEV)
    outs = pkg.gar_aggregate_multi("multi_bulyan", parts, f, dist_out=dist, selection_out=sels)
    torch.cuda.synchronize()
    sel_host = read_selections(pkg, sels, count)
    for t, (g, o) in enumerate(zip(parts, outs)):
        check_tensor(pkg, "multi_bulyan", g.cpu().numpy(), f, o.cpu().numpy(), sel_host[t], dist[t].cpu().numpy())


def test_repeatable_and_equal_to_single_calls_where_the_kernels_coincide(pkg):
    # two calls give the same bits; tensors below the tensor-core kernel's size and of n > 16 run
    # the same difference-form distance kernel as gar_aggregate_ex, so the selections are identical
    cfg = 2
    wl = pkg.workloads.WORKLOADS[cfg]
    _, parts, _ = layers(pkg, cfg, [4099, 1000, 20_000])
    ws = torch.zeros(pkg.gar_multi_workspace_bytes("multi_bulyan", wl.n, wl.f, len(parts)), dtype=torch.uint8, device=DEV)
    a = [o.clone() for o in pkg.gar_aggregate_multi("multi_bulyan", parts, wl.f, workspace=ws)]
    ws.fill_(0xAB)                            # the workspace may hold anything on entry
    b = pkg.gar_aggregate_multi("multi_bulyan", parts, wl.f, workspace=ws)
    for x, y, g in zip(a, b, parts):
        assert torch.equal(x, y)
        sel = pkg.new_selection(DEV)
        single = pkg.gar_aggregate_ex("multi_bulyan", g, wl.f, selection_out=sel)
        assert pkg.read_selection(sel).status == 0
        assert_outputs_match(x.cpu().numpy(), single.cpu().numpy().astype(np.float64))


def test_many_tensors(pkg):
    # 300 tensors of 1 to 3000 coordinates: one CTA each in every stage
    n, f = 11, 2
    rng = np.random.default_rng(5)
    dims = [int(v) for v in rng.integers(1, 3000, size=300)]
    gen = torch.Generator(device=DEV)
    gen.manual_seed(77)
    parts = [torch.randn(n, d, generator=gen, device=DEV, dtype=torch.float32) for d in dims]
    outs = pkg.gar_aggregate_multi("multi_bulyan", parts, f)
    torch.cuda.synchronize()
    for t in (0, 1, 17, 150, 299):
        want, _, _ = O.multi_bulyan(parts[t].cpu().numpy(), f)
        got = outs[t].cpu().numpy()
        # random rows: scores are close, so compare loosely on the selection and exactly on range
        assert got.shape == want.shape and np.all(np.isfinite(got))
        lo, hi = parts[t].min(0).values.cpu().numpy(), parts[t].max(0).values.cpu().numpy()
        assert np.all(got >= lo - 1e-6) and np.all(got <= hi + 1e-6)


def test_argument_errors(pkg):
    n, f = 11, 2
    g = torch.zeros(n, 8, dtype=torch.float32, device=DEV)
    with pytest.raises(pkg.GarError) as e:
        pkg.gar_aggregate_multi("multi_bulyan", [g], 3)                # n < 4f + 3
    assert e.value.status == 2
    with pytest.raises(pkg.GarError) as e:
        pkg.gar_aggregate_multi("multi_bulyan", [g], f, workspace=torch.zeros(256, dtype=torch.uint8, device=DEV))
    assert e.value.status == 4
    with pytest.raises(ValueError):
        pkg.gar_aggregate_multi("multi_bulyan", [g, torch.zeros(n + 1, 8, dtype=torch.float32, device=DEV)], f)


@pytest.mark.parametrize("joint", [False, True])
@pytest.mark.parametrize("momentum", [False, True])
def test_fused_sgd_step_per_tensor(pkg, joint, momentum):
    """The SGD step of Eq. 2 fused into every tensor's store: x <- x - lr (mu v + g), with g the
    aggregate the same call returns for the tensor when asked to store it."""
    cfg = 1
    wl = pkg.workloads.WORKLOADS[cfg]
    dims = [7, 1000, 4099, 65_536, 30_001]
    _, parts, _ = layers(pkg, cfg, dims, strided=True)
    lr, mu = 0.1, 0.9
    gen = torch.Generator(device=DEV)
    gen.manual_seed(9)
    xs = [torch.randn(d, generator=gen, device=DEV, dtype=torch.float32) for d in dims]
    vs = [torch.randn(d, generator=gen, device=DEV, dtype=torch.float32) for d in dims] if momentum else None
    x0 = [x.cpu().numpy().astype(np.float64) for x in xs]
    v0 = [v.cpu().numpy().astype(np.float64) for v in vs] if momentum else None
    # the aggregates alone, then the same call with the step and no stored aggregate
    gs = [g.clone() for g in pkg.gar_aggregate_multi("multi_bulyan", parts, wl.f, joint=joint)]
    res = pkg.gar_aggregate_multi("multi_bulyan", parts, wl.f, joint=joint, sgd_params=xs, sgd_momentum_bufs=vs,
                                  sgd_lr=lr, sgd_momentum=mu if momentum else 0.0, store_out=False)
    torch.cuda.synchronize()
    assert res is None
    for t in range(len(dims)):
        g = gs[t].cpu().numpy().astype(np.float64)
        want_x, want_v = O.sgd_step(x0[t], g, lr, momentum_buf=v0[t] if momentum else None, momentum=mu)
        got_x = xs[t].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got_x - want_x) <= 1e-6 * (1.0 + np.abs(want_x)))
        if momentum:
            got_v = vs[t].cpu().numpy().astype(np.float64)
            assert np.all(np.abs(got_v - want_v) <= 1e-6 * (1.0 + np.abs(want_v)))
    # both at once: the stored aggregates are the ones the step used
    outs = pkg.gar_aggregate_multi("multi_bulyan", parts, wl.f, joint=joint, sgd_params=xs, sgd_momentum_bufs=vs,
                                   sgd_lr=lr, sgd_momentum=mu if momentum else 0.0)
    torch.cuda.synchronize()
    for a, b in zip(outs, gs):
        assert torch.equal(a, b)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("cfg", [1, 2])
@pytest.mark.parametrize("joint", [False, True])
def test_sixteen_bit_gradients(pkg, dtype, cfg, joint):
    """bfloat16 / binary16 tensors: every value is widened to fp32 exactly when a kernel loads it,
    so the oracle fed the same 16-bit values is the reference (exact ties between 16-bit values
    are frequent: up to 1 % of the coordinates may rest on the tie-aware check)."""
    wl = pkg.workloads.WORKLOADS[cfg]
    n, f = wl.n, wl.f
    dims = [3, 1000, 4099, 65_536, 30_001, 262_144]
    G32, parts32, _ = layers(pkg, cfg, dims, strided=True)
    parts = []
    for k, g in enumerate(parts32):
        if g.is_contiguous():
            parts.append(g.to(dtype))
        else:                                         # keep a strided, misaligned view
            wide = torch.zeros(n, g.shape[1] + 5, dtype=dtype, device=DEV)
            wide[:, 3:3 + g.shape[1]] = g.to(dtype)
            parts.append(wide[:, 3:3 + g.shape[1]])
    count = len(parts)
    nsel = 1 if joint else count
    sels = torch.zeros(nsel * C.sizeof(pkg.GarSelection), dtype=torch.uint8, device=DEV)
    dist = torch.empty(nsel, n, n, dtype=torch.float64, device=DEV)
    outs = pkg.gar_aggregate_multi("multi_bulyan", parts, f, joint=joint, dist_out=dist, selection_out=sels)
    torch.cuda.synchronize()
    sel_host = read_selections(pkg, sels, nsel)
    problems = [(torch.cat([p.to(torch.float32) for p in parts], dim=1), torch.cat(outs), 0)] if joint else \
        [(p.to(torch.float32), o, t) for t, (p, o) in enumerate(zip(parts, outs))]
    for gh, o, t in problems:
        Gh = gh.cpu().numpy()
        got = o.cpu().numpy()
        want, tab = rule_tables("multi_bulyan", Gh, f)
        D = dist[t].cpu().numpy()
        wantD = O.pairwise_sq_distances(Gh)
        pos = wantD > 0
        assert np.max(np.abs(D - wantD)[pos] / wantD[pos]) <= 1e-6 and np.all(D[~pos] == 0)
        sel = sel_host[t]
        assert sel.status == 0
        compared = assert_selection_match(sel, tab["rounds"], True)
        if compared == len(tab["rounds"]):
            assert_outputs_match(got, want, G=Gh, tables=tab, max_tie_frac=1e-2)
        else:
            winners = [sel.winners[r] for r in range(sel.theta)]
            sets = [[i for i in range(n) if (sel.sets[r] >> i) & 1] for r in range(sel.theta)]
            want2, gap2 = O.coordinate_phase(Gh, winners, sets, sel.beta)
            assert_outputs_match(got, want2, G=Gh, tables=dict(winners=winners, sets=sets, beta=sel.beta, gap=gap2),
                                 max_tie_frac=1e-2)
