"""The allocation-free distance entry point (gar_pairwise_distances_static).

It exists for callers that cannot allocate device memory when they aggregate --
code running inside another framework's memory pool, under a fixed memory
budget, or in a latency-critical loop -- so its scratch is a fixed array inside
the library.  Here it is called through the C ABI twice in a row (the array keeps
the first call's contents, so the second call checks that what must start at
zero is cleared) and compared with the ordinary entry point, which uses a
workspace.  This file is collected last on purpose."""
import pytest
import torch

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module")
def pkg():
    import __graft_entry__ as entry
    entry.build()
    import paper_1905_04374_b200 as p
    return p


@pytest.mark.parametrize("cfg,d", [(5, 300_004), (3, 200_003), (4, 70_000)])
def test_static_scratch_matches_workspace_path_twice(pkg, cfg, d):
    G, _ = pkg.workloads.make_gradients(cfg, d=d, device=DEV)
    n = G.shape[0]
    want = pkg.gar_pairwise_distances(G).clone()
    got = torch.full((n, n), -1.0, dtype=torch.float64, device=DEV)
    for call in range(2):
        got.fill_(-1.0)
        pkg.gar_pairwise_distances_static(G, got)
        torch.cuda.synchronize()
        # same kernels, same reduction order: the tolerance of the distance tests (1e-6 relative)
        # is met with room to spare -- the results are in fact identical
        assert torch.allclose(got, want, rtol=1e-6, atol=0.0), f"call {call}: max diff {(got - want).abs().max()}"
        assert torch.equal(got, got.T) and torch.all(torch.diagonal(got) == 0)


def test_static_scratch_rejects_too_many_rows(pkg):
    fake = 4096
    L = pkg.lib()
    assert L.gar_pairwise_distances_static(fake, 65, 100, 100, fake, None) == 3      # GAR_ERR_UNSUPPORTED
    assert L.gar_pairwise_distances_static(None, 10, 100, 100, fake, None) == 1
    assert "64" in pkg.gar_status_string(3)
