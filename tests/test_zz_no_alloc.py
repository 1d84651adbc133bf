"""The allocation-free distance entry point (gar_pairwise_distances_static).

It exists for callers that cannot allocate device memory when they aggregate --
code running inside another framework's memory pool, under a fixed memory
budget, or in a latency-critical loop -- so its scratch is a fixed array inside
the library.  Here it is called through the C ABI twice in a row (the array keeps
the first call's contents, so the second call checks that what must start at
zero is cleared) and compared with the ordinary entry point, which uses a
workspace.  This file is collected last on purpose."""
import os
import subprocess
import sys

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


_FRESH_PROCESS = r"""
import sys, torch
sys.path.insert(0, sys.argv[1])
import paper_1905_04374_b200 as pkg
dev = "cuda:0"
inputs = []
for n, d in ((15, 300_032), (39, 200_064), (64, 70_016)):
    G = pkg.workloads.make_uniform(n, d, device=dev, seed=n)
    inputs.append((G, torch.empty(n, n, dtype=torch.float64, device=dev)))
# first call on the device: looks up the scratch array's address and loads the kernels (module
# loading may reserve device memory once; that is the library image, not an allocation per call)
for G, D in inputs:
    pkg.gar_pairwise_distances_static(G, D)
torch.cuda.synchronize()
free_before, _ = torch.cuda.mem_get_info()
for _ in range(3):
    for G, D in inputs:
        pkg.gar_pairwise_distances_static(G, D)
torch.cuda.synchronize()
free_after, _ = torch.cuda.mem_get_info()
assert free_after == free_before, (free_before, free_after)
for G, D in inputs:
    n = G.shape[0]
    ref = torch.cdist(G.double(), G.double()) ** 2
    off = ~torch.eye(n, dtype=torch.bool, device=dev)
    assert torch.allclose(D[off], ref[off], rtol=1e-6, atol=0.0)
print("no-allocation check ok", free_before)
"""


def test_static_entry_allocates_nothing_in_a_fresh_process():
    """What the entry point is for: in a process where no other call of the library has run (so no
    cached workspace exists), repeated calls leave the device's free memory exactly as it was."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-c", _FRESH_PROCESS, root], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "no-allocation check ok" in res.stdout
