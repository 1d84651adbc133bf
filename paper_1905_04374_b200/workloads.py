"""Seeded synthetic worker gradients for the aggregation benchmarks and tests.

This module only draws inputs.  It holds none of the aggregation rules'
arithmetic and is the one piece shared by the CUDA path's tests and the CPU
oracle's tests: both sides receive the very same fp32 bits.

Each workload is n rows (workers) of dimension d, f of which are "Byzantine"
rows built from the honest ones.  Columns are drawn chunk by chunk, every chunk
from its own generator seeded by (seed, chunk index), so a matrix of tens of GB
is produced in place on the device without large temporaries and any column
range can be re-drawn alone.  A CPU generator and a CUDA generator give
different numbers for the same seed; draw once and copy.

"honest mean" / "honest std" are the per-coordinate mean and population
standard deviation over the n-f honest rows of the chunk.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

CHUNK = 1 << 21          # columns per independently seeded chunk
BASE_SEED = 190504374


@dataclass(frozen=True)
class Workload:
    name: str
    n: int
    f: int
    d: int
    honest: str          # kind of honest noise
    mean_std: float      # std of the shared mean vector
    noise_std: float     # std (scale) of the per-worker noise
    attack: str          # kind of Byzantine rows


WORKLOADS = {
    # shared mean N(0, 0.1) read as variance 0.1; i.i.d. N(0,1) noise; f rows = -10 x honest mean
    1: Workload("n11_f2_d1e5", 11, 2, 100_000, "normal", 0.1 ** 0.5, 1.0, "neg_mean_x10"),
    # shared mean N(0,1) + N(0,0.5^2); f rows = honest mean - 1.5 x honest std
    2: Workload("n23_f5_d1e6", 23, 5, 1_000_000, "normal", 1.0, 0.5, "small_perturbation"),
    # shared mean N(0,1e-3) (variance) + N(0,(1e-2)^2); f rows ~ N(0,100^2) each
    3: Workload("n39_f9_d25.6e6", 39, 9, 25_600_000, "normal", 1e-3 ** 0.5, 1e-2, "large_random"),
    # shared mean N(0,1) + Student-t(3); half sign-flipped mean, half small perturbation
    4: Workload("n51_f12_d1e8", 51, 12, 100_000_000, "student_t3", 1.0, 1.0, "mixed_flip_perturbation"),
    # shared mean N(0,1) + N(0,0.1^2); f rows = -10 x honest mean
    5: Workload("n15_f3_d1e9", 15, 3, 1_000_000_000, "normal", 1.0, 0.1, "neg_mean_x10"),
}


def byzantine_rows(n: int, f: int, seed: int, placement: str = "random"):
    """Which rows are Byzantine: a seeded random f-subset, or the last f rows."""
    if placement == "last":
        return list(range(n - f, n))
    rs = np.random.RandomState(seed % (2 ** 31))
    return sorted(int(i) for i in rs.choice(n, f, replace=False))


def _fill_chunk(G, c0, c1, wl: Workload, byz, seed, chunk_idx):
    dev = G.device
    gen = torch.Generator(device=dev)
    gen.manual_seed((seed * 1_000_003 + chunk_idx) % (2 ** 62))
    c = c1 - c0
    n, f = wl.n, wl.f
    honest = [i for i in range(n) if i not in byz]
    h = len(honest)
    mu = torch.randn(c, generator=gen, device=dev, dtype=torch.float32) * wl.mean_std
    if wl.honest == "normal":
        noise = torch.randn(h, c, generator=gen, device=dev, dtype=torch.float32)
    elif wl.honest == "student_t3":
        z = torch.randn(h, c, generator=gen, device=dev, dtype=torch.float32)
        chi = torch.zeros(h, c, device=dev, dtype=torch.float32)
        for _ in range(3):
            chi += torch.randn(h, c, generator=gen, device=dev, dtype=torch.float32) ** 2
        noise = z / torch.sqrt(chi / 3.0)
        del z, chi
    else:
        raise ValueError(wl.honest)
    H = noise.mul_(wl.noise_std).add_(mu)           # h x c honest rows
    hmean = H.mean(dim=0)
    for k, i in enumerate(honest):
        G[i, c0:c1] = H[k]
    if f == 0:
        return
    if wl.attack == "neg_mean_x10":
        for i in byz:
            G[i, c0:c1] = -10.0 * hmean
    elif wl.attack == "small_perturbation":
        hstd = H.std(dim=0, unbiased=False)
        for i in byz:
            G[i, c0:c1] = hmean - 1.5 * hstd
    elif wl.attack == "large_random":
        for i in byz:
            G[i, c0:c1] = torch.randn(c, generator=gen, device=dev, dtype=torch.float32) * 100.0
    elif wl.attack == "mixed_flip_perturbation":
        hstd = H.std(dim=0, unbiased=False)
        for k, i in enumerate(byz):
            G[i, c0:c1] = (-hmean) if k % 2 == 0 else (hmean - 1.5 * hstd)
    else:
        raise ValueError(wl.attack)


def make_gradients(cfg: int, d: int | None = None, device="cpu", seed: int | None = None,
                   placement: str = "random", n: int | None = None, f: int | None = None,
                   out: torch.Tensor | None = None, columns: tuple | None = None):
    """Draw workload `cfg` (1..5), optionally at another dimension d (and n, f).

    Returns (G, byz): G is an fp32 tensor [n, d] on `device`, byz the sorted
    list of Byzantine row indices.  `out`, if given, is filled instead of a
    new tensor (it must be [n, >= d] fp32; only the first d columns are set).
    `columns` = (c0, c1), c0 a multiple of CHUNK, draws only that column range
    of the d-dimensional workload (the slice one GPU of a sharded run owns): the
    result is [n, c1 - c0] and equals G[:, c0:c1] of the full draw bit for bit.
    """
    wl = WORKLOADS[cfg]
    if d is not None or n is not None or f is not None:
        wl = Workload(wl.name, n or wl.n, wl.f if f is None else f, d or wl.d,
                      wl.honest, wl.mean_std, wl.noise_std, wl.attack)
    if seed is None:
        seed = BASE_SEED + cfg
    byz = byzantine_rows(wl.n, wl.f, seed, placement)
    lo, hi = (0, wl.d) if columns is None else columns
    if lo % CHUNK != 0 or not (0 <= lo < hi <= wl.d):
        raise ValueError("columns must start on a multiple of CHUNK and lie inside [0, d]")
    G = out if out is not None else torch.empty(wl.n, hi - lo, dtype=torch.float32, device=device)
    for c0 in range(lo, hi, CHUNK):
        c1 = min(c0 + CHUNK, wl.d, hi)
        # a chunk is always drawn whole (its generator is consumed in a fixed order) ...
        if c1 - c0 == min(CHUNK, wl.d - c0):
            _fill_chunk(G, c0 - lo, c1 - lo, wl, byz, seed, c0 // CHUNK)
        else:                                 # ... and cut afterwards when the range ends inside it
            full = torch.empty(wl.n, min(CHUNK, wl.d - c0), dtype=torch.float32, device=G.device)
            _fill_chunk(full, 0, full.shape[1], wl, byz, seed, c0 // CHUNK)
            G[:, c0 - lo:c1 - lo] = full[:, :c1 - c0]
    return G, byz


def shard_columns(d: int, world: int, rank: int):
    """Column range [c0, c1) of rank `rank` when d columns are split over `world` GPUs in whole
    chunks of CHUNK columns (the last rank takes the ragged end)."""
    chunks = (d + CHUNK - 1) // CHUNK
    per = (chunks + world - 1) // world
    c0 = min(rank * per * CHUNK, d)
    c1 = min((rank + 1) * per * CHUNK, d)
    return c0, c1


def make_uniform(n: int, d: int, device="cpu", seed: int = BASE_SEED):
    """The paper's own timing inputs (Section 5.1): n rows i.i.d. U(0,1)^d."""
    G = torch.empty(n, d, dtype=torch.float32, device=device)
    for ci, c0 in enumerate(range(0, d, CHUNK)):
        gen = torch.Generator(device=G.device)
        gen.manual_seed((seed * 1_000_003 + ci) % (2 ** 62))
        c1 = min(c0 + CHUNK, d)
        G[:, c0:c1] = torch.rand(n, c1 - c0, generator=gen, device=G.device, dtype=torch.float32)
    return G
