"""Seeded synthetic inputs: the p process buffers a reduction starts from.

This module only draws random numbers; it contains nothing of the reduction
method (no schedule, no combine order, no cost model), so that the library's
tests, its benchmark and the independent CPU checker can all be fed the very
same bytes.

The paper reduces arbitrary vectors (its MPI experiment uses `int` with `+`)
and uses no public data set, so each workload is described by its shape
(p processes x n elements), element type, value distribution and seed.
"""
from __future__ import annotations

import torch

DISTRIBUTIONS = ("int_pm2p20", "normal", "uniform_pm1")


def make_inputs(p: int, n: int, dist: str, seed: int, device: str = "cpu") -> torch.Tensor:
    """Return a [p, n] tensor: row i is process i's message.

    dist:
      "int_pm2p20"  int32, uniform integers in [-2^20, 2^20]
      "normal"      float32, N(0, 1)
      "uniform_pm1" float32, uniform in [-1, 1)
    The stream depends on (seed, device type); a consumer that needs the same
    bytes elsewhere copies the tensor rather than regenerating it.
    """
    if dist not in DISTRIBUTIONS:
        raise ValueError("unknown distribution %r" % (dist,))
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    if dist == "int_pm2p20":
        return torch.randint(-(1 << 20), (1 << 20) + 1, (p, n), dtype=torch.int32, device=device, generator=gen)
    if dist == "normal":
        out = torch.empty((p, n), dtype=torch.float32, device=device)
        # row by row keeps the temporary small for multi-GB arenas
        for i in range(p):
            out[i].normal_(0.0, 1.0, generator=gen)
        return out
    out = torch.empty((p, n), dtype=torch.float32, device=device)
    for i in range(p):
        out[i].uniform_(-1.0, 1.0, generator=gen)
    return out


# The workloads the benchmark and the parity tests name.  Each stands in for the
# paper's simulated / cluster workloads with the same shape.
WORKLOADS = {
    # name: (p, n, dist, seed, segment bytes, alpha, beta, gamma)
    "config1": dict(p=8, n=4096, dist="int_pm2p20", seed=0, seg_bytes=2048,
                    alpha=2e-6, beta=1e-10, gamma=5e-11),
    "config2": dict(p=64, n=1 << 20, dist="normal", seed=1, seg_bytes=16 << 10,
                    alpha=2e-6, beta=1e-10, gamma=5e-11),
    "config3": dict(p=256, n=1 << 22, dist="uniform_pm1", seed=2, seg_bytes=64 << 10,
                    alpha=2e-6, beta=1e-10, gamma=5e-11),
    "config4": dict(p=32, n=1 << 28, dist="normal", seed=3, seg_bytes=1 << 20,
                    alpha=5e-6, beta=2.5e-11, gamma=1e-11),
}
