"""Helpers shared by the GPU parity tests: one context per session, tensor plumbing."""
import numpy as np
import torch

from paper_2603_05035_b200 import binding, inputs


def make_ctx(n=4300, k=0, d=4096, p=12288, dtype="bf16"):
    ctx = binding.Context(0)
    ctx.ensure_workspace(n, k, d, p, dtype)
    return ctx


def dev(x, dtype=torch.float32):
    return torch.as_tensor(np.ascontiguousarray(x)).to(device="cuda", dtype=dtype).contiguous()


def f64(t):
    return inputs.to_f64_numpy(t)


def padded(m, ld, dtype):
    return torch.full((m, ld), float("nan"), device="cuda", dtype=dtype)


def sample_rows(n, count, seed, extra=(), tile=128):
    """Row subset for sampled parity: first, last, both sides of every tile edge (so every `tile`-row tile of the
    output contributes at least two rows), the rows named in `extra`, and random rows up to `count` (the edge rows are
    kept even where they exceed it)."""
    rng = np.random.default_rng(seed)
    rows = {0, n - 1, *[r for r in extra if 0 <= r < n]}
    for edge in range(tile, n, tile):
        rows.update((edge - 1, edge))
    for t0 in range(0, n, tile):                       # a last, short tile still gets two rows
        t1 = min(n, t0 + tile)
        rows.update((t0, t1 - 1))
    while len(rows) < min(count, n):
        rows.add(int(rng.integers(0, n)))
    return np.array(sorted(rows), dtype=np.int64)
