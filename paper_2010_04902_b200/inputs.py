"""Seeded synthetic inputs for the aggregation path: true file gradients, attack payloads and the
[r][f][d] replica array a parameter server would hold after all K workers have reported.

This module only *produces inputs*.  It contains none of the method's arithmetic (no vote, no
median, no distances, no assignment, no subset search): the worker-to-file table and the set of
Byzantine workers are arguments.  It is the one module that both the CUDA path's callers and the
CPU checker's callers may use, so that the two sides see identical bytes.

Shapes follow the paper's clusters (Sec. 6.1: K = 15 with (l, r) = (5, 3), K = 25 with
(l, r) = (5, 5); appendix tables for l = 7); the gradient length d is a free parameter.  The
three attacks are those of Sec. 6.1: ALIE (a function of the per-coordinate mean and standard
deviation of the batch's gradients), constant, and reversed gradient.
"""
from __future__ import annotations

import torch

_CHUNK = 1 << 21  # coordinates generated per step; part of the recipe (changes the stream)


def true_gradients(f: int, d: int, seed: int = 0, sigma: float = 0.1, heavy_tail_frac: float = 0.0,
                   device="cpu") -> torch.Tensor:
    """g[f][d] fp32 with g[i][j] = mu_j + sigma * z_ij, mu_j ~ N(0,1) per coordinate, z_ij ~ N(0,1).

    With heavy_tail_frac > 0, that fraction of the coordinates (chosen by a seeded uniform draw)
    uses z_ij ~ Student-t with 2 degrees of freedom instead, drawn through its closed-form
    quantile (2u - 1) / sqrt(2u(1 - u)).
    """
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(int(seed))
    g = torch.empty((f, d), dtype=torch.float32, device=dev)
    for j0 in range(0, d, _CHUNK):
        n = min(_CHUNK, d - j0)
        mu = torch.randn(n, generator=gen, device=dev, dtype=torch.float32)
        z = torch.randn((f, n), generator=gen, device=dev, dtype=torch.float32)
        if heavy_tail_frac > 0.0:
            heavy = torch.rand(n, generator=gen, device=dev) < heavy_tail_frac
            u = torch.rand((f, n), generator=gen, device=dev, dtype=torch.float32).clamp_(1e-6, 1.0 - 1e-6)
            t = (2.0 * u - 1.0) / torch.sqrt(2.0 * u * (1.0 - u))
            z = torch.where(heavy.unsqueeze(0), t, z)
        g[:, j0:j0 + n] = mu.unsqueeze(0) + sigma * z
    return g


def integer_gradients(f: int, d: int, seed: int = 0, lo: int = -8, hi: int = 8, device="cpu") -> torch.Tensor:
    """Small-integer-valued fp32 rows: every sum and product on them is exact in fp32 and fp64."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(int(seed))
    return torch.randint(lo, hi + 1, (f, d), generator=gen).to(torch.float32).to(device)


def alie_payload(g: torch.Tensor, z: float = 1.0) -> torch.Tensor:
    """One vector for all colluding workers: per-coordinate mean minus z population standard
    deviations, both taken over the f true file gradients."""
    out = torch.empty(g.shape[1], dtype=torch.float32, device=g.device)
    for j0 in range(0, g.shape[1], _CHUNK):
        blk = g[:, j0:j0 + _CHUNK]
        out[j0:j0 + _CHUNK] = blk.mean(dim=0) - z * blk.std(dim=0, unbiased=False)
    return out


def build_replicas(g: torch.Tensor, file_workers, byzantine, attack: str = "none", *, alie_z: float = 1.0,
                   reverse_scale: float = 100.0, constant: float = -100.0, seed: int = 1) -> torch.Tensor:
    """replicas[k][i] = g[i] when worker file_workers[i][k] is honest, else the attack payload.

    attack: "none" | "alie" | "reversed" | "constant" | "independent".  The first three after
    "none" are colluding attacks (all Byzantine copies of a file are identical); "independent"
    makes every Byzantine copy a different random vector, which exercises the plurality rule of
    the vote when honest copies are in the minority.
    """
    f, d = g.shape
    r = len(file_workers[0])
    byz = set(int(u) for u in byzantine)
    rep = torch.empty((r, f, d), dtype=torch.float32, device=g.device)
    payload = None
    if attack == "alie":
        payload = alie_payload(g, alie_z)
    gen = torch.Generator(device=g.device)
    gen.manual_seed(int(seed))
    for i in range(f):
        for k in range(r):
            if int(file_workers[i][k]) not in byz or attack == "none":
                rep[k, i] = g[i]
            elif attack == "alie":
                rep[k, i] = payload
            elif attack == "reversed":
                rep[k, i] = -reverse_scale * g[i]
            elif attack == "constant":
                rep[k, i].fill_(constant)
            elif attack == "independent":
                rep[k, i] = torch.randn(d, generator=gen, device=g.device, dtype=torch.float32)
            else:
                raise ValueError("unknown attack %r" % (attack,))
    return rep
