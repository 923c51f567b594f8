"""Seeded synthetic inputs shared by the oracle tests and the CUDA tests.

Only random draws and dtype rounding live here -- none of the method's arithmetic.
Recipe (one torch CPU generator per workload, float64 draws, fixed order Q, K, V, E, F, W,
each rounded once to the I/O dtype):
  Q, K, V ~ N(0,1) * d^(-1/4)      [B,H,N,d]   (so that q.k has the 1/sqrt(d) softmax scale)
  E, F    ~ N(0, 1/k)              [k,N]       (Section 2.1 of arxiv 2306.15799)
  W       block-orthogonal Gaussian [m,d]: for every block of d rows, the rows of an orthogonal
          matrix (sign-fixed QR factor of a d x d Gaussian, i.e. Haar distributed) rescaled to the norms of independent d-dimensional
          Gaussian vectors (chi_d distributed); the last block is truncated when d does not
          divide m.  RNN workloads have no W.
"""
from __future__ import annotations

import torch

from .configs import PERFORMER, FusedWorkload, Workload


def _io_dtype(io: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "fp32": torch.float32}[io]


def block_orthogonal_features(m: int, d: int, gen: torch.Generator) -> torch.Tensor:
    """[m,d] float64 random-feature matrix with orthogonal rows inside each block of d rows."""
    blocks = []
    rows_left = m
    while rows_left > 0:
        g = torch.randn(d, d, generator=gen, dtype=torch.float64)
        q, r = torch.linalg.qr(g)
        q = q * torch.sign(torch.diagonal(r))[None, :]      # Haar-distributed (sign-fixed) factor
        norms = torch.randn(d, d, generator=gen, dtype=torch.float64).norm(dim=1)
        blk = q.t() * norms[:, None]
        take = min(d, rows_left)
        blocks.append(blk[:take])
        rows_left -= take
    return torch.cat(blocks, dim=0)


def make_inputs(w: Workload) -> dict:
    """CPU tensors in the workload's I/O dtype: Q, K, V [B,H,N,d], E, F [k,N], W [m,d] or None."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(w.seed)
    dt = _io_dtype(w.io)
    scale = float(w.d) ** -0.25

    def draw(shape, s):
        x = torch.randn(*shape, generator=gen, dtype=torch.float64)
        return x.mul_(s).to(dt)

    out = {}
    for name in ("Q", "K", "V"):
        out[name] = draw((w.B, w.H, w.N, w.d), scale)
    for name in ("E", "F"):
        out[name] = draw((w.k, w.N), float(w.k) ** -0.5)
    if w.variant == PERFORMER:
        out["W"] = block_orthogonal_features(w.m, w.d, gen).to(dt)
    else:
        out["W"] = None
    return out


def make_fused_inputs(w: FusedWorkload) -> dict:
    """CPU tensors for the entry point with un-projected inputs, drawn in the order Xq, Xk, Xv (one X when
    `w.shared_x`), Wq, Wk, Wv, E, F, W:  X ~ N(0,1) [B,N,dm];  Wq, Wk, Wv ~ N(0, 1/dm) * d^(-1/4) [dm,H*d], so
    that X W has the distribution make_inputs gives Q, K and V;  E, F, W as in make_inputs."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(w.seed)
    dt = _io_dtype(w.io)

    def draw(shape, s):
        x = torch.randn(*shape, generator=gen, dtype=torch.float64)
        return x.mul_(s).to(dt)

    out = {}
    if w.shared_x:
        out["Xq"] = out["Xk"] = out["Xv"] = draw((w.B, w.N, w.dm), 1.0)
    else:
        for name in ("Xq", "Xk", "Xv"):
            out[name] = draw((w.B, w.N, w.dm), 1.0)
    for name in ("Wq", "Wk", "Wv"):
        out[name] = draw((w.dm, w.H * w.d), float(w.dm) ** -0.5 * float(w.d) ** -0.25)
    for name in ("E", "F"):
        out[name] = draw((w.k, w.N), float(w.k) ** -0.5)
    out["W"] = block_orthogonal_features(w.m, w.d, gen).to(dt) if w.variant == PERFORMER else None
    return out
