"""The benchmark / parity workloads: shapes, I/O dtype and seeds.

Shapes follow the five FLuRKA forward configurations this library is measured on
(Linformer-Performer and Linformer-RNN instances of arxiv 2306.15799, Section 4).
No arithmetic of the method lives here.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

PERFORMER = 0
RNN = 1

BASE_SEED = 230615


@dataclass(frozen=True)
class Workload:
    name: str
    variant: int          # PERFORMER or RNN
    io: str               # "bf16" or "fp32"
    B: int
    H: int
    N: int
    d: int
    k: int
    m: int                # 0 for RNN
    seed: int

    @property
    def tokens(self) -> int:
        return self.B * self.H * self.N

    @property
    def elem_bytes(self) -> int:
        return 4 if self.io == "fp32" else 2

    def flops(self) -> int:
        """Counted FLOPs (2 per multiply-add) of one forward pass, all heads.

        PERFORMER: 4Nkd (down-projections) + 2(N+k)dm (feature GEMMs) + 2kmd + 2Nmd.
        RNN: the feature dimension is d and there is no W GEMM: 4Nkd + 2kd^2 + 2Nd^2.
        """
        N, d, k, m = self.N, self.d, self.k, self.m
        if self.variant == PERFORMER:
            per_head = 4 * N * k * d + 2 * (N + k) * d * m + 2 * k * m * d + 2 * N * m * d
        else:
            per_head = 4 * N * k * d + 2 * k * d * d + 2 * N * d * d
        return per_head * self.B * self.H

    def compulsory_bytes(self) -> int:
        """Q, K, V read and O written once; E, F read once (shared); W read once."""
        s = self.elem_bytes
        return 4 * self.B * self.H * self.N * self.d * s + 2 * self.k * self.N * s + self.m * self.d * s


@dataclass(frozen=True)
class FusedWorkload(Workload):
    """Eq. (2) with its linear maps inside the call: un-projected inputs [B,N,dm], maps [dm,H*d].
    `shared_x`: queries, keys and values are one and the same input (self-attention)."""
    dm: int = 0
    shared_x: bool = True

    def flops(self) -> int:
        """Appendix B's steps, 2 FLOPs per multiply-add: the contraction of the un-projected keys and values
        (4 N k dm per batch), W^Q on the N queries (2 N dm Hd), W^K and W^V on the k contracted rows
        (4 k dm Hd), then the per-head work of the plain forward without its own down-projection."""
        N, d, k, dm, Hd = self.N, self.d, self.k, self.dm, self.H * self.d
        per_batch = 4 * N * k * dm + 2 * N * dm * Hd + 4 * k * dm * Hd
        return per_batch * self.B + super().flops() - 4 * N * k * d * self.B * self.H

    def compulsory_bytes(self) -> int:
        """The inputs read once (one X when shared), O written once, E, F, the three maps and W read once."""
        s = self.elem_bytes
        x = self.B * self.N * self.dm * s * (1 if self.shared_x else 3)
        return x + self.tokens * self.d * s + 2 * self.k * self.N * s + 3 * self.dm * self.H * self.d * s + self.m * self.d * s


C1 = Workload("c1_perf_fp32_n256", PERFORMER, "fp32", 1, 2, 256, 32, 32, 64, BASE_SEED + 1000)
C2 = Workload("c2_rnn_bf16_n4096", RNN, "bf16", 8, 12, 4096, 64, 256, 0, BASE_SEED + 2000)
C3 = Workload("c3_perf_bf16_n16384", PERFORMER, "bf16", 4, 16, 16384, 64, 256, 256, BASE_SEED + 3000)
C4 = Workload("c4_perf_bf16_n131072", PERFORMER, "bf16", 1, 8, 131072, 128, 512, 256, BASE_SEED + 4000)


def c5(k: int, m: int) -> Workload:
    """Projection-size sweep point: k in {64,128,256,512}, m in {64,128,256}."""
    return Workload("c5_perf_bf16_n8192_k%d_m%d" % (k, m), PERFORMER, "bf16", 8, 12, 8192, 64, k, m,
                    BASE_SEED + 5000 + 8 * k + m // 64)


C5_GRID = [(k, m) for k in (64, 128, 256, 512) for m in (64, 128, 256)]

# c3's shape with the linear maps inside the call: d_m = H d = 1024, self-attention
F1 = FusedWorkload("f1_fused_perf_bf16_n16384_dm1024", PERFORMER, "bf16", 4, 16, 16384, 64, 256, 256, BASE_SEED + 6000,
                   dm=1024, shared_x=True)

BY_NAME = {w.name: w for w in (C1, C2, C3, C4, F1)}
BY_NAME.update({c5(k, m).name: c5(k, m) for (k, m) in C5_GRID})
ALIASES = {"c1": C1, "c2": C2, "c3": C3, "c4": C4, "f1": F1}


def get(name: str) -> Workload:
    if name in ALIASES:
        return ALIASES[name]
    return BY_NAME[name]


def shrink(w: Workload, **kw) -> Workload:
    """A smaller workload with the same recipe (used by parity tests)."""
    return replace(w, **kw)
