"""Algorithmic bytes of one layer call: what the method itself has to move from HBM.

Counts follow the paper's per-projection load table (Appendix "Exact engine-work counts"):
shared loads of the code book (16 K d bits) and the basis (16 in r bits) once per token batch,
expert-private loads of the index map ((in out / d) b_J bits) and coefficients (16 out r bits)
once per distinct activated expert (Section 5.6: every batch size loads only the activated
experts), plus the router matrix, the dense bf16 projections where a projection is kept
uncompressed (Section 3.1), and the token vectors in and out.
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass(frozen=True)
class LayerBytes:
    router: int
    shared: int            # distinct code books and bases
    per_expert_gateup: int
    per_expert_down: int
    tokens_io: int
    n_active: int          # distinct activated experts, shared experts included
    lookups_per_expert_gateup: int = 0   # code-word selections (one per length-d block), gate + up
    lookups_per_expert_down: int = 0

    @property
    def per_expert(self) -> int:
        return self.per_expert_gateup + self.per_expert_down

    @property
    def total(self) -> int:
        return self.router + self.shared + self.n_active * self.per_expert + self.tokens_io

    @property
    def gateup_kernel(self) -> int:
        """Bytes the gate/up stage streams: private gate+up payloads of the active experts."""
        return self.n_active * self.per_expert_gateup

    @property
    def down_kernel(self) -> int:
        return self.n_active * self.per_expert_down

    @property
    def lookups(self) -> int:
        """Code-word selections of the whole layer (the paper's `H I / d` per projection and expert)."""
        return self.n_active * (self.lookups_per_expert_gateup + self.lookups_per_expert_down)


def index_bits(K: int, idx12: bool = False) -> int:
    """Deployed index width b_J(K): one byte up to K = 256, two bytes beyond, or twelve bits packed."""
    return 8 if K <= 256 else (12 if idx12 else 16)


def projection_private_bytes(kind_vq: bool, out_dim: int, in_dim: int, d: int, K: int, r: int,
                             idx12: bool = False) -> int:
    if kind_vq:
        return out_dim * (in_dim // d) * index_bits(K, idx12) // 8 + 2 * out_dim * r
    return 2 * out_dim * in_dim


def layer_bytes(*, H: int, I: int, E: int, d: int, K: int, r: int, T: int, mode: str,
                n_active: int, n_codebooks: int = 1, gate_up_share_basis: bool = False,
                up_only: bool = False, idx12: bool = False) -> LayerBytes:
    """mode: "full" (gate/up/down VQ+LR), "paper" (down dense bf16), "dense" (all dense bf16).
    n_active counts distinct activated experts including always-on shared experts.
    up_only: experts without a gate projection (one projection onto the intermediate size)."""
    n_gu = 1 if up_only else 2
    vq_gu = mode in ("full", "paper")
    vq_d = mode == "full"
    shared = 0
    if vq_gu or vq_d:
        shared += n_codebooks * 2 * K * d
    if vq_gu and r > 0:
        shared += (1 if gate_up_share_basis or up_only else 2) * 2 * r * H
    if vq_d and r > 0:
        shared += 2 * r * I
    return LayerBytes(router=2 * E * H, shared=shared,
                      per_expert_gateup=n_gu * projection_private_bytes(vq_gu, I, H, d, K, r, idx12),
                      per_expert_down=projection_private_bytes(vq_d, H, I, d, K, r, idx12),
                      tokens_io=2 * 2 * T * H, n_active=n_active,
                      lookups_per_expert_gateup=n_gu * I * (H // d) if vq_gu else 0,
                      lookups_per_expert_down=H * (I // d) if vq_d else 0)


def dense_equivalent_bytes(H: int, I: int, n_active: int) -> int:
    """bf16 bytes of the same experts stored uncompressed (3 H I weights each)."""
    return n_active * 3 * 2 * H * I
