"""Seeded synthetic layers drawn directly on the GPU (timing inputs).

Same shapes and distributions as ``synth.make_layer`` but generated with a torch CUDA
generator, so that dozens of distinct layers can be built in seconds.  The values differ from
the numpy generator's; parity tests use ``synth``, the benchmark uses this module.  No method
arithmetic lives here.
"""
from __future__ import annotations

import torch

from .synth import LayerShape


def _normal_bf16(gen, size, std, device):
    return (torch.randn(size, generator=gen, device=device, dtype=torch.float32) * std).to(torch.bfloat16)


def _indices(gen, size, K, device):
    v = torch.randint(0, K, size, generator=gen, device=device, dtype=torch.int32)
    if K <= 256:
        return v.to(torch.uint8)
    # store the low 16 bits; values >= 32768 wrap to the same bit pattern in int16
    return torch.where(v >= 32768, v - 65536, v).to(torch.int16)


def _pack12(idx16: torch.Tensor) -> torch.Tensor:
    """Twelve-bit packing (two indices to three bytes, little end first) of an int16 index tensor
    whose last dimension is even; same byte layout as ``synth.pack12``."""
    v = idx16.to(torch.int32) & 0xFFFF
    lo, hi = v[..., 0::2], v[..., 1::2]
    out = torch.stack([lo & 0xFF, (lo >> 8) | ((hi & 0xF) << 4), hi >> 4], dim=-1).to(torch.uint8)
    return out.reshape(*idx16.shape[:-1], idx16.shape[-1] // 2 * 3).contiguous()


def make_device_layer(shp: LayerShape, seed: int, device="cuda") -> dict:
    """Returns keyword arguments for ``binding.MoeVqlrLayer`` plus ``x`` ([T][H] bf16)."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    H, I, E, S, d, K, r, T = shp.H, shp.I, shp.E, shp.S, shp.d, shp.K, shp.r, shp.T
    n_exp = E + S
    router_w = _normal_bf16(gen, (E, H), 0.02, device)
    bias = torch.randn(E, generator=gen, device=device, dtype=torch.float32) if shp.router_bias else None
    x = _normal_bf16(gen, (T, H), 1.0, device)
    dims = {"gate": (I, H), "up": (I, H), "down": (H, I)}
    vq = {"gate": shp.mode in ("full", "paper"), "up": shp.mode in ("full", "paper"),
          "down": shp.mode == "full"}
    shared_book = None
    projs = {}
    for p in (("up", "down") if shp.act == "relu2" else ("gate", "up", "down")):     # up-only experts: no gate
        out_dim, in_dim = dims[p]
        if vq[p]:
            if shp.per_projection_codebook or shared_book is None:
                book = _normal_bf16(gen, (K, d), 0.02, device)
                if not shp.per_projection_codebook:
                    shared_book = book
            else:
                book = shared_book
            idx = _indices(gen, (n_exp, out_dim, in_dim // d), K, device)
            projs[p] = dict(codebook=book,
                            idx=_pack12(idx) if shp.idx12 else idx,
                            basis=_normal_bf16(gen, (r, in_dim), in_dim ** -0.5, device) if r > 0 else None,
                            factor=_normal_bf16(gen, (n_exp, out_dim, r), 0.01, device) if r > 0 else None)
        else:
            projs[p] = dict(dense=_normal_bf16(gen, (n_exp, out_dim, in_dim), 0.02, device))
    return dict(H=H, I=I, E=E, k=shp.k, S=S, d=d, K=K if any(vq.values()) else 0, r=r,
                max_tokens=max(T, 1), router_w=router_w, router_bias=bias, gate=projs.get("gate"),
                up=projs["up"], down=projs["down"], act=shp.act, x=x,
                **({"idx12": True} if shp.idx12 else {}))
