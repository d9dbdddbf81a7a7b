"""Seeded synthetic MoE layers in the VQ + shared-basis low-rank form.

This module only draws random tensors and packs them; it holds none of the method's
arithmetic (no routing, no reconstruction, no FFN).  Both the CPU oracle's tests and the
CUDA path's tests/bench take their inputs from here, so the two sides see the same bits.

Storage conventions (paper notation in brackets; Table 1 and Eq. 1 of the paper):
  * every bf16 tensor is a numpy ``uint16`` array holding the bf16 bit patterns;
  * ``codebook[K][d]``                    [weight code book, K words of length d]
  * ``idx[E+S][out][in/d]`` u8 / u16      [J_e, one index per length-d block along the
                                           contraction dimension]
  * ``basis[r][in]``  = D^T               [shared low-rank basis]
  * ``factor[E+S][out][r]`` = C_e^T       [expert-private coefficients]
  * ``dense[E+S][out][in]``               [uncompressed bf16 projection, W_e^T]
Projections: gate and up are ``I x H`` (out x in), down is ``H x I``.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace  # noqa: F401 (replace is re-exported)
from typing import Dict, Optional

import numpy as np

PROJ_VQLR = 0
PROJ_DENSE_BF16 = 1


@dataclass(frozen=True)
class LayerShape:
    """Shape of one MoE layer and of its compressed representation."""
    name: str
    H: int            # hidden size
    I: int            # expert intermediate size
    E: int            # routed experts
    k: int            # experts selected per token
    S: int = 0        # always-on shared experts (ids E..E+S-1)
    d: int = 8        # VQ block length
    K: int = 256      # code book size
    r: int = 16       # low-rank rank
    T: int = 1        # tokens in the decode batch
    router_bias: bool = False   # per-expert bias ~N(0,1) that skews routing
    # "full": gate/up/down all VQ+LR;  "paper": gate/up VQ+LR, down dense bf16;
    # "dense": all three dense bf16 (the uncompressed comparison layer)
    mode: str = "full"
    per_projection_codebook: bool = False   # False: one code book aliased by all projections
    act: str = "silu"                       # expert activation phi: "silu" (SwiGLU), "gelu_tanh" (GeGLU) or
                                            # "relu2": up-only experts, p = relu(up)^2, no gate projection
    idx12: bool = False                     # 256 < K <= 4096: indices stored as 12 bits, two to three bytes

    @property
    def idx_dtype(self):
        return np.uint8 if self.K <= 256 else np.uint16


# The workloads named by the build's configuration list.  T is the default batch.
SHAPES: Dict[str, LayerShape] = {
    "tiny": LayerShape("tiny", H=256, I=128, E=8, k=2, d=8, K=256, r=16, T=1),
    "qwen3": LayerShape("qwen3", H=2048, I=768, E=128, k=8, d=8, K=4096, r=64, T=1),
    "qwen3_b16": LayerShape("qwen3_b16", H=2048, I=768, E=128, k=8, d=8, K=4096, r=64, T=16,
                            router_bias=True),
    # the batch sizes between the two headline points (Section 5.6's batch axis)
    "qwen3_b2": LayerShape("qwen3_b2", H=2048, I=768, E=128, k=8, d=8, K=4096, r=64, T=2),
    "qwen3_b4": LayerShape("qwen3_b4", H=2048, I=768, E=128, k=8, d=8, K=4096, r=64, T=4),
    "qwen3_b8": LayerShape("qwen3_b8", H=2048, I=768, E=128, k=8, d=8, K=4096, r=64, T=8),
    "dsv2lite": LayerShape("dsv2lite", H=2048, I=1408, E=64, k=6, S=2, d=8, K=256, r=32, T=1),
    "dsv2lite_b8": LayerShape("dsv2lite_b8", H=2048, I=1408, E=64, k=6, S=2, d=8, K=256, r=32,
                              T=8),
    "mixtral": LayerShape("mixtral", H=4096, I=14336, E=8, k=2, d=8, K=4096, r=128, T=1),
    "mixtral_b4": LayerShape("mixtral_b4", H=4096, I=14336, E=8, k=2, d=8, K=4096, r=128, T=4),
    "mixtral_b16": LayerShape("mixtral_b16", H=4096, I=14336, E=8, k=2, d=8, K=4096, r=128,
                              T=16),
    # the paper's own deployed operating points (evaluation-setup table): K = 256, uint8 indices,
    # gate/up compressed, down kept in bf16 ("paper" mode), one code book per projection
    "qwen3_deployed": LayerShape("qwen3_deployed", H=2048, I=768, E=128, k=8, d=8, K=256, r=384, T=1,
                                 mode="paper", per_projection_codebook=True),
    "qwen3_deployed_b16": LayerShape("qwen3_deployed_b16", H=2048, I=768, E=128, k=8, d=8, K=256, r=384,
                                     T=16, router_bias=True, mode="paper", per_projection_codebook=True),
    "dsv2lite_deployed": LayerShape("dsv2lite_deployed", H=2048, I=1408, E=64, k=6, d=8, K=256, r=384, T=1,
                                    mode="paper", per_projection_codebook=True),
    "gemma4_deployed": LayerShape("gemma4_deployed", H=2816, I=704, E=128, k=8, d=8, K=256, r=384, T=1,
                                  mode="paper", per_projection_codebook=True, act="gelu_tanh"),
    # the d = 8 points of the storage-rate sweep (Section 5.5: K = 256, r chosen for about 3, 4 and
    # 5 bits per original weight on the Qwen3 shape; r rounded to a multiple of 8)
    "qwen3_3bit": LayerShape("qwen3_3bit", H=2048, I=768, E=128, k=8, d=8, K=256, r=248, T=1,
                             mode="paper", per_projection_codebook=True),
    "qwen3_4bit": LayerShape("qwen3_4bit", H=2048, I=768, E=128, k=8, d=8, K=256, r=376, T=1,
                             mode="paper", per_projection_codebook=True),
    "qwen3_5bit": LayerShape("qwen3_5bit", H=2048, I=768, E=128, k=8, d=8, K=256, r=504, T=1,
                             mode="paper", per_projection_codebook=True),
    # ... and its d = 4 points: the index term alone is 2 bits per weight, r = 128 / 248 / 376
    "qwen3_d4_3bit": LayerShape("qwen3_d4_3bit", H=2048, I=768, E=128, k=8, d=4, K=256, r=128, T=1,
                                mode="paper", per_projection_codebook=True),
    "qwen3_d4_4bit": LayerShape("qwen3_d4_4bit", H=2048, I=768, E=128, k=8, d=4, K=256, r=248, T=1,
                                mode="paper", per_projection_codebook=True),
    "qwen3_d4_5bit": LayerShape("qwen3_d4_5bit", H=2048, I=768, E=128, k=8, d=4, K=256, r=376, T=1,
                                mode="paper", per_projection_codebook=True),
    # the (4, 256, 256) point on the OLMoE shape: four-value code words
    # Nemotron-3-Nano-shaped layer at its deployed point (8, 256, 512): up-only ReLU^2 experts, bf16 down projection
    "nemotron_deployed": LayerShape("nemotron_deployed", H=2688, I=1856, E=128, k=6, d=8, K=256, r=512, T=1,
                                    mode="paper", per_projection_codebook=True, act="relu2"),
    # the Qwen3-shaped layer with its K = 4096 indices packed to twelve bits
    "qwen3_idx12": LayerShape("qwen3_idx12", H=2048, I=768, E=128, k=8, d=8, K=4096, r=64, T=1, idx12=True),
    "olmoe_deployed": LayerShape("olmoe_deployed", H=2048, I=1024, E=64, k=8, d=4, K=256, r=256, T=1,
                                 mode="paper", per_projection_codebook=True),
    "olmoe_deployed_b8": LayerShape("olmoe_deployed_b8", H=2048, I=1024, E=64, k=8, d=4, K=256, r=256, T=8,
                                    mode="paper", per_projection_codebook=True),
    "olmoe_deployed_b16": LayerShape("olmoe_deployed_b16", H=2048, I=1024, E=64, k=8, d=4, K=256, r=256,
                                     T=16, mode="paper", per_projection_codebook=True),
}


def shape(name: str, **overrides) -> LayerShape:
    return replace(SHAPES[name], **overrides)


# ---------------------------------------------------------------------------------------
# bf16 <-> float helpers (format conversion only)
# ---------------------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even) and return the uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# ---------------------------------------------------------------------------------------
# layer container
# ---------------------------------------------------------------------------------------
@dataclass
class Projection:
    kind: int
    out_dim: int
    in_dim: int
    codebook: Optional[np.ndarray] = None   # [K][d] bf16 bits
    idx: Optional[np.ndarray] = None        # [E+S][out][in/d] u8/u16; idx_bits == 12: packed bytes [E+S][out][in/d*3/2]
    idx_bits: int = 0                       # 12 for the packed twelve-bit encoding, else 8 * itemsize of idx
    basis: Optional[np.ndarray] = None      # [r][in] bf16 bits
    factor: Optional[np.ndarray] = None     # [E+S][out][r] bf16 bits
    dense: Optional[np.ndarray] = None      # [E+S][out][in] bf16 bits


@dataclass
class Layer:
    shape: LayerShape
    router_w: np.ndarray                    # [E][H] bf16 bits
    router_bias: Optional[np.ndarray]       # [E] f32 or None
    x: np.ndarray                           # [T][H] bf16 bits
    gate: Projection = None
    up: Projection = None
    down: Projection = None
    seed: int = 0
    notes: dict = field(default_factory=dict)


def _normal_bf16(rng: np.random.Generator, size, std: float) -> np.ndarray:
    return f32_to_bf16_bits(rng.standard_normal(size, dtype=np.float32) * np.float32(std))


def pack12(idx: np.ndarray) -> np.ndarray:
    """Twelve-bit packing of an index array whose last dimension is even: indices 2q and 2q+1 of a
    row go to bytes 3q .. 3q+2, little end first (low eight bits of the first; its high four bits
    with the low four of the second; high eight bits of the second)."""
    a = np.ascontiguousarray(idx, dtype=np.uint16)
    assert a.shape[-1] % 2 == 0 and int(a.max(initial=0)) < 4096
    lo, hi = a[..., 0::2], a[..., 1::2]
    out = np.empty(a.shape[:-1] + (a.shape[-1] // 2, 3), np.uint8)
    out[..., 0] = lo & 0xFF
    out[..., 1] = (lo >> 8) | ((hi & 0xF) << 4)
    out[..., 2] = hi >> 4
    return out.reshape(a.shape[:-1] + (a.shape[-1] // 2 * 3,))


def make_layer(shp: LayerShape, seed: int = 0) -> Layer:
    """Draw one layer.  Draw order is fixed (router, bias, tokens, code books, bases, indices,
    factors, dense matrices) so that a given (shape, seed) always yields the same bits."""
    rng = np.random.default_rng(seed)
    H, I, E, S, d, K, r, T = shp.H, shp.I, shp.E, shp.S, shp.d, shp.K, shp.r, shp.T
    n_exp = E + S
    router_w = _normal_bf16(rng, (E, H), 0.02)
    bias = rng.standard_normal(E, dtype=np.float32) if shp.router_bias else None
    x = _normal_bf16(rng, (T, H), 1.0)

    dims = {"gate": (I, H), "up": (I, H), "down": (H, I)}
    vq = {"gate": shp.mode in ("full", "paper"), "up": shp.mode in ("full", "paper"),
          "down": shp.mode == "full"}
    if shp.mode not in ("full", "paper", "dense"):
        raise ValueError(f"unknown mode {shp.mode!r}")
    names = ("up", "down") if shp.act == "relu2" else ("gate", "up", "down")     # up-only experts: nothing is drawn for a gate
    if shp.idx12 and not (256 < K <= 4096 and d == 8):
        raise ValueError("idx12 needs 256 < K <= 4096 and d == 8")

    # code books: one per layer (aliased) unless per_projection_codebook
    books = {}
    shared_book = None
    for p in names:
        if not vq[p]:
            continue
        if shp.per_projection_codebook or shared_book is None:
            book = _normal_bf16(rng, (K, d), 0.02)
            if not shp.per_projection_codebook:
                shared_book = book
        else:
            book = shared_book
        books[p] = book
    # shared bases, std in^-1/2 so that z = B x has about unit variance
    bases = {}
    for p in names:
        if vq[p] and r > 0:
            out_dim, in_dim = dims[p]
            bases[p] = _normal_bf16(rng, (r, in_dim), in_dim ** -0.5)
    # private index maps, iid uniform on [0, K)
    idxs = {}
    for p in names:
        if vq[p]:
            out_dim, in_dim = dims[p]
            idxs[p] = rng.integers(0, K, size=(n_exp, out_dim, in_dim // d),
                                   dtype=shp.idx_dtype)
    # private coefficients
    factors = {}
    for p in names:
        if vq[p] and r > 0:
            out_dim, in_dim = dims[p]
            factors[p] = _normal_bf16(rng, (n_exp, out_dim, r), 0.01)
    # dense projections
    denses = {}
    for p in names:
        if not vq[p]:
            out_dim, in_dim = dims[p]
            denses[p] = _normal_bf16(rng, (n_exp, out_dim, in_dim), 0.02)

    projs = {}
    for p in names:
        out_dim, in_dim = dims[p]
        if vq[p]:
            projs[p] = Projection(PROJ_VQLR, out_dim, in_dim, codebook=books[p],
                                  idx=pack12(idxs[p]) if shp.idx12 else idxs[p], idx_bits=12 if shp.idx12 else 0,
                                  basis=bases.get(p), factor=factors.get(p))
        else:
            projs[p] = Projection(PROJ_DENSE_BF16, out_dim, in_dim, dense=denses[p])
    return Layer(shape=shp, router_w=router_w, router_bias=bias, x=x, gate=projs.get("gate"),
                 up=projs["up"], down=projs["down"], seed=seed)


def duplicate_router_rows(layer: Layer, src: int, dst: int) -> None:
    """Make expert ``dst`` an exact routing twin of ``src`` (same router row and bias), so
    that their logits tie bit for bit under any fixed summation order."""
    layer.router_w[dst] = layer.router_w[src]
    if layer.router_bias is not None:
        layer.router_bias[dst] = layer.router_bias[src]
