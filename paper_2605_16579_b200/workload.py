"""Seeded synthetic inputs shaped like the paper's autoregressive video-diffusion workload.

This module only draws random numbers and builds lookup tables that the layer takes as
INPUTS (Q, K, V, gate logits, feature-map weights, rotary tables).  It contains none of
the layer's arithmetic, so both the CUDA path and the CPU oracle may be fed from it.

Geometry: a 832x480 video gives 30x52 = 1560 latent tokens per frame; an autoregressive
block is one frame (1560 tokens) or three (4680); the 1.3B base model has 12 heads of
dimension 128, the wider stand-in 40 heads.  Values are Gaussian as the configurations
state; combine-gate logits are N(0, 0.1) so that sigmoid(g) stays in the 0.45-0.55 band
the paper reports for learned gates; decay logits are one per (stream, head) per block.
All draws come from a CPU ``torch.Generator`` so that the same bytes are available with
or without a GPU.  bf16 tensors are drawn in fp32 and rounded to nearest-even.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    cfg_id: int
    B: int
    H: int
    D: int
    L: int
    blocks: int
    steps: int
    dtype: str          # "fp32" | "bf16": dtype of Q, K, V, O and of the feature-map weights
    qkv_std: float      # std of Q, K, V
    per_head_scale: bool  # extra per (tensor, head) scale ~U(0.3, 1.5), drawn once per run
    decay_mean: float   # decay logits a[b, h] ~ N(mean, std), redrawn every block
    decay_std: float

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "fp32" else 2


CONFIGS = {
    "tiny": Config("tiny", 1, 1, 2, 64, 256, 4, 2, "fp32", 1.0, False, 2.0, 0.5),
    "small": Config("small", 2, 1, 12, 128, 1560, 8, 4, "bf16", 0.5, False, 3.0, 0.5),
    "chunked": Config("chunked", 3, 1, 12, 128, 4680, 16, 4, "bf16", 1.0, True, 3.0, 0.5),
    "batched": Config("batched", 4, 8, 12, 128, 4680, 32, 4, "bf16", 1.0, False, 3.0, 1.0),
    "long": Config("long", 5, 1, 40, 128, 4680, 120, 4, "bf16", 1.0, False, 3.0, 0.5),
}

COMMIT_STEP = 99  # the "step" index that seeds a block's clean-pass inputs


def custom(name="custom", B=1, H=2, D=64, L=100, blocks=2, steps=2, dtype="fp32",
           qkv_std=1.0, per_head_scale=False, decay_mean=3.0, decay_std=0.5, cfg_id=9):
    """A configuration of arbitrary shape (ragged tails, edge cases)."""
    return Config(name, cfg_id, B, H, D, L, blocks, steps, dtype, qkv_std, per_head_scale,
                  decay_mean, decay_std)


def _gen(cfg: Config, block: int, step: int, salt: int = 0) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(cfg.cfg_id * 10_000_000 + block * 1000 + step * 10 + salt)
    return g


def _head_scales(cfg: Config) -> torch.Tensor:
    """[3, H] scale per tensor in (q, k, v) and head; ones unless the config asks for them."""
    if not cfg.per_head_scale:
        return torch.ones(3, cfg.H)
    g = torch.Generator(device="cpu")
    g.manual_seed(cfg.cfg_id * 10_000_000 + 7_777_777)
    return 0.3 + 1.2 * torch.rand(3, cfg.H, generator=g)


def _qkv(cfg: Config, gen: torch.Generator, which: int) -> torch.Tensor:
    x = torch.randn(cfg.B, cfg.L, cfg.H, cfg.D, generator=gen, dtype=torch.float32)
    x *= cfg.qkv_std
    if cfg.per_head_scale:
        x *= _head_scales(cfg)[which].view(1, 1, cfg.H, 1)
    return x.to(cfg.torch_dtype)


def step_inputs(cfg: Config, block: int, step: int):
    """Q, K, V [B, L, H, D] in the config's dtype and combine-gate logits g [B, L, H] fp32."""
    gen = _gen(cfg, block, step)
    q = _qkv(cfg, gen, 0)
    k = _qkv(cfg, gen, 1)
    v = _qkv(cfg, gen, 2)
    g = 0.1 * torch.randn(cfg.B, cfg.L, cfg.H, generator=gen, dtype=torch.float32)
    return q, k, v, g


def commit_inputs(cfg: Config, block: int):
    """Clean-pass K, V [B, L, H, D] and decay logits a [B, H] fp32 for one block."""
    gen = _gen(cfg, block, COMMIT_STEP)
    kc = _qkv(cfg, gen, 1)
    vc = _qkv(cfg, gen, 2)
    a = cfg.decay_mean + cfg.decay_std * torch.randn(cfg.B, cfg.H, generator=gen,
                                                     dtype=torch.float32)
    return kc, vc, a


def beta_logits(cfg: Config, block: int, mean: float = -3.0, std: float = 1.0):
    """Learning-rate logits [B, L, H] fp32 for the delta-rule commit of one block.

    The default mean keeps sigmoid(beta) near 0.05: with L >> D tokens applied against the same
    old state, larger rates make the block-level step overshoot.
    """
    gen = _gen(cfg, block, COMMIT_STEP, salt=7)
    return mean + std * torch.randn(cfg.B, cfg.L, cfg.H, generator=gen, dtype=torch.float32)


def token_gate_logits(cfg: Config, block: int, alpha_mean: float = 7.0, beta_mean: float = 0.0):
    """Per-token forget-gate and learning-rate logits, each [B, L, H] fp32, for the token-sequential
    commit of one block.  The forget gates sit near 1 (sigmoid(7) = 0.9991) so that a block of a
    few thousand tokens does not erase the state."""
    gen = _gen(cfg, block, COMMIT_STEP, salt=8)
    alpha = alpha_mean + torch.randn(cfg.B, cfg.L, cfg.H, generator=gen, dtype=torch.float32)
    beta = beta_mean + torch.randn(cfg.B, cfg.L, cfg.H, generator=gen, dtype=torch.float32)
    return alpha, beta


def feature_weights(cfg: Config):
    """W_phi_q, W_phi_k, W_phi_v, each [H, D, D] (in, out) = I + 0.02 N(0, 1), config dtype."""
    gen = _gen(cfg, 0, 0, salt=5)
    eye = torch.eye(cfg.D, dtype=torch.float32).expand(cfg.H, cfg.D, cfg.D)
    ws = []
    for _ in range(3):
        w = eye + 0.02 * torch.randn(cfg.H, cfg.D, cfg.D, generator=gen, dtype=torch.float32)
        ws.append(w.to(cfg.torch_dtype).contiguous())
    return tuple(ws)


def rope_tables(L: int, D: int, base: float = 10000.0):
    """cos, sin [L, D/2] fp32 for 1-D positions 0..L-1 and frequencies base^(-2m/D).

    A structural stand-in for the video model's 3-D rotary embedding: the layer takes the
    tables as inputs and does not care how the angles were chosen.
    """
    m = torch.arange(D // 2, dtype=torch.float64)
    freq = torch.exp(-math.log(base) * 2.0 * m / D)
    ang = torch.arange(L, dtype=torch.float64).view(L, 1) * freq.view(1, D // 2)
    return ang.cos().float().contiguous(), ang.sin().float().contiguous()


def sample_units(cfg: Config, heads_per_stream: int = 3):
    """Seeded (b, h) pairs for parity at full size: per stream head 0, the last head and randomly
    drawn heads from the middle of the grid, up to ``heads_per_stream`` (fixed for a whole run, so
    that a checker can follow their states from the first block to the last)."""
    gen = _gen(cfg, 0, 0, salt=4)
    out = []
    for b in range(cfg.B):
        heads = {0, cfg.H - 1}
        while len(heads) < min(heads_per_stream, cfg.H):
            heads.add(int(torch.randint(0, cfg.H, (1,), generator=gen)))
        out.extend((b, h) for h in sorted(heads))
    return out


def sample_rows(cfg: Config, block: int, step: int, heads_per_stream: int = 2,
                rows_per_head: int = 64, tile: int = 128, units=None):
    """Seeded (b, h, i) triples for sampled parity at full size.

    Units: ``units`` if given, else per stream head 0, the last head and random others up to
    ``heads_per_stream``; per unit: rows 0, tile-1, tile, the last row of the last full tile, every
    row of the ragged tail tile (or the last 8 rows when L is a multiple of the tile) and random
    rows up to ``rows_per_head``.
    """
    gen = _gen(cfg, block, step, salt=3)
    if units is None:
        units = []
        for b in range(cfg.B):
            heads = {0, cfg.H - 1}
            while len(heads) < min(heads_per_stream, cfg.H):
                heads.add(int(torch.randint(0, cfg.H, (1,), generator=gen)))
            units.extend((b, h) for h in sorted(heads))
    out = []
    for b, h in units:
        full = (cfg.L // tile) * tile
        rows = {0, min(tile - 1, cfg.L - 1), min(tile, cfg.L - 1), max(full - 1, 0)}
        tail = range(full, cfg.L) if full < cfg.L else range(max(cfg.L - 8, 0), cfg.L)
        rows.update(tail)
        while len(rows) < min(rows_per_head + len(tail), cfg.L):
            rows.add(int(torch.randint(0, cfg.L, (1,), generator=gen)))
        out.extend((b, h, i) for i in sorted(rows))
    return out
