"""Seeded synthetic inputs for the BAPS attention workloads.

This module only draws random numbers and shapes them; it contains none of the method's
arithmetic, so both the CUDA tests and the CPU checker can be fed from it.  The shapes stand in
for the language-model prefill and the multi-modal (patch-token) attention workloads the paper
evaluates on: unit-Gaussian Q/K/V per head, with optional key outliers that create large score
excursions (which is what triggers the method's restarts) and an optional per-token key bias.

Draw order is always Q, K, V, then extras, from one ``torch.Generator`` seeded with ``seed``;
values are drawn in float32 on the CPU and then cast to the storage dtype.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class AttnWorkload:
    name: str
    B: int
    H: int
    Hkv: int
    S: int
    D: int
    causal: bool
    block_q: int
    block_k: int
    dtype: str = "bf16"          # "bf16" or "f32"
    outlier_frac: float = 0.0    # fraction of K rows multiplied by outlier_scale
    outlier_scale: float = 8.0
    key_bias_var: float = 0.0    # variance of a per-token additive bias on K
    seed: int = 0

    @property
    def flops(self) -> float:
        f = 4.0 * self.B * self.H * float(self.S) ** 2 * self.D
        return f / 2 if self.causal else f

    @property
    def n_query_tiles(self) -> int:
        return self.B * self.H * (self.S // self.block_q)


# The five configurations of the benchmark definition ("N(a, b)" read as mean a, variance b).
WORKLOADS = {
    "c1_single_head": AttnWorkload("c1_single_head", 1, 1, 1, 128, 64, False, 64, 64, dtype="f32"),
    "c2_llm_prefill_mha": AttnWorkload("c2_llm_prefill_mha", 1, 32, 32, 4096, 128, True, 128, 128,
                                       outlier_frac=0.01),
    "c3_llm_prefill_gqa": AttnWorkload("c3_llm_prefill_gqa", 2, 32, 8, 8192, 128, True, 128, 128),
    "c4_vit_encoder": AttnWorkload("c4_vit_encoder", 32, 16, 16, 1024, 64, False, 128, 128,
                                   key_bias_var=0.5),
    "c5_long_context": AttnWorkload("c5_long_context", 1, 32, 8, 32768, 128, True, 128, 128),
}


def make_qkv(w: AttnWorkload, device: str = "cpu"):
    """Return (q, k, v) torch tensors, q [B,H,S,D], k/v [B,Hkv,S,D], in the storage dtype."""
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed)
    q = torch.randn(w.B, w.H, w.S, w.D, generator=g, dtype=torch.float32)
    k = torch.randn(w.B, w.Hkv, w.S, w.D, generator=g, dtype=torch.float32)
    v = torch.randn(w.B, w.Hkv, w.S, w.D, generator=g, dtype=torch.float32)
    if w.outlier_frac > 0.0:
        n_out = max(1, int(round(w.outlier_frac * w.S)))
        rows = torch.randperm(w.S, generator=g)[:n_out]
        k[:, :, rows, :] *= w.outlier_scale
    if w.key_bias_var > 0.0:
        beta = torch.randn(w.B, w.Hkv, w.S, 1, generator=g, dtype=torch.float32) * (w.key_bias_var ** 0.5)
        k = k + beta
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    q, k, v = q.to(dt), k.to(dt), v.to(dt)
    if device != "cpu":
        q, k, v = q.to(device), k.to(device), v.to(device)
    return q, k, v


def small_variant(w: AttnWorkload, *, B=None, H=None, Hkv=None, S=None, seed=None) -> AttnWorkload:
    """Same recipe at a reduced size (for parity cases the CPU checker finishes in seconds)."""
    from dataclasses import replace
    kw = {}
    if B is not None: kw["B"] = B
    if H is not None: kw["H"] = H
    if Hkv is not None: kw["Hkv"] = Hkv
    if S is not None: kw["S"] = S
    if seed is not None: kw["seed"] = seed
    return replace(w, name=w.name + "_small", **kw)


def make_rising_max_qkv(S: int, H: int = 4, D: int = 128, rise_per_tile: float = 0.05, score_noise: float = 0.02,
                        v_slope: float = 0.05, block_k: int = 128, seed: int = 0, device: str = "cpu"):
    """Inputs for the accumulated-error experiment: the row maximum rises a little with every key
    tile, so that a real-valued running max moves at every tile while an integer one moves once in
    1 / rise_per_tile tiles.  Non-causal, B = 1.  In the first two coordinates a query constant
    a = 256 meets a per-tile key offset b_j (split into a coarse and a fine part so that both survive
    the bf16 cast) chosen such that the base-2 score of every key of tile j is lifted by
    j * rise_per_tile; the other coordinates are Gaussian, scaled so that the base-2 scores scatter
    by score_noise around that.  V = v_slope * j + N(0, 1/4): the output is a weighted mean of the
    tile index, which makes a drift of the weights of older tiles visible.
    Returns bf16 (q, k, v) of shapes [1, H, S, D]."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    c = 1.4426950408889634 / (D ** 0.5)                  # base-2 score = c * q . k
    sig = (score_noise / (c * (D - 2) ** 0.5)) ** 0.5
    q = torch.randn(1, H, S, D, generator=g, dtype=torch.float32) * sig
    k = torch.randn(1, H, S, D, generator=g, dtype=torch.float32) * sig
    v = torch.randn(1, H, S, D, generator=g, dtype=torch.float32) * 0.5
    a = 256.0
    tile = torch.arange(S) // block_k
    b = tile.to(torch.float64) * rise_per_tile / (a * c)
    coarse = torch.floor(b * 64.0) / 64.0
    q[..., 0] = a; q[..., 1] = a
    k[..., 0] = coarse.to(torch.float32)[None, None, :]
    k[..., 1] = (b - coarse).to(torch.float32)[None, None, :]
    v += (tile.to(torch.float32) * v_slope)[None, None, :, None]
    q, k, v = q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)
    if device != "cpu":
        q, k, v = q.to(device), k.to(device), v.to(device)
    return q, k, v


def quantize_e4m3_tiles(x: torch.Tensor, tile_rows: int = 128):
    """Input preparation for the quantised-input entry point: x [..., S, D] (any float dtype) ->
    (codes uint8 [..., S, D] holding FP8 E4M3, scales float32 [..., S / tile_rows], dequantised float32
    [..., S, D]).  One power-of-two scale per tile of tile_rows rows, the smallest that brings the
    tile's largest magnitude into E4M3's range (448); the dequantised tensor -- value(code) * scale,
    exact in float32 -- is what a reference computation is fed with."""
    xf = x.float()
    *lead, S, D = xf.shape
    t = xf.reshape(*lead, S // tile_rows, tile_rows * D)
    amax = t.abs().amax(dim=-1).clamp(min=2.0 ** -100)
    scale = torch.exp2(torch.ceil(torch.log2(amax / 448.0)))
    q = (t / scale[..., None]).to(torch.float8_e4m3fn)
    deq = (q.float() * scale[..., None]).reshape(xf.shape)
    return q.view(torch.uint8).reshape(xf.shape).contiguous(), scale.contiguous(), deq


def make_rows(rows: int, cols: int, var: float = 4.0, seed: int = 0, device: str = "cpu"):
    """fp32 logits ~ N(0, var), [rows, cols] (the standalone encode / row-softmax sweep)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    x = torch.randn(rows, cols, generator=g, dtype=torch.float32) * (var ** 0.5)
    return x.to(device) if device != "cpu" else x


def sample_tiles(w: AttnWorkload, n_random: int = 4, seed: int = 1):
    """A fixed sample of query tiles (b, h, i): first, second, middle and last tile of at least
    four heads spanning two kv groups in every batch, plus a few random ones."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    nq = w.S // w.block_q
    heads = sorted({0, min(w.H - 1, 1), w.H // 2, w.H - 1})
    picks = sorted({0, min(1, nq - 1), nq // 2, nq - 1})
    out = []
    for b in range(w.B):
        for h in heads:
            for i in picks:
                out.append((b, h, i))
    for _ in range(n_random):
        b = int(torch.randint(0, w.B, (1,), generator=g))
        h = int(torch.randint(0, w.H, (1,), generator=g))
        i = int(torch.randint(0, nq, (1,), generator=g))
        out.append((b, h, i))
    return sorted(set(out))
