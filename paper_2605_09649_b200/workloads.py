"""Seeded synthetic inputs shaped like the paper's workloads.

This module only DRAWS data (random tensors, random-init projection weights and the
matrix products that turn hidden states into K/V/Q inputs).  It contains none of the
method's arithmetic: no gate, no score, no selection, no attention.  Both the CUDA
path and the CPU oracle read tensors produced here (generate once on one device and
hand the same bytes to both).

The five named workloads stand in for the shapes of the paper's settings (long-context
text decode, vision-language prompts with contiguous image blocks, multi-turn
dialogue with a persistent budget, and a long-context stress case).  They are
synthetic: hidden states are N(0,1); K/V/Q come from random-init projections; no
benchmark item, dataset record or trained weight is involved.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    kv_heads: int
    q_heads: int
    head_dim: int
    hidden: int
    batch: int
    budget_entries: int          # M_global per sequence, in entries
    kv_dtype: str                # "f32" | "bf16"
    context: int                 # prompt tokens per sequence before the decode loop
    decode_steps: int
    chunk: int                   # prefill chunk (tokens per append before an eviction)
    gate_hidden: int = 512       # d_g (Sec. 5.1)
    gate_embed: int = 64         # d_e (width of Proj's output; the paper does not state it)
    horizon: int = 2             # T - t at inference (Sec. 5.1)
    b_g: float = 18.0            # shared bias (its initial value, Sec. 5.1)
    visual_period: int = 0       # >0: every `visual_period` tokens end with `visual_len` visual tokens
    visual_len: int = 0
    turns: int = 1               # multi-turn: `turns` x (context tokens + decode_steps)

    @property
    def group(self) -> int:
        return self.q_heads // self.kv_heads

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


WORKLOADS = {
    # tiny reference: the case the oracle runs in full
    "tiny": Workload("tiny", 2, 2, 4, 64, 256, 1, 128, "f32", 512, 16, 512),
    # Llama-3-8B-shaped decode, 32K context, batch 8, 4096 tokens' worth
    "llama8b_32k": Workload("llama8b_32k", 32, 8, 32, 128, 4096, 8, 4096 * 32 * 8, "bf16", 32768, 256, 512),
    # Qwen2.5-VL-7B-shaped: 16 x (768 text + 256 visual), batch 4, 2048 tokens' worth
    "qwen_vl_16k": Workload("qwen_vl_16k", 28, 4, 28, 128, 3584, 4, 2048 * 28 * 4, "bf16", 16384, 128, 512,
                            visual_period=1024, visual_len=256),
    # multi-turn dialogue: batch 32, 8 turns x (2048 user tokens + 256 decoded)
    "multiturn": Workload("multiturn", 32, 8, 32, 128, 4096, 32, 2048 * 32 * 8, "bf16", 2048, 256, 512, turns=8),
    # long-context stress: 64 layers, 128K context, batch 1, 8192 tokens' worth
    "stress_128k": Workload("stress_128k", 64, 8, 64, 128, 5120, 1, 8192 * 64 * 8, "bf16", 131072, 64, 512),
}


def torch_dtype(kv_dtype: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[kv_dtype]


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def _mix(*parts: int) -> int:
    """Deterministic integer mix of a seed with stream identifiers."""
    s = 0x9E3779B97F4A7C15
    for p in parts:
        s = (s ^ (int(p) + 0x9E3779B97F4A7C15 + ((s << 6) & 0xFFFFFFFFFFFFFFFF) + (s >> 2))) & 0xFFFFFFFFFFFFFFFF
    return s


def gate_params(w: Workload, seed: int, device="cpu", std: float = 0.02):
    """Random-init gate weights: N(0, std) matrices, zero biases.

    Returns (per_layer, w_g) with per_layer[l] = (W1 [d_g, D], b1 [d_g], W2 [H, d_e, d_g], b2 [H, d_e]).
    """
    per_layer = []
    for l in range(w.layers):
        g = _gen(_mix(seed, 101, l), device)
        W1 = torch.randn(w.gate_hidden, w.hidden, generator=g, device=device, dtype=torch.float32) * std
        W2 = torch.randn(w.kv_heads, w.gate_embed, w.gate_hidden, generator=g, device=device, dtype=torch.float32) * std
        b1 = torch.zeros(w.gate_hidden, device=device, dtype=torch.float32)
        b2 = torch.zeros(w.kv_heads, w.gate_embed, device=device, dtype=torch.float32)
        per_layer.append((W1, b1, W2, b2))
    g = _gen(_mix(seed, 102), device)
    w_g = torch.randn(w.gate_embed, generator=g, device=device, dtype=torch.float32) * std
    return per_layer, w_g


def head_logit_offsets(w: Workload, seed: int, std: float, device="cpu") -> torch.Tensor:
    """[L, H] offsets used by the 'skewed' variant of a workload (added to b2 . w_g by the
    harness through b2): makes per-(layer, head) retention differ strongly so that pools
    become ragged.  Pure data."""
    g = _gen(_mix(seed, 103), device)
    return torch.randn(w.layers, w.kv_heads, generator=g, device=device, dtype=torch.float32) * std


class ProjectionBank:
    """Random-init q/k/v projections per layer, N(0, 1/sqrt(D)), cached in the compute dtype."""

    def __init__(self, w: Workload, seed: int, device="cpu"):
        self.w, self.seed, self.device = w, seed, device
        self._cache = {}
        self.dtype = torch.float32 if w.kv_dtype == "f32" else torch.bfloat16

    def get(self, layer: int):
        if layer not in self._cache:
            w = self.w
            g = _gen(_mix(self.seed, 201, layer), self.device)
            sc = 1.0 / math.sqrt(w.hidden)
            Wq = (torch.randn(w.hidden, w.q_heads * w.head_dim, generator=g, device=self.device) * sc).to(self.dtype)
            Wk = (torch.randn(w.hidden, w.kv_heads * w.head_dim, generator=g, device=self.device) * sc).to(self.dtype)
            Wv = (torch.randn(w.hidden, w.kv_heads * w.head_dim, generator=g, device=self.device) * sc).to(self.dtype)
            self._cache[layer] = (Wq, Wk, Wv)
        return self._cache[layer]


def is_visual(w: Workload, token_index: torch.Tensor) -> torch.Tensor:
    """Boolean mask: which absolute token indices (0-based) are visual tokens."""
    if w.visual_period <= 0:
        return torch.zeros_like(token_index, dtype=torch.bool)
    return (token_index % w.visual_period) >= (w.visual_period - w.visual_len)


def hidden_states(w: Workload, seed: int, layer: int, token_offset: int, n_tokens: int, device="cpu") -> torch.Tensor:
    """x [B, n, D] fp32 for tokens [token_offset, token_offset + n) of every sequence at `layer`.

    Text tokens: N(0,1).  Visual tokens (workloads with image blocks): 0.5*N(0,1) plus an
    offset vector N(0,1)^D shared by all tokens of the same (sequence, image block).
    """
    g = _gen(_mix(seed, 301, layer, token_offset), device)
    x = torch.randn(w.batch, n_tokens, w.hidden, generator=g, device=device, dtype=torch.float32)
    if w.visual_period > 0:
        idx = torch.arange(token_offset, token_offset + n_tokens, device=device)
        vis = is_visual(w, idx)
        if bool(vis.any()):
            blocks = (idx // w.visual_period)
            for blk in torch.unique(blocks[vis]).tolist():
                gb = _gen(_mix(seed, 302, blk), device)
                off = torch.randn(w.batch, 1, w.hidden, generator=gb, device=device, dtype=torch.float32)
                m = vis & (blocks == blk)
                x[:, m, :] = 0.5 * x[:, m, :] + off
    return x


def project_qkv(w: Workload, bank: ProjectionBank, layer: int, x: torch.Tensor):
    """(q [B,n,Hq,d], k [B,n,H,d], v [B,n,H,d]) in the workload's KV dtype from x [B,n,D]."""
    Wq, Wk, Wv = bank.get(layer)
    xb = x.to(bank.dtype)
    B, n, _ = x.shape
    q = (xb @ Wq).view(B, n, w.q_heads, w.head_dim).contiguous()
    k = (xb @ Wk).view(B, n, w.kv_heads, w.head_dim).contiguous()
    v = (xb @ Wv).view(B, n, w.kv_heads, w.head_dim).contiguous()
    return q, k, v


def selection_scores(n: int, seed: int, device="cpu", lo: float = -8.0, hi: float = 0.0) -> torch.Tensor:
    """n fp32 log-retention scores, uniform in [lo, hi] (the standalone selection sweep)."""
    g = _gen(_mix(seed, 401, n), device)
    return torch.rand(n, generator=g, device=device, dtype=torch.float32) * (hi - lo) + lo


def shard_sequences(batch: int, rank: int, world: int):
    """Contiguous, balanced split of `batch` independent sequences over `world` ranks."""
    base, rem = divmod(batch, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)
