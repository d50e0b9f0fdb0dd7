"""Seeded synthetic K/V streams shaped like the paper's Llama/Qwen workloads.

This module only draws random inputs.  It holds none of the eviction method's
arithmetic (no norms, anchors, scores, selection or compaction) so that the CUDA
path and the CPU oracle can both be fed from it without sharing method code.

The paper evaluates on LongBench / Math-500 prompts run through Llama-3.1-8B,
Llama-3.2-3B, Qwen2.5-7B and DeepSeek-R1-Distill models (Sec. 4 "Setup"); neither the
prompts nor the weights are available here, so the key statistics the paper
reports -- keys nearly collinear with their mean, a few large-magnitude channels
(App. C, key-norm statistics) -- are imitated by the recipes below and the shapes
(layers, KV heads, head_dim, budget N, block B) follow the named models.

Every tensor is bf16, laid out [U, rows, d] with U = n_layers * batch * n_kv_heads
independent units ordered (layer, batch, head), row = token, d = head_dim.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    batch: int
    n_kv_heads: int
    head_dim: int
    budget: int          # N: cache budget in tokens (Sec. 2.3)
    block: int           # B: tokens appended per step (Sec. 2.4)
    key_model: str       # "offset" | "outlier" | "clusters" | "drift"
    total_tokens: int    # prompt (or prompt+generation) length streamed
    seed: int

    @property
    def units(self) -> int:
        return self.n_layers * self.batch * self.n_kv_heads

    @property
    def fill_steps(self) -> int:
        """Steps that only append (cache not yet over budget)."""
        return self.budget // self.block

    @property
    def evict_steps(self) -> int:
        return (self.total_tokens - self.budget) // self.block


# BASELINE configs 1..5 (index = position in the list, seed = index - 1).
WORKLOADS = {
    # one eviction step: N=512 + one block of 128
    "single_step_n512": Workload("single_step_n512", 1, 1, 8, 128, 512, 128, "offset", 640, 0),
    # Llama-3.2-3B-shaped; 2048 + 119*128 tokens so that exactly 119 steps evict
    "llama32_3b_n2048": Workload("llama32_3b_n2048", 28, 1, 8, 128, 2048, 128, "outlier", 17280, 1),
    # Llama-3.1-8B-shaped headline config: 32K prompt, all layers in one call
    "llama31_8b_n8192": Workload("llama31_8b_n8192", 32, 1, 8, 128, 8192, 128, "outlier", 32768, 2),
    # Qwen2.5-7B-shaped, batch 8, clustered keys
    "qwen25_7b_n4096": Workload("qwen25_7b_n4096", 28, 8, 4, 128, 4096, 256, "clusters", 4096 + 32 * 256, 3),
    # decode-time eviction every 32 tokens, batch 32, drifting key mean
    "decode_b32_n8192": Workload("decode_b32_n8192", 32, 32, 8, 128, 8192, 32, "drift", 65536, 4),
}
CONFIG_ORDER = ["single_step_n512", "llama32_3b_n2048", "llama31_8b_n8192",
                "qwen25_7b_n4096", "decode_b32_n8192"]


def scaled(wl: Workload, **kw) -> Workload:
    """A smaller/larger variant of a workload (same key model and seed)."""
    return replace(wl, **kw)


def _gen(device, *keys: int) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for k in keys:
        s = (s ^ (int(k) + 0x9E3779B97F4A7C15 + ((s << 6) & 0xFFFFFFFFFFFFFFFF) + (s >> 2))) & 0xFFFFFFFFFFFFFFFF
    g.manual_seed(s & 0x7FFFFFFFFFFFFFFF)
    return g


class KVStream:
    """Stream of (new_k, new_v) blocks for all U units of a workload.

    ``next_block(B)`` returns two bf16 tensors [U, B, d]; blocks must be drawn in
    order (the "drift" model carries a running mean).  ``rank`` offsets the seed so
    that data-parallel replicas draw different sequences.
    """

    def __init__(self, wl: Workload, device="cpu", rank: int = 0):
        self.wl, self.device, self.rank = wl, torch.device(device), rank
        self.t = 0
        U, d = wl.units, wl.head_dim
        g = _gen(self.device, wl.seed, rank, 0xA11CE)
        f32 = dict(dtype=torch.float32, device=self.device)
        if wl.key_model in ("offset", "outlier", "drift"):
            # per-(unit, channel) offset shared across tokens, N(0, variance 2)
            self.offset = torch.randn(U, 1, d, generator=g, **f32) * (2.0 ** 0.5)
        if wl.key_model == "outlier":
            # 4 channels per unit carry a 10x gain
            gain = torch.ones(U, 1, d, **f32)
            idx = torch.rand(U, d, generator=g, **f32).argsort(dim=1)[:, :4]
            gain.scatter_(2, idx.unsqueeze(1), 10.0)
            self.gain = gain
        if wl.key_model == "clusters":
            # per unit: shared offset N(0,I), 64 centres = offset + N(0,I)
            off = torch.randn(U, 1, d, generator=g, **f32)
            self.centres = off + torch.randn(U, 64, d, generator=g, **f32)

    def next_block(self, B: int | None = None):
        wl = self.wl
        B = wl.block if B is None else B
        U, d = wl.units, wl.head_dim
        g = _gen(self.device, wl.seed, self.rank, 0xB10C, self.t)
        f32 = dict(dtype=torch.float32, device=self.device)
        z = torch.randn(U, B, d, generator=g, **f32)
        if wl.key_model == "offset":
            k = self.offset + z
        elif wl.key_model == "outlier":
            k = self.gain * (self.offset + z)
        elif wl.key_model == "clusters":
            cid = torch.randint(0, 64, (U, B), generator=g, device=self.device)
            centre = torch.gather(self.centres, 1, cid.unsqueeze(-1).expand(U, B, d))
            is_out = torch.rand(U, B, 1, generator=g, **f32) < 0.05
            k = torch.where(is_out, 3.0 * z, centre + 0.3 * z)
        elif wl.key_model == "drift":
            steps = 0.01 * torch.randn(U, B, d, generator=g, **f32)
            walk = self.offset + torch.cumsum(steps, dim=1)
            self.offset = walk[:, -1:, :].clone()
            k = walk + z
        else:
            raise ValueError(wl.key_model)
        v = torch.randn(U, B, d, generator=g, **f32)
        self.t += B
        return k.to(torch.bfloat16).contiguous(), v.to(torch.bfloat16).contiguous()


def prefilled_cache(wl: Workload, device="cpu", rank: int = 0, length: int | None = None):
    """Cache tensors [U, N, d] with the first ``length`` (default N) rows drawn from the
    stream, plus the stream positioned right after them."""
    length = wl.budget if length is None else length
    U, N, d = wl.units, wl.budget, wl.head_dim
    stream = KVStream(wl, device, rank)
    k_cache = torch.zeros(U, N, d, dtype=torch.bfloat16, device=device)
    v_cache = torch.zeros(U, N, d, dtype=torch.bfloat16, device=device)
    pos = 0
    while pos < length:
        b = min(wl.block, length - pos)
        k, v = stream.next_block(b)
        k_cache[:, pos:pos + b] = k
        v_cache[:, pos:pos + b] = v
        pos += b
    return k_cache, v_cache, stream
