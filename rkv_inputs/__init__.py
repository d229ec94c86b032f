"""Seeded synthetic KV-cache workloads shaped like the paper's distilled-reasoning models.

This module serves both the CUDA library's tests/benchmark and the CPU oracle's tests.
It draws random tensors with a given shape, value distribution and duplicate-span
structure; it holds none of the compression method's arithmetic and imports neither
the product package nor the oracle.

The paper's experiments run DeepSeek-R1-distilled Llama-8B / Qwen-14B (Section 4.1) with
B_buffer = 128, alpha = 8, lambda = 0.1; the caches below stand in for those models'
KV caches: same shapes, keys with a few large-magnitude channels, and a share of
tokens that are noisy copies of earlier spans (the redundancy the method targets).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import torch

BASE_SEED = 20250524


@dataclass(frozen=True)
class CacheSpec:
    name: str
    layers: int
    batch: int
    n_kv_heads: int
    n_q_heads: int
    head_dim: int
    budget: int
    buffer: int
    alpha: int
    lam: float
    dtype: str                 # "bf16" | "f32" | "fp8" (caches as 8-bit E4M3 codes, queries bf16)
    span: int                  # tokens per copied span
    copy_frac: float           # share of spans (tokens) that are noisy copies
    copy_sigma: float          # noise added to a copied span
    outlier_channels: int      # channels scaled by outlier_scale, drawn per (layer, KV head)
    outlier_scale: float
    single_token_copies: int = 0   # Tiny only: this many positions become noisy copies of earlier ones

    @property
    def cap(self) -> int:
        return self.budget + self.buffer

    @property
    def folded_batch(self) -> int:      # layers are folded into the leading dimension
        return self.layers * self.batch

    @property
    def head_problems(self) -> int:
        return self.folded_batch * self.n_kv_heads

    @property
    def torch_dtype(self) -> torch.dtype:
        return {"bf16": torch.bfloat16, "f32": torch.float32, "fp8": torch.float8_e4m3fn}[self.dtype]

    @property
    def query_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "fp8" else self.torch_dtype


SPECS: Dict[str, CacheSpec] = {
    # 1 layer, 1 KV head x 4 query heads, 96 cached tokens, fp32, 16 single-token noisy copies
    "tiny": CacheSpec("tiny", 1, 1, 1, 4, 128, 64, 32, 8, 0.1, "f32", 1, 0.0, 0.05, 0, 1.0, 16),
    # R1-Distill-Llama-8B cache shape, batch 1, budget 1024
    "llama8b_b1": CacheSpec("llama8b_b1", 32, 1, 8, 32, 128, 1024, 128, 8, 0.1, "bf16", 32, 0.30, 0.05, 4, 8.0),
    # same shape, batch 16, budget 4096
    "llama8b_b16": CacheSpec("llama8b_b16", 32, 16, 8, 32, 128, 4096, 128, 8, 0.1, "bf16", 32, 0.30, 0.05, 4, 8.0),
    # R1-Distill-Qwen-7B cache shape, batch 64, budget 2048, heavy redundancy
    "qwen7b_b64": CacheSpec("qwen7b_b64", 28, 64, 4, 28, 128, 2048, 128, 8, 0.1, "bf16", 64, 0.50, 0.02, 4, 8.0),
    # R1-Distill-Qwen-14B cache shape, batch 32, budget 4096 (streamed: see make_stream_block)
    "qwen14b_b32": CacheSpec("qwen14b_b32", 48, 32, 8, 40, 128, 4096, 128, 8, 0.1, "bf16", 32, 0.30, 0.05, 4, 8.0),
}
CONFIG_ORDER = ["tiny", "llama8b_b1", "llama8b_b16", "qwen7b_b64", "qwen14b_b32"]
# a multi-head-attention cache (G = 1, Eq. 1: every query head has its own KV head), shaped like a 7B model with 32
# layers x 32 heads, batch 8, budget 2048: beside the five configurations above, which are all grouped-query
SPECS["mha7b_b8"] = CacheSpec("mha7b_b8", 32, 8, 32, 32, 128, 2048, 128, 8, 0.1, "bf16", 32, 0.30, 0.05, 4, 8.0)
# the second configuration's shape at batch 16 with the caches stored as 8-bit E4M3 codes (queries stay bf16)
# a cache with 64-dimensional heads (the shape of a 1B-parameter model of the same family: 16 layers, 8 KV heads x 4
# query heads), batch 64, budget 2048
SPECS["llama1b_b64_d64"] = CacheSpec("llama1b_b64_d64", 16, 64, 8, 32, 64, 2048, 128, 8, 0.1, "bf16", 32, 0.30, 0.05, 4, 8.0)
SPECS["llama8b_b16_fp8"] = CacheSpec("llama8b_b16_fp8", 32, 16, 8, 32, 128, 4096, 128, 8, 0.1, "fp8", 32, 0.30, 0.05, 4, 8.0)


def scaled(spec: CacheSpec, *, layers: Optional[int] = None, batch: Optional[int] = None,
           name: Optional[str] = None) -> CacheSpec:
    """The same cache shape with fewer layers / sequences (for parity samples and ncu captures)."""
    from dataclasses import replace
    return replace(spec, layers=layers if layers is not None else spec.layers,
                   batch=batch if batch is not None else spec.batch,
                   name=name or f"{spec.name}[layers={layers or spec.layers},batch={batch or spec.batch}]")


@dataclass
class Workload:
    spec: CacheSpec
    k_cache: torch.Tensor      # [layers*batch, n_kv_heads, cap, d]
    v_cache: torch.Tensor      # same
    q_window: torch.Tensor     # [layers*batch, n_q_heads, alpha, d]
    seq_lens: torch.Tensor     # [layers*batch] int32
    seed: int
    extra: dict = field(default_factory=dict)


def _generator(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _outlier_scales(spec: CacheSpec, gen: torch.Generator, device) -> torch.Tensor:
    """[layers, 1, Hkv, 1, d] multipliers: outlier_channels channels per (layer, KV head) get outlier_scale."""
    scale = torch.ones(spec.layers, 1, spec.n_kv_heads, 1, spec.head_dim, device=device)
    if spec.outlier_channels > 0:
        order = torch.rand(spec.layers, spec.n_kv_heads, spec.head_dim, generator=gen, device=device).argsort(-1)
        chosen = order[..., :spec.outlier_channels]
        flat = scale.view(spec.layers, spec.n_kv_heads, spec.head_dim)
        flat.scatter_(-1, chosen, spec.outlier_scale)
    return scale


def _copy_spans(k: torch.Tensor, spec: CacheSpec, gen: torch.Generator, first_span: int = 1) -> None:
    """Overwrite a share of spans, per folded sequence, with an earlier span plus N(0, sigma) noise.

    k: [Bf, H, T, d] float32 (modified in place).  Spans first_span.. are candidates; exactly
    floor(copy_frac * (#candidate spans)) of them, chosen without replacement per sequence, become
    copies.  Spans are visited in ascending order, so a source that is itself a copy is final when read.
    """
    Bf, H, T, d = k.shape
    n_spans = T // spec.span
    cand = n_spans - first_span
    n_copy = int(spec.copy_frac * cand)
    if n_copy <= 0:
        return
    dev = k.device
    rank = torch.rand(Bf, cand, generator=gen, device=dev).argsort(-1).argsort(-1)
    is_copy = rank < n_copy                                   # [Bf, cand]
    src_u = torch.rand(Bf, cand, generator=gen, device=dev)
    for c in range(cand):
        s = first_span + c
        rows = is_copy[:, c].nonzero().flatten()
        if rows.numel() == 0:
            continue
        src = (src_u[rows, c] * s).long().clamp_(max=s - 1)  # uniform over earlier spans
        tok = src[:, None] * spec.span + torch.arange(spec.span, device=dev)[None, :]   # [r, span]
        block = k[rows[:, None], :, tok, :]                   # [r, span, H, d]
        noise = torch.randn(block.shape, generator=gen, device=dev) * spec.copy_sigma
        dst = s * spec.span + torch.arange(spec.span, device=dev)
        k[rows[:, None], :, dst[None, :], :] = block + noise


def make_workload(spec: CacheSpec, device="cpu", seed: Optional[int] = None,
                  seq_lens: Optional[torch.Tensor] = None) -> Workload:
    """Draw K, V, Q for one firing of the compression step with every cache full (L = budget + buffer),
    unless seq_lens is given.  Values are rounded to the spec's dtype once, at the end."""
    if seed is None:
        seed = BASE_SEED + (CONFIG_ORDER.index(spec.name) + 1 if spec.name in CONFIG_ORDER else 0)
    dev = torch.device(device)
    gen = _generator(dev, seed)
    Bf, H, Hq, cap, d = spec.folded_batch, spec.n_kv_heads, spec.n_q_heads, spec.cap, spec.head_dim

    k = torch.randn(spec.layers, spec.batch, H, cap, d, generator=gen, device=dev)
    k *= _outlier_scales(spec, gen, dev)
    k = k.view(Bf, H, cap, d)
    _copy_spans(k, spec, gen)
    if spec.single_token_copies > 0:
        # distinct positions p in [1, cap) become K[s_p] + noise with s_p uniform in [0, p)
        pos = (torch.rand(Bf, H, cap - 1, generator=gen, device=dev).argsort(-1)[..., :spec.single_token_copies] + 1)
        pos, _ = pos.sort(-1)
        u = torch.rand(pos.shape, generator=gen, device=dev)
        for t in range(spec.single_token_copies):
            p = pos[..., t]                                   # [Bf, H]
            s = (u[..., t] * p).long().clamp_(min=0)
            s = torch.minimum(s, p - 1)
            bi = torch.arange(Bf, device=dev)[:, None].expand(Bf, H)
            hi = torch.arange(H, device=dev)[None, :].expand(Bf, H)
            noise = torch.randn(Bf, H, d, generator=gen, device=dev) * spec.copy_sigma
            k[bi, hi, p] = k[bi, hi, s] + noise
    v = torch.randn(Bf, H, cap, d, generator=gen, device=dev)
    q = torch.randn(Bf, Hq, spec.alpha, d, generator=gen, device=dev)
    dt = spec.torch_dtype
    if seq_lens is None:
        seq_lens = torch.full((Bf,), cap, dtype=torch.int32, device=dev)
    else:
        seq_lens = seq_lens.to(device=dev, dtype=torch.int32)
        assert seq_lens.shape == (Bf,)
    return Workload(spec, k.to(dt).contiguous(), v.to(dt).contiguous(), q.to(spec.query_dtype).contiguous(), seq_lens, seed)


def make_stream_block(spec: CacheSpec, k_cache: torch.Tensor, v_cache: torch.Tensor, seq_lens: torch.Tensor,
                      gen: torch.Generator, scale: torch.Tensor) -> torch.Tensor:
    """Append one buffer's worth (spec.buffer tokens) of new K/V rows to every head's cache in place and
    return fresh observation queries.  A share copy_frac of the new spans are noisy copies of a span taken
    uniformly from the rows currently cached for that sequence.  seq_lens is advanced by spec.buffer.
    `scale` is the [layers, 1, Hkv, 1, d] outlier multiplier from stream_state()."""
    Bf, H, cap, d = k_cache.shape
    dev = k_cache.device
    nb, sp = spec.buffer, spec.span
    new_k = torch.randn(spec.layers, spec.batch, H, nb, d, generator=gen, device=dev) * scale
    new_k = new_k.view(Bf, H, nb, d)
    L = seq_lens.long()
    n_sp = nb // sp
    is_copy = torch.rand(Bf, n_sp, generator=gen, device=dev) < spec.copy_frac
    src_u = torch.rand(Bf, n_sp, generator=gen, device=dev)
    ar = torch.arange(sp, device=dev)
    for s in range(n_sp):
        rows = (is_copy[:, s] & (L >= sp)).nonzero().flatten()
        if rows.numel() == 0:
            continue
        start = (src_u[rows, s] * (L[rows] - sp + 1).float()).long()
        start = torch.minimum(start, L[rows] - sp).clamp_(min=0)
        tok = start[:, None] + ar[None, :]
        block = k_cache[rows[:, None], :, tok, :].float()
        noise = torch.randn(block.shape, generator=gen, device=dev) * spec.copy_sigma
        new_k[rows, :, s * sp:(s + 1) * sp, :] = (block + noise).permute(0, 2, 1, 3)
    new_v = torch.randn(Bf, H, nb, d, generator=gen, device=dev)
    pos = L[:, None] + torch.arange(nb, device=dev)[None, :]              # [Bf, nb]
    assert int(pos.max()) < cap, "append would overflow the cache"
    bi = torch.arange(Bf, device=dev)[:, None].expand(Bf, nb)
    k_cache[bi, :, pos, :] = new_k.to(k_cache.dtype).permute(0, 2, 1, 3)
    v_cache[bi, :, pos, :] = new_v.to(v_cache.dtype).permute(0, 2, 1, 3)
    seq_lens += nb
    return torch.randn(Bf, spec.n_q_heads, spec.alpha, d, generator=gen, device=dev).to(spec.query_dtype)


def stream_state(spec: CacheSpec, device="cpu", seed: Optional[int] = None):
    """Empty caches, zero lengths, the generator and the outlier multipliers for a streamed workload."""
    if seed is None:
        seed = BASE_SEED + 5
    dev = torch.device(device)
    gen = _generator(dev, seed)
    Bf, H, cap, d = spec.folded_batch, spec.n_kv_heads, spec.cap, spec.head_dim
    k = torch.zeros(Bf, H, cap, d, dtype=spec.torch_dtype, device=dev)
    v = torch.zeros(Bf, H, cap, d, dtype=spec.torch_dtype, device=dev)
    seq = torch.zeros(Bf, dtype=torch.int32, device=dev)
    scale = _outlier_scales(spec, gen, dev)
    return k, v, seq, gen, scale
