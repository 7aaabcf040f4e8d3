"""Seeded workload recipes: ragged KV lengths, fragmented page tables, logits, prompts.

These stand in for the paper's RL rollout batches (64 prompts x 8 responses of up
to 8k-16k tokens on 4B-7B models): only shapes, length mixes and value
distributions matter for the cost of a speculative step, not token content.
"""
from __future__ import annotations

import numpy as np

from .weights import bf16_round


def kv_lengths_uniform(batch: int, lo: int, hi: int, seed: int = 3) -> np.ndarray:
    """Committed-context lengths drawn uniformly from {lo..hi}."""
    rng = np.random.Generator(np.random.Philox(seed))
    return rng.integers(lo, hi + 1, size=batch, dtype=np.int64).astype(np.int32)


def kv_lengths_lognormal(batch: int, median: int = 4096, sigma: float = 0.7,
                         lo: int = 256, hi: int = 32768, seed: int = 3) -> np.ndarray:
    """Long-tail lengths: round(exp(N(ln median, sigma))) clipped to [lo, hi]."""
    rng = np.random.Generator(np.random.Philox(seed))
    x = np.exp(rng.normal(np.log(median), sigma, size=batch))
    return np.clip(np.rint(x), lo, hi).astype(np.int32)


def make_page_tables(capacity_tokens: np.ndarray, page_size: int = 16, seed: int = 7,
                     slack_pages: int = 0):
    """Fragmented page tables: the physical pool is a seeded random permutation.

    ``capacity_tokens[b]`` is the number of token slots row ``b`` must be able to
    hold.  Returns ``(table[B, max_pages] int32, num_pages)``; unused entries are -1;
    no physical page is shared between rows.
    """
    capacity_tokens = np.asarray(capacity_tokens, dtype=np.int64)
    pages = (capacity_tokens + page_size - 1) // page_size
    total = int(pages.sum()) + slack_pages
    rng = np.random.Generator(np.random.Philox(seed))
    perm = rng.permutation(total).astype(np.int32)
    max_pages = int(pages.max()) if len(pages) else 0
    table = np.full((len(pages), max_pages), -1, np.int32)
    off = 0
    for b, n in enumerate(pages):
        table[b, :n] = perm[off:off + n]
        off += int(n)
    return table, total


def sampler_only_logits(batch: int, k: int, vocab: int, sigma: float = 0.908,
                        logit_std: float = 3.0, seed: int = 4):
    """Sampler-only inputs: target logits ~ N(0, logit_std) for k+1 positions and draft
    logits = target + N(0, sigma) for the first k positions, both rounded to bf16.

    Returns ``(target[B, k+1, V], draft[B, k, V])`` as float32 arrays of bf16 values.
    """
    rng = np.random.Generator(np.random.Philox(seed))
    tgt = rng.standard_normal((batch, k + 1, vocab), dtype=np.float32) * np.float32(logit_std)
    noise = rng.standard_normal((batch, k, vocab), dtype=np.float32) * np.float32(sigma)
    drf = tgt[:, :k, :] + noise
    return bf16_round(tgt), bf16_round(drf)


def random_prompts(batch: int, prompt_len: int, vocab: int, seed: int = 1) -> np.ndarray:
    """Prompt token ids uniform in [0, vocab)."""
    rng = np.random.Generator(np.random.Philox(seed))
    return rng.integers(0, vocab, size=(batch, prompt_len), dtype=np.int64).astype(np.int32)


def random_u24(shape, seed: int = 6) -> np.ndarray:
    """Explicit 24-bit uniforms (for callers that bypass the counter-based generator)."""
    rng = np.random.Generator(np.random.Philox(seed))
    return rng.integers(0, 1 << 24, size=shape, dtype=np.int64).astype(np.uint32)
