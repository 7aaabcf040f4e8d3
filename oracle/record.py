"""The per-cycle record a speculative rollout leaves for the head update (App. D.2, "Recording in Rollout").

Five items per cycle: the backbone hidden state at the cycle's start, the K drafts, the verification
distributions, the accepted length and the absolute position of the start.  The verification distributions
are kept as the target's top-64 log-probabilities in bf16; they keep their full-vocabulary normalisation
(they are NOT renormalised over the retained set), so the mass outside the retained set is 1 - sum exp.

Ordering convention (the paper fixes none): entries sorted by logit descending, ties by token id ascending,
so the retained set is unique even when bf16 logits tie at the cut.
"""
from __future__ import annotations

import numpy as np

from .model import round_bf16

TOP = 64


def top_logprobs(logits, temperature: float = 1.0, top: int = TOP):
    """(indices[top], logprob_bf16[top]) of one row of logits; rows shorter than `top` are padded with
    index -1 and log-prob -inf."""
    x = np.asarray(logits, dtype=np.float64)
    y = x * (1.0 / float(temperature))
    m = y.max()
    lse = m + np.log(np.exp(y - m).sum())
    order = np.lexsort((np.arange(len(x)), -x))[:top]           # logit descending, then token id ascending
    idx = np.full(top, -1, np.int64)
    lp = np.full(top, -np.inf, np.float32)
    idx[:len(order)] = order
    lp[:len(order)] = round_bf16((y[order] - lse).astype(np.float32))
    return idx, lp


def cycle_record(start_hidden, drafts, target_logits, accept_len, start_pos, temperature: float = 1.0):
    """The five items of one cycle.  target_logits [K+1, V]: only the K verification rows are recorded.
    The accepted length counts the final token too (a + 1), as the paper's single integer does."""
    K = len(drafts)
    tops = [top_logprobs(target_logits[k], temperature) for k in range(K)]
    return {
        "start_hidden": np.asarray(start_hidden),
        "drafts": np.asarray(drafts, np.int64),
        "top_index": np.stack([t[0] for t in tops]) if K else np.zeros((0, TOP), np.int64),
        "top_logprob": np.stack([t[1] for t in tops]) if K else np.zeros((0, TOP), np.float32),
        "accepted": int(accept_len) + 1,
        "start_pos": int(start_pos),
    }


def sparsified_overlap(p_top_idx, p_top_logprob, q_full):
    """Overlap sum_d min(p, q) estimated from a record: the head distribution q (full vocabulary) gathered at
    the target's retained indices, plus one residual bin holding the remaining mass of each (App. D.2)."""
    keep = p_top_idx >= 0
    p_kept = np.exp(np.asarray(p_top_logprob, np.float64)[keep])
    q_kept = np.asarray(q_full, np.float64)[p_top_idx[keep]]
    return float(np.minimum(p_kept, q_kept).sum() + min(max(1.0 - p_kept.sum(), 0.0), max(1.0 - q_kept.sum(), 0.0)))
