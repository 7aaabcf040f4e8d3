"""One draft-then-verify cycle, and the state it advances (Sec. 2.2; App. E restart equations).

Per sequence the committed tokens are x[0..Len-1].  The target cache holds positions
0..Len-2: the last committed token x[Len-1] has not been fed to the target yet.  The head
consumes pairs (H_{i-1}, x_i): the target hidden state that produced token x_i, and that
token's embedding; pair i is stored in the head cache at position i-1 and its output
predicts x_{i+1}.

A cycle at context length Len with depth K:
  draft 1   the head runs over the pending pairs i = Len-n .. Len-1 (n = tokens committed by
            the previous cycle), overwriting whatever the previous chain wrote there, so
            every entry behind the boundary comes from target features (restart equations);
            the last row g_1 -> q_1 -> d_1.
  draft k   pair (g_{k-1}, d_{k-1}) at head position Len+k-3 -> g_k -> q_k -> d_k.
  verify    target forward on [x[Len-1], d_1..d_K] at positions Len-1..Len+K-1;
            p_{j+1} = softmax(logits(H_j) / T), j = 0..K.
  accept    rejection sampling (sampler.decide): a accepted drafts, token t*.
  commit    x += d_1..d_a, t*;  Len += a+1;  the rejected positions' cache entries are left
            to be overwritten;  pending pairs = (H_l, token at Len_old + l), l = 0..a.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import philox, sampler
from .model import (PagedKV, head_forward, head_logits, round_bf16, target_forward,
                    target_logits)


@dataclass
class SeqState:
    tokens: list                       # committed tokens x[0..Len-1]
    pending_hidden: np.ndarray         # [n, d] target hidden states H_{i-1} of the pending pairs
    pending_tok: list                  # [n] tokens x_i of the pending pairs (last = x[Len-1])

    @property
    def kv_len(self) -> int:           # entries in the target cache = Len - 1
        return len(self.tokens) - 1


@dataclass
class BatchState:
    seqs: list
    kv: PagedKV                        # target cache
    hkv: PagedKV                       # draft-head cache (one layer)
    step: int = 0
    history: list = field(default_factory=list)


def _maybe_round(x, on: bool):
    return round_bf16(x).astype(np.float64) if on else x


def prefill(w, cfg, prompts, page_table, num_pages, head_page_table, head_num_pages,
            temperature=1.0, seed=0, round_interface=True) -> BatchState:
    """Full causal forward over each prompt; samples the first response token (slot FINAL of
    step 0), fills the head cache from the pairs (H_{i-1}, x_i), i = 1..P-1, and leaves the
    pair (H_{P-1}, x_P) pending.  ``prompts`` is a [B, P] array or a list of B token
    sequences of different lengths (each at least one token)."""
    B = len(prompts)
    kv = PagedKV(cfg.n_layers, cfg.n_kv_heads, cfg.head_dim, page_table, num_pages, cfg.page_size)
    hkv = PagedKV(1, cfg.n_kv_heads, cfg.head_dim, head_page_table, head_num_pages, cfg.page_size)
    seqs = []
    for b in range(B):
        toks = [int(t) for t in prompts[b]]
        P = len(toks)
        H = target_forward(w, toks, np.arange(P), kv, b, cfg)
        H = _maybe_round(H, round_interface)
        logits = _maybe_round(target_logits(w, H[-1:], cfg), round_interface)
        p = sampler.softmax_probs(logits[0], temperature)
        first, _ = sampler.draw_token(p, philox.u24(seed, 0, b, philox.SLOT_FINAL))
        if P > 1:
            head_forward(w, H[:P - 1], toks[1:], np.arange(P - 1), hkv, b, cfg)
        seqs.append(SeqState(toks + [first], H[P - 1:P].copy(), [first]))
    return BatchState(seqs, kv, hkv, step=1)


def draft(w, cfg, st: BatchState, b: int, K: int, temperature: float, u24_draft,
          round_interface=True, forced=None):
    """K recurrent applications of the head; returns (d[K], draft_logits[K, V], q[K, V]).

    ``forced``: K recorded draft tokens to feed back instead of sampling (the draft-path
    reconstruction of Eq. 4: s_{k+1} = [s_k, d_k] with the recorded d_k, nothing sampled); the
    distributions q_k are then those the head assigns along that recorded path."""
    s = st.seqs[b]
    n = len(s.pending_tok)
    L1 = s.kv_len                       # = Len - 1
    d, logits_out, q_out = [], [], []
    g = head_forward(w, s.pending_hidden, s.pending_tok, np.arange(L1 - n, L1), st.hkv, b, cfg)[-1:]
    for k in range(1, K + 1):
        if k > 1:
            g = head_forward(w, g, [d[-1]], np.array([L1 + k - 2]), st.hkv, b, cfg)
        lg = _maybe_round(head_logits(w, g, cfg)[0], round_interface)
        q = sampler.softmax_probs(lg, temperature)
        tok, _ = sampler.draw_token(q, u24_draft[k - 1])
        d.append(tok if forced is None else int(forced[k - 1]))
        logits_out.append(lg)
        q_out.append(q)
    return d, np.array(logits_out), np.array(q_out)


def verify(w, cfg, st: BatchState, b: int, d, temperature: float, round_interface=True, top_p: float = 1.0):
    """Target forward over [x[Len-1], d_1..d_K]; returns (logits[K+1, V], H[K+1, d], p[K+1, V]);
    p is truncated to its top-p sets when top_p < 1."""
    s = st.seqs[b]
    toks = [s.tokens[-1]] + list(d)
    pos = np.arange(s.kv_len, s.kv_len + len(toks))
    H = _maybe_round(target_forward(w, toks, pos, st.kv, b, cfg), round_interface)
    logits = _maybe_round(target_logits(w, H, cfg), round_interface)
    return logits, H, sampler.nucleus_filter(sampler.softmax_probs(logits, temperature), top_p)


def commit(st: BatchState, b: int, d, a: int, t_star: int, H):
    """Append the accepted prefix and the final token; a+1 pairs become pending."""
    s = st.seqs[b]
    new = [int(t) for t in d[:a]] + [int(t_star)]
    s.tokens.extend(new)
    s.pending_hidden = np.array(H[:a + 1], dtype=np.float64)
    s.pending_tok = new


def spec_step(w, cfg, st: BatchState, K: int, temperature: float = 1.0, seed: int = 0,
              do_commit: bool = True, round_interface: bool = True,
              u24_draft=None, u24_accept=None, forced_draft=None, top_p: float = 1.0):
    """One cycle for every sequence.  Returns a dict of per-row outputs.  ``forced_draft`` [B, K]
    replays recorded draft tokens (see ``draft``).  ``top_p`` < 1 truncates the target's
    distributions to their nucleus before the accept test."""
    B = len(st.seqs)
    ud = philox.u24_draft(seed, st.step, B, K) if u24_draft is None else u24_draft
    ua = philox.u24_accept(seed, st.step, B, K) if u24_accept is None else u24_accept
    out = {k: [] for k in ("draft_tok", "draft_logits", "q", "target_logits", "target_hidden",
                           "p", "accept_len", "next_token", "warn")}
    for b in range(B):
        d, dl, q = draft(w, cfg, st, b, K, temperature, ud[b], round_interface,
                         None if forced_draft is None else forced_draft[b])
        tl, H, p = verify(w, cfg, st, b, d, temperature, round_interface, top_p)
        a, t_star, warn = sampler.decide(p, q, d, ua[b])
        if do_commit:
            commit(st, b, d, a, t_star, H)
        for key, val in (("draft_tok", d), ("draft_logits", dl), ("q", q), ("target_logits", tl),
                         ("target_hidden", H), ("p", p), ("accept_len", a),
                         ("next_token", t_star), ("warn", warn)):
            out[key].append(val)
    if do_commit:
        st.step += 1
    return {k: np.array(v) for k, v in out.items()}


# ---- a whole rollout: cycles until every response has ended --------------------------------------------
#
# Responses are capped (App. B.2: 8192 tokens, 16384 for one model).  A response is the token the prefill
# drew followed by the tokens each cycle commits; it ends with the first end-of-sequence token (kept) or when
# it reaches the cap; what a cycle commits beyond either is dropped.  A finished sequence sits out the remaining
# cycles with its state frozen.  A row's uniforms depend on (seed, step, row) only, so the others are unaffected.

RUNNING, HIT_EOS, HIT_CAP = 0, 1, 2


def append_committed(response: list, new_tokens, eos: int, max_new: int) -> int:
    """Append a cycle's committed tokens to ``response``; returns RUNNING, HIT_EOS or HIT_CAP."""
    if len(response) >= max_new:
        return HIT_CAP
    for t in new_tokens:
        response.append(int(t))
        if int(t) == eos:
            return HIT_EOS
        if len(response) >= max_new:
            return HIT_CAP
    return RUNNING


def rollout(w, cfg, st: BatchState, K: int, temperature: float = 1.0, seed: int = 0, max_steps: int = 1 << 30,
            eos: int = -1, max_new: int = 8192, round_interface: bool = True, top_p: float = 1.0):
    """Run cycles from a prefilled state.  Returns (responses, status[B], cycles run)."""
    B = len(st.seqs)
    responses = [[] for _ in range(B)]
    status = [append_committed(responses[b], [st.seqs[b].tokens[-1]], eos, max_new) for b in range(B)]
    steps = 0
    while steps < max_steps and any(s == RUNNING for s in status):
        ud = philox.u24_draft(seed, st.step, B, K)
        ua = philox.u24_accept(seed, st.step, B, K)
        for b in range(B):
            if status[b] != RUNNING:
                continue
            d, _, q = draft(w, cfg, st, b, K, temperature, ud[b], round_interface)
            _, H, p = verify(w, cfg, st, b, d, temperature, round_interface, top_p)
            a, t_star, _ = sampler.decide(p, q, d, ua[b])
            commit(st, b, d, a, t_star, H)
            status[b] = append_committed(responses[b], list(d[:a]) + [t_star], eos, max_new)
        st.step += 1
        steps += 1
    return responses, status, steps
