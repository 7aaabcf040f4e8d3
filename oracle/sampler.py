"""Speculative rejection sampling of one draft-then-verify cycle (Sec. 2.2, Eq. 1).

The rule: draft token d_k is accepted with probability min(1, p_k(d_k)/q_k(d_k));
at the first rejection a replacement is drawn from the corrected distribution
norm(max(0, p - q)); if all K drafts are accepted a bonus token is drawn from
p_{K+1}.  The committed tokens are then distributed exactly as the target's own
autoregressive samples.

To make the outcome a single-valued function of (p, q, d, uniforms) the rule is
stated on fp32 probabilities and 24-bit uniforms u = u24 * 2^-24:

* accept test   p[d] >= q[d]  or  fl32(u * q[d]) < p[d]        (one fp32 multiply)
* a draw from weights r >= 0 goes through integers:  w[v] = trunc(r[v] * 2^44),
  W = sum w (64-bit, order-free), t = floor(u24 * W / 2^24), token = the first v
  whose inclusive prefix sum exceeds t.

Quantising to 2^-44 drops at most V * 2^-44 of mass, far below fp32 softmax error.
"""
from __future__ import annotations

import numpy as np

_SCALE = np.float32(2.0 ** 44)
_INV24 = np.float32(2.0 ** -24)

WARN_ZERO_RESIDUAL = 1      # residual mass underflowed: drew from p instead
WARN_ZERO_MASS = 2          # even p quantised to zero: took argmax


def softmax_probs(logits, temperature: float = 1.0) -> np.ndarray:
    """softmax(logits / T) along the last axis, computed in fp64, returned as fp32."""
    x = np.asarray(logits, dtype=np.float64) * (1.0 / float(temperature))
    x = x - x.max(axis=-1, keepdims=True)
    e = np.exp(x)
    return (e / e.sum(axis=-1, keepdims=True)).astype(np.float32)


def integer_weights(r: np.ndarray) -> np.ndarray:
    """w[v] = trunc(r[v] * 2^44) for r[v] > 0, else 0 (r fp32, result uint64)."""
    r = np.asarray(r, dtype=np.float32)
    scaled = r * _SCALE                     # exact: power-of-two scaling
    return np.where(r > 0, scaled, np.float32(0)).astype(np.uint64)


def icdf_draw(r: np.ndarray, u24: int):
    """Draw a token from weights ``r`` (fp32, need not be normalised) with uniform ``u24``.

    Returns (token, W).  W == 0 means there was no mass; token is then -1.
    """
    w = integer_weights(r)
    cs = np.cumsum(w, dtype=np.uint64)
    W = int(cs[-1])
    if W == 0:
        return -1, 0
    t = (int(u24) * W) >> 24                # 0 <= t <= W-1 because u24 < 2^24
    tok = int(np.searchsorted(cs, np.uint64(t), side="right"))
    return tok, W


def draw_token(q: np.ndarray, u24: int):
    """Sample one token from the fp32 distribution ``q``; returns (token, warn)."""
    tok, W = icdf_draw(q, u24)
    if W == 0:
        return int(np.argmax(q)), WARN_ZERO_MASS
    return tok, 0


def accept_test(p_d: np.float32, q_d: np.float32, u24: int) -> bool:
    """Accept with probability min(1, p/q) (Eq. 1), decided in fp32."""
    p_d = np.float32(p_d)
    q_d = np.float32(q_d)
    if p_d >= q_d:
        return True
    u = np.float32(int(u24)) * _INV24       # exact
    return bool(np.float32(u * q_d) < p_d)


def decide(p: np.ndarray, q: np.ndarray, d, u24s):
    """The decision function of one cycle.

    p: fp32 [K+1, V] target distributions p_1..p_{K+1};  q: fp32 [K, V] head
    distributions;  d: K draft tokens;  u24s: K accept uniforms then the final one.
    Returns (a, next_token, warn): a = number of accepted drafts in 0..K,
    next_token = the replacement (a < K) or the bonus token (a == K).
    """
    p = np.asarray(p, dtype=np.float32)
    K = p.shape[0] - 1
    q = np.asarray(q, dtype=np.float32).reshape(K, p.shape[1])
    a = 0
    while a < K and accept_test(p[a, d[a]], q[a, d[a]], u24s[a]):
        a += 1
    warn = 0
    if a < K:
        r = p[a] - q[a]                     # fp32 subtraction, one rounding
        tok, W = icdf_draw(r, u24s[K])
        if W == 0:
            warn |= WARN_ZERO_RESIDUAL
            tok, W = icdf_draw(p[a], u24s[K])
    else:
        tok, W = icdf_draw(p[K], u24s[K])
    if W == 0:
        warn |= WARN_ZERO_MASS
        tok = int(np.argmax(p[a]))
    return a, tok, warn


def accept_batch(target_logits, draft_logits, draft_tok, u24s, temperature: float = 1.0, top_p: float = 1.0):
    """Rows of a batch through softmax (+ top-p truncation of the target rows) + decide.

    target_logits [B, K+1, V], draft_logits [B, K, V], draft_tok [B, K], u24s [B, K+1].
    Returns (accept_len[B], next_token[B], warn[B]).
    """
    B = len(target_logits)
    a_out = np.zeros(B, np.int32)
    t_out = np.zeros(B, np.int32)
    w_out = np.zeros(B, np.int32)
    for b in range(B):
        p = nucleus_filter(softmax_probs(target_logits[b], temperature), top_p)
        q = softmax_probs(draft_logits[b], temperature)
        a_out[b], t_out[b], w_out[b] = decide(p, q, draft_tok[b], u24s[b])
    return a_out, t_out, w_out


# ---- nucleus (top-p) truncation of the target distribution ---------------------------------
#
# The paper's evaluation samples with top-p 0.7 (its rollouts with top-p 1, i.e. none).  The
# truncation is applied to the distribution whose samples the cycle must reproduce - the
# target's p_1..p_{K+1}; the head's q is left as it is (the accept rule is exact for any q).
# Stated so that it is single-valued whatever order the masses are added in: with integer
# weights w = trunc(r * 2^44), W = sum w and tp24 = round(top_p * 2^24), token v is kept iff
# w[v] > 0 and  (sum of w over tokens with r strictly larger than r[v]) * 2^24 < tp24 * W.
# That is the textbook rule (sort by probability, keep tokens while the mass before them is
# below top_p) with every member of a tie at the cut kept.

def nucleus_keep(r, top_p: float) -> np.ndarray:
    """Boolean mask of the top-p set of non-negative weights r (fp32, any normalisation)."""
    if not (0.0 < float(top_p) <= 1.0):
        raise ValueError("top_p must be in (0, 1]")
    r = np.asarray(r, dtype=np.float32)
    w = integer_weights(r)
    tp24 = int(round(float(np.float32(top_p)) * (1 << 24)))
    W = int(w.sum(dtype=np.uint64))
    order = np.argsort(-r, kind="stable")
    keep = np.zeros(r.shape, bool)
    above = 0                       # weight of the tokens strictly larger than the current tie group
    i = 0
    while i < len(order):
        j = i
        group = 0
        while j < len(order) and r[order[j]] == r[order[i]]:
            group += int(w[order[j]])
            j += 1
        if (above << 24) < tp24 * W:
            for t in order[i:j]:
                keep[t] = w[t] > 0
        above += group
        i = j
    return keep


def nucleus_filter(p, top_p: float) -> np.ndarray:
    """Rows of p [..., V] truncated to their top-p sets and renormalised (fp64 division), fp32 out."""
    p = np.asarray(p, dtype=np.float32)
    if float(top_p) >= 1.0:
        return p
    flat = p.reshape(-1, p.shape[-1])
    out = np.zeros_like(flat)
    for i, row in enumerate(flat):
        kept = np.where(nucleus_keep(row, top_p), row.astype(np.float64), 0.0)
        out[i] = (kept / kept.sum()).astype(np.float32)
    return out.reshape(p.shape)


# ---- closed forms used as pins (Eq. 5 and Eq. 6) ---------------------------------------

def acceptance_probability(p, q) -> float:
    """alpha = sum_d min(p(d), q(d)) = 1 - TV(p, q)   (Eq. 5)."""
    return float(np.minimum(np.asarray(p, np.float64), np.asarray(q, np.float64)).sum())


def expected_accepted_length(alphas) -> float:
    """sum_{l=1..K} prod_{i<=l} alpha_i   (Eq. 6, context-free acceptance rates)."""
    return float(np.cumprod(np.asarray(alphas, np.float64)).sum())


# ---- many draws against fixed distributions (statistical pins) ---------------------------

def icdf_draw_many(r: np.ndarray, u24s: np.ndarray) -> np.ndarray:
    """``icdf_draw`` for an array of uniforms against one weight vector.

    floor(u24 * W / 2^24) is formed without 128-bit integers by splitting W = Wh * 2^24 + Wl:
    the product's first part is a multiple of 2^24, so the quotient is u24*Wh + (u24*Wl >> 24).
    """
    w = integer_weights(r)
    cs = np.cumsum(w, dtype=np.uint64)
    W = int(cs[-1])
    if W == 0:
        return np.full(len(u24s), -1, np.int64)
    u = np.asarray(u24s, dtype=np.uint64)
    t = u * np.uint64(W >> 24) + ((u * np.uint64(W & 0xFFFFFF)) >> np.uint64(24))
    return np.searchsorted(cs, t, side="right").astype(np.int64)


def decide_many(p: np.ndarray, q: np.ndarray, d: np.ndarray, u24s: np.ndarray):
    """``decide`` for N independent cycles that share context-free tables p [K+1, V], q [K, V].

    d [N, K] draft tokens, u24s [N, K+1].  Returns (a[N], next_token[N]).  Rows whose residual
    or target mass quantises to zero are not handled here (use ``decide``).
    """
    p = np.asarray(p, dtype=np.float32)
    K = p.shape[0] - 1
    q = np.asarray(q, dtype=np.float32).reshape(K, p.shape[1])
    N = len(u24s)
    a = np.zeros(N, np.int64)
    alive = np.ones(N, bool)
    for k in range(K):
        pd, qd = p[k, d[:, k]], q[k, d[:, k]]
        u = u24s[:, k].astype(np.float32) * _INV24
        ok = (pd >= qd) | ((u * qd).astype(np.float32) < pd)
        alive &= ok
        a += alive
    tok = np.zeros(N, np.int64)
    for j in range(K + 1):
        rows = np.nonzero(a == j)[0]
        if len(rows) == 0:
            continue
        r = p[j] - q[j] if j < K else p[K]
        tok[rows] = icdf_draw_many(r, u24s[rows, K])
    return a, tok
