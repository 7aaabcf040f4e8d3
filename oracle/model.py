"""Dense decoder blocks, paged KV cache and the recurrent MTP draft head, in fp64.

Target model: a generic pre-norm decoder (RMSNorm, rotary positions, grouped-query
attention, SwiGLU feed-forward).  The decoder-layer families the paper names (App. B.1)
differ in the attention projections only: one adds a bias to the query/key/value
projections (keys "bq", "bk", "bv" of a layer), one normalises every query and key head
with an RMSNorm over the head dimension before the rotary embedding (keys "qnorm",
"knorm").  A layer without those keys has neither.  Draft head (App. B.1): ONE such
decoder layer with its own KV cache; embedding table and output head are the backbone's.
Its input at position i is z_i = W_proj [RMSNorm_e(E[x_i]) ; RMSNorm_h(h_{i-1})] with a
bias-free W_proj of shape [d, 2d]: x_i the token at that position, h_{i-1} the backbone
state that produced it.

Conventions the paper leaves open (see the package docstring): the concatenation is
[norm(embedding) ; norm(hidden)]; the hidden state is the backbone's residual stream
before its final norm; the head's output goes through a head-owned RMSNorm before the
shared LM head; a head entry sits at the position of its hidden state.

Everything is written out directly: explicit-softmax attention over every key, no
blocking, no fusion.  Weights arrive as float arrays holding bf16 values.
"""
from __future__ import annotations

import numpy as np


def f64(x) -> np.ndarray:
    return np.asarray(x, dtype=np.float64)


def round_bf16(x) -> np.ndarray:
    """Nearest bf16 value, ties to even (bit arithmetic on the fp32 encoding); fp32 out."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    b = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return b.view(np.float32)


# ---- element-wise blocks -----------------------------------------------------------------

def rmsnorm(x, w, eps: float) -> np.ndarray:
    """x * rsqrt(mean(x^2) + eps) * w over the last axis."""
    x = f64(x)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * f64(w)


def silu(x) -> np.ndarray:
    x = f64(x)
    return x / (1.0 + np.exp(-x))


def rope(x, pos, base: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing: dims (i, i + hd/2) turn by pos * base^(-2i/hd).

    x: [T, H, hd]; pos: [T] integer positions.
    """
    x = f64(x)
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = base ** (-np.arange(half, dtype=np.float64) * 2.0 / hd)
    ang = f64(pos)[:, None] * inv_freq[None, :]            # [T, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def attention(q, k, v, q_pos, k_pos) -> np.ndarray:
    """Causal grouped-query attention with an explicit softmax over every key.

    q [T, n_q, hd]; k, v [S, n_kv, hd]; query t sees key s iff k_pos[s] <= q_pos[t].
    Query head h uses key/value head h // (n_q / n_kv).
    """
    q, k, v = f64(q), f64(k), f64(v)
    T, n_q, hd = q.shape
    n_kv = k.shape[1]
    g = n_q // n_kv
    visible = np.asarray(k_pos)[None, :] <= np.asarray(q_pos)[:, None]      # [T, S]
    out = np.zeros_like(q)
    for h in range(n_q):
        s = q[:, h, :] @ k[:, h // g, :].T / np.sqrt(hd)                     # [T, S]
        s = np.where(visible, s, -np.inf)
        s = s - s.max(axis=1, keepdims=True)
        e = np.exp(s)
        pr = e / e.sum(axis=1, keepdims=True)
        out[:, h, :] = pr @ v[:, h // g, :]
    return out


# ---- paged KV cache -----------------------------------------------------------------------

class PagedKV:
    """Per-sequence KV cache in fixed-size pages: pool[layer, 0|1, page, kv_head, slot, hd].

    ``page_table[b, i]`` is the physical page holding positions i*page .. (i+1)*page-1 of
    sequence b.  Writing a position that already holds an entry overwrites it.
    """

    def __init__(self, n_layers, n_kv, hd, page_table, num_pages, page_size=16):
        self.page = page_size
        self.table = np.asarray(page_table, dtype=np.int64)
        self.pool = np.zeros((n_layers, 2, num_pages, n_kv, page_size, hd), np.float64)

    def write(self, layer, b, pos, k, v):
        for t, p in enumerate(np.asarray(pos)):
            pg = self.table[b, p // self.page]
            assert pg >= 0, "position beyond the pages of this sequence"
            self.pool[layer, 0, pg, :, p % self.page, :] = k[t]
            self.pool[layer, 1, pg, :, p % self.page, :] = v[t]

    def gather(self, layer, b, n):
        """Contiguous K, V [n, n_kv, hd] of positions 0..n-1."""
        idx = np.arange(n)
        pg = self.table[b, idx // self.page]
        sl = idx % self.page
        k = self.pool[layer, 0, pg, :, sl, :]
        v = self.pool[layer, 1, pg, :, sl, :]
        return k, v


# ---- decoder layer, target forward, draft head ----------------------------------------------

def project_qkv(lw, h, cfg):
    """Query/key/value heads of normalised rows h [T, d], before the rotary embedding.

    q [T, n_q, hd], k and v [T, n_kv, hd].  Optional per-family steps (App. B.1): a bias
    on each projection; an RMSNorm over the head dimension on every query and key head.
    """
    T = h.shape[0]
    q = h @ f64(lw["wq"]).T
    k = h @ f64(lw["wk"]).T
    v = h @ f64(lw["wv"]).T
    if "bq" in lw:
        q, k, v = q + f64(lw["bq"]), k + f64(lw["bk"]), v + f64(lw["bv"])
    q = q.reshape(T, cfg.n_q_heads, cfg.head_dim)
    k = k.reshape(T, cfg.n_kv_heads, cfg.head_dim)
    v = v.reshape(T, cfg.n_kv_heads, cfg.head_dim)
    if "qnorm" in lw:
        q = rmsnorm(q, lw["qnorm"], cfg.rms_eps)
        k = rmsnorm(k, lw["knorm"], cfg.rms_eps)
    return q, k, v


def ffn_block(lw, x, cfg) -> np.ndarray:
    """The feed-forward half of a pre-norm decoder layer (App. B.1): x + W_d (silu(W_g u) * (W_u u)), u = RMSNorm(x; ln2)."""
    x = f64(x)
    h2 = rmsnorm(x, lw["ln2"], cfg.rms_eps)
    act = silu(h2 @ f64(lw["wg"]).T) * (h2 @ f64(lw["wu"]).T)
    return x + act @ f64(lw["wd"]).T


def attention_block(lw, x, pos, kv: PagedKV, layer: int, b: int, cfg) -> np.ndarray:
    """The attention half of a pre-norm decoder layer over new rows x [T, d] at positions pos, against the cache:
    x + W_o attention(...).  The rows' keys/values are written to the cache first; each row then attends every
    cached position <= its own."""
    x = f64(x)
    T = x.shape[0]
    pos = np.asarray(pos)
    h = rmsnorm(x, lw["ln1"], cfg.rms_eps)
    q, k, v = project_qkv(lw, h, cfg)
    q = rope(q, pos, cfg.rope_base)
    k = rope(k, pos, cfg.rope_base)
    kv.write(layer, b, pos, k, v)
    n = int(pos.max()) + 1
    kc, vc = kv.gather(layer, b, n)
    o = attention(q, kc, vc, pos, np.arange(n)).reshape(T, cfg.q_dim)
    return x + o @ f64(lw["wo"]).T


def decoder_layer(lw, x, pos, kv: PagedKV, layer: int, b: int, cfg) -> np.ndarray:
    """One pre-norm decoder layer over new rows x [T, d] at positions pos, against the cache."""
    return ffn_block(lw, attention_block(lw, x, pos, kv, layer, b, cfg), cfg)


def target_forward(w, tokens, pos, kv: PagedKV, b: int, cfg) -> np.ndarray:
    """Backbone over new tokens at positions pos; returns the residual stream H [T, d]
    BEFORE the final norm (the feature the draft head consumes)."""
    x = f64(w["embed"])[np.asarray(tokens)]
    for l, lw in enumerate(w["layers"]):
        x = decoder_layer(lw, x, pos, kv, l, b, cfg)
    return x


def target_logits(w, hidden, cfg) -> np.ndarray:
    """LM head on the final-normed hidden state."""
    return rmsnorm(hidden, w["final_norm"], cfg.rms_eps) @ f64(w["lm_head"]).T


def head_input(w, hidden, tokens, cfg) -> np.ndarray:
    """Input of the head's layer for pairs (hidden_i, token_i) (App. B.1): the token embedding and the hidden state, each
    through its own RMSNorm, concatenated and projected from 2d to d by a bias-free matrix.

    The two normalised inputs are concatenated [embedding ; hidden]; a head whose
    "concat" entry is "hidden_first" takes them in the opposite order (App. B.1: one
    family's native head does)."""
    hw = w["head"]
    e = f64(w["embed"])[np.asarray(tokens)]
    parts = [rmsnorm(e, hw["enorm"], cfg.rms_eps), rmsnorm(hidden, hw["hnorm"], cfg.rms_eps)]
    if hw.get("concat", "embedding_first") == "hidden_first":
        parts.reverse()
    z = np.concatenate(parts, axis=-1)
    return z @ f64(hw["proj"]).T


def head_forward(w, hidden, tokens, pos, hkv: PagedKV, b: int, cfg) -> np.ndarray:
    """Draft head over pairs (hidden_i, token_i) at positions pos; returns g [T, d], the
    head layer's residual output (its recurrent state)."""
    return decoder_layer(w["head"]["layer"], head_input(w, hidden, tokens, cfg), pos, hkv, 0, b, cfg)


def head_logits(w, g, cfg) -> np.ndarray:
    """Shared LM head on the head's own final-normed state."""
    return rmsnorm(g, w["head"]["final_norm"], cfg.rms_eps) @ f64(w["lm_head"]).T
