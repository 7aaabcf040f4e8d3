"""Forward pass of the draft-head update: draft-path reconstruction and the acceptance objective
(Sec. 3.2 Eq. 4; Sec. 3.3 Eq. 5-7; Sec. 3.4 Eq. 8-9; App. D.2-D.3).  Test infrastructure only.

Reconstruction.  A recorded cycle r started at context length Len (its record's start position) with the
committed tokens x[0..Len-1].  The head's chain is replayed on recorded inputs: its cache is rebuilt from
the recorded pairs (H_{i-1}, x_i), i = 1..Len-1 (the rollout-time target hidden states and token ids),
restricted to the committed prefix; the first application's output at head position Len-2 is the state
g_1; application k >= 2 consumes (g_{k-1}, d_{k-1}) - the *recorded* draft - at head position Len+k-3,
seeing the prefix and the chain's own earlier entries only.  Nothing is sampled.  q_k = softmax(logits(g_k)/T).

Objective.  alpha_k = sum_d min(p_k(d), q_k(d)) (Eq. 5), estimated from the record's top-64 target
log-probabilities plus one residual bin (App. D.2); the chain surrogate -sum_l prod_{i<=l} alpha_i (Eq. 6),
its logarithmic form (Eq. 7) and the truncation of the chain sum at min(j, K), j the first rejected
position, K+1 if none (Eq. 9).  The update minimises the mean over cycles.

First step of the backward pass: the gradient of that mean with respect to the reconstructed head logits.
dL/dalpha_k is Eq. 8 with the chain sums cut at min(j, K) (zero beyond the cut).  alpha_k is piecewise linear
in q_k: on a retained token the slope is 1 where q < p, and the residual bin, q_res = 1 - (sum of q over the
retained tokens), contributes -1 on every retained token where q_res < p_res; at a tie the slope is taken as 0.
The chain rule through q = softmax(logits / T) gives dalpha/dlogit_v = q_v (g_v - sum_d q_d g_d) / T.

Second step (Alg. 1, "update phi"): from the logits back to the head state g_k that produced them.  The head's logits
are LMhead(RMSNorm_hf(g_k)) with the backbone's LM head (App. B.1), so dL/dy = (dL/dlogits) W_lm for the normed state y
and dL/dg follows from the derivative of the RMSNorm.  This is the partial derivative through the logits of position
k alone; the recurrence g_k -> g_{k+1} (Eq. 4) adds further terms in a later step of the backward pass.

Third step: through the feed-forward half of the head's decoder layer (App. B.1: the head is one more layer of the
backbone's shape), g = x + W_d (silu(W_g u) * (W_u u)) with u = RMSNorm(x; ln2).  Given dL/dg it returns dL/dx (the
residual path plus the path through the block) and the gradients of the block's four parameter tensors, which are the
first of the head's own weights the update step touches (Alg. 1, "update phi").

The attention core of the head's layer (scores, softmax, weighted values) has its backward as an operator of its own:
gradients with respect to the queries and to every cached key and value, whichever pass wrote them (the committed
prefix is shared by all chains of a sequence, so its entries collect terms from all of them).

Fourth step: through the head's input (App. B.1), z = W_p [RMSNorm_e(E[token]) ; RMSNorm_h(hidden)].  Given dL/dz it returns
the gradients of the projection and of the two norm weights (the embedding table is the backbone's: no gradient), and
dL/d(hidden) - which, for a draft application k >= 2, is a further term of dL/dg_{k-1}: the recurrence of Eq. 4.

The attention half of the head's layer around that core: the output projection, the rotary embedding (its backward is
the rotation by the opposite angle), the optional per-head norms and projection biases, the query / key / value
projections and the first norm.  With it the pieces chain into the gradient of the whole objective with respect to
every parameter of the head (`head_update_grad`): applications are walked from the last draft back to the pass over
the committed prefix, a state's gradient collecting the term through its own logits and the term through the next
application's input (Eq. 4), a cache entry's gradient collecting the terms of every later row that attended to it
before the application that wrote it is walked.

The update itself: AdamW on the head's parameter group, with the head's learning-rate schedule (App. B, optimizer and
learning rate: linear warm-up over 10 steps, then a cosine decay to a tenth of the peak).  The paper names the
optimizer and the rates only; the moment coefficients, the stabilising constant and the weight decay are the defaults
of the optimizer it names (0.9, 0.999, 1e-8, 0.01), with the decay applied to the parameter directly (decoupled).
"""
from __future__ import annotations

import numpy as np

from . import record, sampler
from .model import (PagedKV, attention, attention_block, f64, ffn_block, head_forward, head_input, head_logits, project_qkv,
                    rmsnorm, rope, round_bf16)


def reconstruct_states(w, cfg, seq_hidden, seq_tokens, start_len: int, drafts) -> np.ndarray:
    """The recurrence of Eq. 4 for one cycle: g_1 from the committed prefix, g_k from (g_{k-1}, d_{k-1}).
    seq_hidden[i] = H_i, the target hidden state that produced token x_{i+1}; seq_tokens = the sequence's
    committed tokens; start_len = Len >= 2 (a prompt token and the first response token at least).  Returns g [K, d]."""
    Len, K = int(start_len), len(drafts)
    assert Len >= 2 and len(seq_tokens) >= Len and len(seq_hidden) >= Len - 1
    pages = (Len + K + cfg.page_size) // cfg.page_size + 1
    hkv = PagedKV(1, cfg.n_kv_heads, cfg.head_dim, np.arange(pages)[None, :], pages, cfg.page_size)
    g = head_forward(w, np.asarray(seq_hidden)[:Len - 1], list(seq_tokens[1:Len]), np.arange(Len - 1), hkv, 0, cfg)[-1:]
    gs = []
    for k in range(1, K + 1):
        if k > 1:
            g = head_forward(w, g, [int(drafts[k - 2])], np.array([Len + k - 3]), hkv, 0, cfg)
        gs.append(g[0])
    return np.array(gs)


def reconstruct_chain(w, cfg, seq_hidden, seq_tokens, start_len: int, drafts, temperature: float = 1.0,
                      round_interface: bool = True):
    """Eq. 4 for one cycle: q_k = softmax(LMhead(norm(g_k)) / T) from the states above.
    Returns (q[K, V] fp32, logits[K, V])."""
    qs, lgs = [], []
    for g in reconstruct_states(w, cfg, seq_hidden, seq_tokens, start_len, drafts):
        lg = head_logits(w, g[None, :], cfg)[0]
        if round_interface:
            lg = round_bf16(lg).astype(np.float64)
        lgs.append(lg)
        qs.append(sampler.softmax_probs(lg, temperature))
    return np.array(qs), np.array(lgs)


def chain_alphas(rec: dict, q) -> np.ndarray:
    """alpha_k, k = 1..K, of one recorded cycle from its top-64 record and the reconstructed q[K, V]."""
    return np.array([record.sparsified_overlap(rec["top_index"][k], rec["top_logprob"][k], q[k])
                     for k in range(len(q))])


def tv_chain_loss(alphas) -> float:
    """L_TV = - sum_{l=1..K} prod_{i<=l} alpha_i   (Eq. 6)."""
    return -float(np.cumprod(np.asarray(alphas, np.float64)).sum())


def dca_loss(alphas, j: int | None = None) -> float:
    """L_DCA = - log sum_{l=1..L} exp(sum_{i<=l} log alpha_i), L = K (Eq. 7) or min(j, K) (Eq. 9)."""
    a = np.asarray(alphas, np.float64)
    L = len(a) if j is None else min(int(j), len(a))
    assert L >= 1
    with np.errstate(divide="ignore"):
        s = np.cumsum(np.log(a[:L]))
    m = s.max()
    if not np.isfinite(m):
        return float("inf")
    return -float(m + np.log(np.exp(s - m).sum()))


def dca_position_weights(alphas) -> np.ndarray:
    """-dL_DCA/dalpha_k = (prod_{i<k} alpha_i) D_k / (-L_TV), D_k = sum_{l>=k} prod_{i=k+1..l} alpha_i   (Eq. 8)."""
    a = np.asarray(alphas, np.float64)
    K = len(a)
    out = np.zeros(K)
    for k in range(K):
        D = sum(np.prod(a[k + 1:l + 1]) for l in range(k, K))
        out[k] = np.prod(a[:k]) * D / (-tv_chain_loss(a))
    return out


def softmax64(logits, temperature: float) -> np.ndarray:
    x = np.asarray(logits, np.float64) / float(temperature)
    e = np.exp(x - x.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def dca_loss_grad_alpha(alphas, j: int | None = None) -> np.ndarray:
    """dL/dalpha_k of Eq. 9 for one cycle: -(prod_{i<k} alpha_i) D_k / M with M and D_k cut at L = min(j, K);
    0 for k > L (Eq. 8 with the verify gate)."""
    a = np.asarray(alphas, np.float64)
    K = len(a)
    L = K if j is None else min(int(j), K)
    M = np.cumprod(a[:L]).sum()
    g = np.zeros(K)
    for k in range(L):
        D = sum(np.prod(a[k + 1:l + 1]) for l in range(k, L))
        g[k] = -np.prod(a[:k]) * D / M
    return g


def overlap_grad_logits(p_top_idx, p_top_logprob, logits, temperature: float) -> np.ndarray:
    """dalpha/dlogits [V] of the sparsified overlap (App. D.2) at q = softmax(logits / T)."""
    q = softmax64(logits, temperature)
    keep = np.asarray(p_top_idx) >= 0
    idx = np.asarray(p_top_idx)[keep]
    p_kept = np.exp(np.asarray(p_top_logprob, np.float64)[keep])
    q_kept = q[idx]
    p_res, q_res = max(1.0 - p_kept.sum(), 0.0), max(1.0 - q_kept.sum(), 0.0)
    g = np.zeros(len(q))
    g[idx] = (q_kept < p_kept).astype(np.float64) - (1.0 if q_res < p_res else 0.0)
    return q * (g - float((q * g).sum())) / temperature


def head_update_grad_logits(logits, records, temperature: float = 1.0) -> np.ndarray:
    """d(mean over cycles of Eq. 9)/d(reconstructed logits): logits [n, K, V]; records = the n record dicts."""
    logits = np.asarray(logits, np.float64)
    n, K, V = logits.shape
    out = np.zeros((n, K, V))
    for r, rec in enumerate(records):
        q = softmax64(logits[r], temperature)
        ga = dca_loss_grad_alpha(chain_alphas(rec, q), rec["accepted"])
        for k in range(K):
            if ga[k] != 0.0:
                out[r, k] = ga[k] * overlap_grad_logits(rec["top_index"][k], rec["top_logprob"][k], logits[r, k], temperature)
    return out / n


def head_update_loss(w, cfg, sequences, records, temperature: float = 1.0, round_interface: bool = True):
    """Mean of Eq. 9 over recorded cycles.  sequences[s] = (seq_hidden, seq_tokens); records = list of
    (s, record dict as oracle.record.cycle_record builds it).  Returns (loss, alphas[n_cycles, K])."""
    losses, alphas = [], []
    for s, rec in records:
        hid, toks = sequences[s]
        q, _ = reconstruct_chain(w, cfg, hid, toks, rec["start_pos"], rec["drafts"], temperature, round_interface)
        a = chain_alphas(rec, q)
        alphas.append(a)
        losses.append(dca_loss(a, rec["accepted"]))
    return float(np.mean(losses)), np.array(alphas)


def lm_head_input_grad(grad_logits, w_lm) -> np.ndarray:
    """logits = y W_lm^T  =>  dL/dy = (dL/dlogits) W_lm.   grad_logits [..., V], w_lm [V, d]  ->  [..., d]."""
    return np.asarray(grad_logits, np.float64) @ f64(w_lm)


def rmsnorm_grad(dy, x, weight, eps: float) -> np.ndarray:
    """Derivative of y = x r w, r = (mean(x^2) + eps)^(-1/2), with respect to x:
    dL/dx = r (w dy) - x r^3 mean(x w dy)   (the second term is the derivative of r)."""
    x, dy, w = f64(x), f64(dy), f64(weight)
    r = 1.0 / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)
    wdy = w * dy
    return r * wdy - x * r ** 3 * (x * wdy).mean(axis=-1, keepdims=True)


def head_update_grad_state(w, cfg, states, records, temperature: float = 1.0):
    """d(mean over cycles of Eq. 9)/d(head states), through the head's final norm and the shared LM head only.
    states [n, K, d] = g_k of every recorded cycle (what the reconstruction computes); records = the n record dicts.
    Returns (grad_state [n, K, d], grad_normed [n, K, d], logits [n, K, V])."""
    states = np.asarray(states, np.float64)
    n, K, d = states.shape
    logits = head_logits(w, states.reshape(n * K, d), cfg).reshape(n, K, -1)
    gl = head_update_grad_logits(logits, records, temperature)
    gy = lm_head_input_grad(gl, w["lm_head"])
    return rmsnorm_grad(gy, states, w["head"]["final_norm"], cfg.rms_eps), gy, logits


def ffn_block_grad(dg, x, lw, eps: float) -> dict:
    """Backward of model.ffn_block.  dg [T, d] = dL/d(output), x [T, d] = the block's input (residual stream after
    attention), lw = the layer's weights (ln2 [d], wg / wu [F, d], wd [d, F]).
    Returns {"dx", "dln2", "dwg", "dwu", "dwd"} in float64."""
    dg, x = f64(dg), f64(x)
    w2, wg, wu, wd = f64(lw["ln2"]), f64(lw["wg"]), f64(lw["wu"]), f64(lw["wd"])
    r = 1.0 / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)
    u = x * r * w2
    a, b = u @ wg.T, u @ wu.T
    sig = 1.0 / (1.0 + np.exp(-a))
    act = a * sig
    h = act * b
    dh = dg @ wd                                              # y = h W_d^T
    dwd = dg.T @ h
    db = dh * act
    da = dh * b * sig * (1.0 + a * (1.0 - sig))               # d silu(a) / da = sig (1 + a (1 - sig))
    dwg, dwu = da.T @ u, db.T @ u
    du = da @ wg + db @ wu
    dx = dg + rmsnorm_grad(du, x, w2, eps)
    dln2 = (du * x * r).sum(axis=0)
    return {"dx": dx, "dln2": dln2, "dwg": dwg, "dwu": dwu, "dwd": dwd}


def attention_grad(dout, q, k, v, q_pos, k_pos):
    """Backward of model.attention (causal grouped-query attention with an explicit softmax).  dout, q [T, n_q, hd];
    k, v [S, n_kv, hd].  Per head, with P = softmax(S), S = q k^T / sqrt(hd) on the visible keys:
        dP = dout v^T,  dS = P * (dP - rowsum(dP * P)),  dq = dS k / sqrt(hd),  dk += dS^T q / sqrt(hd),  dv += P^T dout
    (keys and values of a KV head collect the terms of every query head of their group).  Returns (dq, dk, dv), float64."""
    dout, q, k, v = f64(dout), f64(q), f64(k), f64(v)
    T, n_q, hd = q.shape
    g = n_q // k.shape[1]
    visible = np.asarray(k_pos)[None, :] <= np.asarray(q_pos)[:, None]
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    scale = 1.0 / np.sqrt(hd)
    for h in range(n_q):
        kh, vh = k[:, h // g, :], v[:, h // g, :]
        sc = np.where(visible, q[:, h, :] @ kh.T * scale, -np.inf)
        e = np.exp(sc - sc.max(axis=1, keepdims=True))
        pr = e / e.sum(axis=1, keepdims=True)
        dpr = dout[:, h, :] @ vh.T
        ds = pr * (dpr - (dpr * pr).sum(axis=1, keepdims=True))
        dq[:, h, :] = ds @ kh * scale
        dk[:, h // g, :] += ds.T @ q[:, h, :] * scale
        dv[:, h // g, :] += pr.T @ dout[:, h, :]
    return dq, dk, dv


def head_input_grad(dz, w, hidden, tokens, cfg) -> dict:
    """Backward of model.head_input.  dz [T, d] = dL/dz; hidden [T, d], tokens [T] = the pairs that entered.
    Returns {"dhidden" [T, d], "dproj" [d, 2d] (columns in the order the head concatenates), "denorm" [d], "dhnorm" [d]}."""
    hw = w["head"]
    dz, hidden = f64(dz), f64(hidden)
    d = hidden.shape[-1]
    e = f64(w["embed"])[np.asarray(tokens)]
    en, hn = rmsnorm(e, hw["enorm"], cfg.rms_eps), rmsnorm(hidden, hw["hnorm"], cfg.rms_eps)
    hidden_first = hw.get("concat", "embedding_first") == "hidden_first"
    zin = np.concatenate([hn, en] if hidden_first else [en, hn], axis=-1)
    dzin = dz @ f64(hw["proj"])
    dproj = dz.T @ zin
    dhn, den = (dzin[:, :d], dzin[:, d:]) if hidden_first else (dzin[:, d:], dzin[:, :d])
    r_e = 1.0 / np.sqrt((e * e).mean(axis=-1, keepdims=True) + cfg.rms_eps)
    r_h = 1.0 / np.sqrt((hidden * hidden).mean(axis=-1, keepdims=True) + cfg.rms_eps)
    return {"dhidden": rmsnorm_grad(dhn, hidden, hw["hnorm"], cfg.rms_eps), "dproj": dproj,
            "denorm": (den * e * r_e).sum(axis=0), "dhnorm": (dhn * hidden * r_h).sum(axis=0)}


def rope_grad(dy, pos, base: float) -> np.ndarray:
    """Backward of model.rope: a rotation is linear and orthogonal, so the gradient turns by the opposite angle.
    dy [T, H, hd], pos [T]."""
    return rope(dy, -f64(pos), base)


def _rms_weight_grad(dy, x, eps: float) -> np.ndarray:
    """dL/dw of y = x r w summed over every leading axis: sum dy x r."""
    x, dy = f64(x), f64(dy)
    r = 1.0 / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)
    return (dy * x * r).reshape(-1, x.shape[-1]).sum(axis=0)


def attention_block_grad(dxmid, x, lw, pos, kc, vc, dkc, dvc, cfg) -> dict:
    """Backward of model.attention_block for rows x [T, d] at positions pos.  dxmid [T, d] = dL/d(output).
    kc, vc [n, n_kv, hd] = cache entries 0..n-1 as the rows saw them (their own included, n = max(pos) + 1).
    dkc, dvc [>= n, n_kv, hd] = gradient already collected on the cache entries from rows of later applications;
    the terms of these rows are added IN PLACE, after which the rows' own entries are complete and are taken back
    through the rotary embedding, the optional head norms and the projections.
    Returns {"dx", "dln1", "dwq", "dwk", "dwv", "dwo"} plus {"dbq", "dbk", "dbv"} / {"dqnorm", "dknorm"} where the
    layer has them."""
    dxmid, x = f64(dxmid), f64(x)
    T = x.shape[0]
    pos = np.asarray(pos)
    n = int(pos.max()) + 1
    eps = cfg.rms_eps
    h = rmsnorm(x, lw["ln1"], eps)
    raw = {k: v for k, v in lw.items() if k not in ("qnorm", "knorm")}
    q0, k0, _ = project_qkv(raw, h, cfg)                       # heads before the optional norm
    qn, _, _ = project_qkv(lw, h, cfg)
    q = rope(qn, pos, cfg.rope_base)
    o = attention(q, kc[:n], vc[:n], pos, np.arange(n)).reshape(T, cfg.q_dim)
    out = {"dwo": dxmid.T @ o}
    do = (dxmid @ f64(lw["wo"])).reshape(T, cfg.n_q_heads, cfg.head_dim)
    dq, dk_all, dv_all = attention_grad(do, q, kc[:n], vc[:n], pos, np.arange(n))
    dkc[:n] += dk_all
    dvc[:n] += dv_all
    dq = rope_grad(dq, pos, cfg.rope_base)
    dk = rope_grad(dkc[pos], pos, cfg.rope_base)
    dv = f64(dvc[pos])
    if "qnorm" in lw:
        out["dqnorm"], out["dknorm"] = _rms_weight_grad(dq, q0, eps), _rms_weight_grad(dk, k0, eps)
        dq, dk = rmsnorm_grad(dq, q0, lw["qnorm"], eps), rmsnorm_grad(dk, k0, lw["knorm"], eps)
    dq, dk, dv = dq.reshape(T, -1), dk.reshape(T, -1), dv.reshape(T, -1)
    if "bq" in lw:
        out["dbq"], out["dbk"], out["dbv"] = dq.sum(axis=0), dk.sum(axis=0), dv.sum(axis=0)
    out["dwq"], out["dwk"], out["dwv"] = dq.T @ h, dk.T @ h, dv.T @ h
    dh = dq @ f64(lw["wq"]) + dk @ f64(lw["wk"]) + dv @ f64(lw["wv"])
    out["dx"] = dxmid + rmsnorm_grad(dh, x, lw["ln1"], eps)
    out["dln1"] = _rms_weight_grad(dh, x, eps)
    return out


def _accumulate(total: dict, part: dict, names) -> None:
    for name in names:
        if name in part:
            total[name] = total.get(name, 0.0) + part[name]


def head_update_grad(w, cfg, sequences, records, temperature: float = 1.0, grad_logits=None) -> dict:
    """Gradient of head_update_loss (no rounding at the logits interface) with respect to every parameter of the head.
    Same arguments as head_update_loss.  grad_logits [n_records, K, V], if given, replaces the objective's own
    d(mean loss)/d(logits) (first step of the backward pass) and everything downstream of it is computed as usual - for
    checking a pipeline whose reconstructed logits differ from these in rounding, where the piecewise-linear overlap
    would pick other branches.  Returns {"proj", "enorm", "hnorm", "final_norm", "layer": {"ln1", "wq", "wk",
    "wv", "wo", "ln2", "wg", "wu", "wd" [, "bq", "bk", "bv"] [, "qnorm", "knorm"]}} in float64; the embedding table
    and the LM head are the backbone's and get none."""
    hw, lw = w["head"], w["head"]["layer"]
    top, lay = {}, {}
    n_rec = len(records)
    for r_i, (s, rec) in enumerate(records):
        hid, toks = sequences[s]
        Len, drafts = int(rec["start_pos"]), rec["drafts"]
        K = len(drafts)
        # forward, keeping each application's input pairs and positions (application 1 = the pass over the prefix)
        pages = (Len + K + cfg.page_size) // cfg.page_size + 1
        hkv = PagedKV(1, cfg.n_kv_heads, cfg.head_dim, np.arange(pages)[None, :], pages, cfg.page_size)
        apps = [(f64(np.asarray(hid)[:Len - 1]), list(toks[1:Len]), np.arange(Len - 1))]
        g = head_forward(w, *apps[0], hkv, 0, cfg)[-1:]
        states = [g[0]]
        for k in range(2, K + 1):
            apps.append((g, [int(drafts[k - 2])], np.array([Len + k - 3])))
            g = head_forward(w, *apps[-1], hkv, 0, cfg)
            states.append(g[0])
        states = np.array(states)
        kc, vc = hkv.gather(0, 0, Len + K - 2)
        # the term of every state through its own logits
        if grad_logits is None:
            dstate, gy, _ = head_update_grad_state(w, cfg, states[None], [rec], temperature)
            dstate, gy = dstate[0] / n_rec, gy[0] / n_rec
        else:
            gy = lm_head_input_grad(grad_logits[r_i], w["lm_head"])
            dstate = rmsnorm_grad(gy, states, hw["final_norm"], cfg.rms_eps)
        top["final_norm"] = top.get("final_norm", 0.0) + _rms_weight_grad(gy, states, cfg.rms_eps)
        # backward, last application first
        dkc, dvc = np.zeros_like(kc), np.zeros_like(vc)
        for a in range(K - 1, -1, -1):
            hidden, tokens, pos = apps[a]
            z = head_input(w, hidden, tokens, cfg)
            akv = PagedKV(1, cfg.n_kv_heads, cfg.head_dim, np.arange(pages)[None, :], pages, cfg.page_size)
            akv.pool[:] = hkv.pool                            # entries beyond these rows' positions are never read
            xmid = attention_block(lw, z, pos, akv, 0, 0, cfg)
            dg = np.zeros_like(xmid)
            dg[-1] = dstate[a]                                # only the last row's state is used (all of them: 1 row, a >= 1)
            f = ffn_block_grad(dg, xmid, lw, cfg.rms_eps)
            n = int(pos.max()) + 1
            at = attention_block_grad(f["dx"], z, lw, pos, kc[:n], vc[:n], dkc, dvc, cfg)
            hi = head_input_grad(at["dx"], w, hidden, tokens, cfg)
            if a >= 1:
                dstate[a - 1] += hi["dhidden"][0]             # Eq. 4: this application consumed g_{a}
            _accumulate(lay, {k[1:]: v for k, v in f.items()}, ("ln2", "wg", "wu", "wd"))
            _accumulate(lay, {k[1:]: v for k, v in at.items()},
                        ("ln1", "wq", "wk", "wv", "wo", "bq", "bk", "bv", "qnorm", "knorm"))
            _accumulate(top, {k[1:]: v for k, v in hi.items()}, ("proj", "enorm", "hnorm"))
    top["layer"] = lay
    return top


def adamw_step(p, g, m, v, step: int, lr: float, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
               weight_decay: float = 0.01):
    """One AdamW update (decoupled weight decay); `step` counts from 1.  Returns (p, m, v), float64.
        m <- b1 m + (1 - b1) g,  v <- b2 v + (1 - b2) g^2,
        p <- p (1 - lr wd) - lr (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps)."""
    p, g, m, v = f64(p), f64(g), f64(m), f64(v)
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    m_hat = m / (1.0 - beta1 ** step)
    v_hat = v / (1.0 - beta2 ** step)
    p = p * (1.0 - lr * weight_decay) - lr * m_hat / (np.sqrt(v_hat) + eps)
    return p, m, v


def head_lr(step: int, peak: float, total_steps: int, warmup: int = 10, floor: float = 0.1) -> float:
    """Learning rate of the head's parameter group at update `step` (from 0): linear warm-up to `peak` over `warmup`
    steps, then half a cosine from `peak` down to `floor * peak` at `total_steps`."""
    if step < warmup:
        return peak * (step + 1) / warmup
    t = min(1.0, (step - warmup) / max(1, total_steps - warmup))
    return peak * (floor + (1.0 - floor) * 0.5 * (1.0 + np.cos(np.pi * t)))
