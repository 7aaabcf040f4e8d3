"""Test-side glue: moves an oracle state into the CUDA library's state tensors and back."""
import numpy as np
import torch

import paper_2609_16648_b200 as gmb
from oracle import step as ostep
from synth_inputs import make_page_tables, make_weights, random_prompts
from synth_inputs.weights import perturb_norm_weights


def rel_err(a, b):
    """Per-tensor normalised max error max|a-b| / max|b|."""
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))


def tiny_setup(cfg, cap_tokens, seed=0, perturb=True, flags=0, max_k=None, prompt_seed=1, rounding=True, concat=None):
    """Oracle prefill of the prompts + a CUDA context/state sharing the same page tables."""
    w = make_weights(cfg, seed)
    if perturb:
        w = perturb_norm_weights(w)
    if concat is not None:
        w["head"]["concat"] = concat          # the order the head's two inputs are concatenated in
    prompts = random_prompts(cfg.batch, cfg.prompt_len, cfg.vocab, seed=prompt_seed)
    pt, npg = make_page_tables(np.full(cfg.batch, cap_tokens), cfg.page_size, seed=7, slack_pages=3)
    hpt, hnpg = make_page_tables(np.full(cfg.batch, cap_tokens), cfg.page_size, seed=8, slack_pages=2)
    ost = ostep.prefill(w, cfg, prompts, pt, npg, hpt, hnpg, temperature=cfg.temperature, seed=5,
                        round_interface=rounding)
    max_k = cfg.k if max_k is None else max_k
    ctx = gmb.Context(cfg, gmb.pack_weights(w), cfg.batch, max_k, pt.shape[1], npg, hnpg, flags=flags)
    gst = gmb.State(ctx, cfg.batch, pt, hpt)
    return w, ost, ctx, gst


def push_state(ost, gst, ctx):
    """Oracle state -> device state (KV rounded to bf16)."""
    B = len(ost.seqs)
    gst.kv_pool.copy_(torch.from_numpy(ost.kv.pool).to(torch.bfloat16))
    gst.head_kv_pool.copy_(torch.from_numpy(ost.hkv.pool).to(torch.bfloat16))
    kv_len = np.array([s.kv_len for s in ost.seqs], np.int32)
    pn = np.array([len(s.pending_tok) for s in ost.seqs], np.int32)
    ptok = np.zeros((B, ctx.max_k + 1), np.int32)
    phid = np.zeros((B, ctx.max_k + 1, ctx.cfg.d_model), np.float32)
    for b, s in enumerate(ost.seqs):
        ptok[b, :pn[b]] = s.pending_tok
        phid[b, :pn[b]] = s.pending_hidden
    gst.kv_len.copy_(torch.from_numpy(kv_len))
    gst.pending_n.copy_(torch.from_numpy(pn))
    gst.pending_tok.copy_(torch.from_numpy(ptok))
    gst.pending_hidden.copy_(torch.from_numpy(phid).to(torch.bfloat16))
    torch.cuda.synchronize()


# ---- "a disagreement is a threshold case": what rounding may explain, and nothing more -----------------------------------
# Both sides run the same rule (checked bit for bit on the device's own probabilities elsewhere); they may still decide
# differently because their logits differ by rounding.  A logit row that is off by at most eps (absolute, after the
# temperature) moves every probability by a factor within exp(+-2 eps) - numerator and normaliser - so the
# distribution moves by at most E(eps) = exp(2 eps) - 1 in total variation mass.  The helpers below accept a
# disagreement only if the oracle's own numbers are within that band of the decision boundary.

def band(eps: float) -> float:
    return float(np.expm1(2.0 * eps))


def softmax64(logits, temperature=1.0):
    x = np.asarray(logits, np.float64) / temperature
    e = np.exp(x - x.max())
    return e / e.sum()


def draw_is_threshold_case(weights_or, u24: int, tok_dev: int, tok_or: int, delta: float) -> bool:
    """The oracle drew tok_or at quantile u from its (unnormalised) weights, the device drew tok_dev != tok_or at the
    same u from its own: explained by rounding iff u lies within `delta` (in normalised CDF mass, the bound on the two
    CDFs' distance) of the oracle's boundary on the device token's side."""
    w = np.asarray(weights_or, np.float64)
    cdf = np.cumsum(w) / w.sum()
    u = u24 / 2.0 ** 24
    dist = cdf[tok_dev - 1] - u if tok_dev > tok_or else u - cdf[tok_dev]
    return dist <= delta + 2.0 ** -20          # + the 24-bit quantile and the 44-bit weight quantisation


def accept_bit_is_threshold_case(p_or: float, q_or: float, u24: int, eps_p: float, eps_q: float) -> bool:
    """Opposite accept bits for the same draft: the margins p - u q have opposite signs on the two sides, so the
    oracle's margin is at most the two sides' difference, which the logit errors bound."""
    u = u24 / 2.0 ** 24
    return abs(p_or - u * q_or) <= band(eps_p) * p_or + band(eps_q) * u * q_or + 1e-12
