"""Pins for the oracle's decoder blocks: closed forms, library routines, brute force, invariants."""
import dataclasses
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import model
from synth_inputs import ModelConfig, make_weights, make_page_tables, bf16_round
from synth_inputs.weights import perturb_norm_weights

CFG = ModelConfig("t", 2, 64, 4, 2, 16, 96, 50, batch=2, k=3, kv_len_min=0, kv_len_max=0,
                  length_law="prompt")


def test_round_bf16_matches_library_conversion():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 1, 5000), rng.normal(0, 1e-20, 100), [0.0, -0.0, 1.0, 65504.0]])
    x = x.astype(np.float32)
    # exact ties: a bf16 value plus half an ulp
    ties = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.0 - 2.0 ** -7], np.float32)
    x = np.concatenate([x, ties])
    np.testing.assert_array_equal(model.round_bf16(x), bf16_round(x))


def test_rmsnorm_closed_forms_and_library():
    w = np.linspace(0.5, 1.5, 64)
    np.testing.assert_allclose(model.rmsnorm(np.full(64, 3.0), w, 1e-12), w, rtol=1e-9)
    np.testing.assert_allclose(model.rmsnorm(np.full(64, -2.0), w, 1e-12), -w, rtol=1e-9)
    rng = np.random.default_rng(1)
    x = rng.normal(0, 2, (7, 64))
    ref = F.rms_norm(torch.from_numpy(x), (64,), torch.from_numpy(w), eps=1e-6).numpy()
    np.testing.assert_allclose(model.rmsnorm(x, w, 1e-6), ref, rtol=1e-12)
    y = model.rmsnorm(x, np.ones(64), 0.0)
    np.testing.assert_allclose(np.mean(y * y, axis=-1), 1.0, rtol=1e-12)      # unit RMS
    np.testing.assert_allclose(model.rmsnorm(5 * x, w, 0.0), model.rmsnorm(x, w, 0.0), rtol=1e-12)


def test_silu_library():
    x = np.linspace(-8, 8, 101)
    np.testing.assert_allclose(model.silu(x), F.silu(torch.from_numpy(x)).numpy(), rtol=1e-12)


def test_rope_properties():
    rng = np.random.default_rng(2)
    hd = 16
    x = rng.normal(size=(5, 3, hd))
    pos = np.array([0, 1, 7, 100, 4000])
    y = model.rope(x, pos, 1e4)
    np.testing.assert_allclose(y[0], x[0], atol=1e-15)                          # position 0 = identity
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    # complex form: (x_i + j x_{i+hd/2}) * exp(j pos base^(-2i/hd))
    z = (x[..., :hd // 2] + 1j * x[..., hd // 2:]) * np.exp(
        1j * pos[:, None, None] * (1e4 ** (-np.arange(hd // 2) * 2.0 / hd))[None, None, :])
    np.testing.assert_allclose(y, np.concatenate([z.real, z.imag], -1), rtol=1e-10, atol=1e-12)
    # head_dim 2: a plane rotation by pos radians
    v = model.rope(np.array([[[1.0, 0.0]]]), np.array([3]), 1e4)[0, 0]
    np.testing.assert_allclose(v, [math.cos(3), math.sin(3)], rtol=1e-12)
    # scores depend on position differences only
    q, k = rng.normal(size=(1, 1, hd)), rng.normal(size=(1, 1, hd))
    s0 = (model.rope(q, [10], 1e4) * model.rope(k, [4], 1e4)).sum()
    s1 = (model.rope(q, [510], 1e4) * model.rope(k, [504], 1e4)).sum()
    assert abs(s0 - s1) < 1e-10


def _loop_attention(q, k, v, q_pos, k_pos):
    """Scalar loops, math.exp: the definition, one number at a time."""
    T, nq, hd = q.shape
    g = nq // k.shape[1]
    out = np.zeros_like(q)
    for t in range(T):
        for h in range(nq):
            vis = [s for s in range(len(k_pos)) if k_pos[s] <= q_pos[t]]
            sc = [sum(q[t, h, i] * k[s, h // g, i] for i in range(hd)) / math.sqrt(hd) for s in vis]
            m = max(sc)
            e = [math.exp(x - m) for x in sc]
            z = sum(e)
            for i in range(hd):
                out[t, h, i] = sum(e[j] * v[s, h // g, i] for j, s in enumerate(vis)) / z
    return out


def test_attention_against_scalar_brute_force_and_library():
    rng = np.random.default_rng(3)
    T, S, nq, nkv, hd = 4, 11, 4, 2, 8
    q, k, v = rng.normal(size=(T, nq, hd)), rng.normal(size=(S, nkv, hd)), rng.normal(size=(S, nkv, hd))
    q_pos, k_pos = np.arange(S - T, S), np.arange(S)
    out = model.attention(q, k, v, q_pos, k_pos)
    np.testing.assert_allclose(out, _loop_attention(q, k, v, q_pos, k_pos), rtol=1e-10, atol=1e-12)
    mask = torch.from_numpy(k_pos[None, :] <= q_pos[:, None])
    ref = F.scaled_dot_product_attention(
        torch.from_numpy(q).permute(1, 0, 2)[None], torch.from_numpy(np.repeat(k, 2, 1)).permute(1, 0, 2)[None],
        torch.from_numpy(np.repeat(v, 2, 1)).permute(1, 0, 2)[None], attn_mask=mask)[0].permute(1, 0, 2)
    np.testing.assert_allclose(out, ref.numpy(), rtol=1e-9, atol=1e-12)


def test_attention_special_cases():
    rng = np.random.default_rng(4)
    nq, nkv, hd = 4, 2, 8
    q = rng.normal(size=(3, nq, hd))
    k1, v1 = rng.normal(size=(1, nkv, hd)), rng.normal(size=(1, nkv, hd))
    out = model.attention(q, k1, v1, [0, 0, 0], [0])                     # one key: out = v_0
    np.testing.assert_allclose(out, np.repeat(v1, 2, 1).repeat(3, 0), rtol=1e-12)
    S = 9
    v = rng.normal(size=(S, nkv, hd))
    keq = np.repeat(rng.normal(size=(1, nkv, hd)), S, 0)                 # equal keys: mean of visible V
    out = model.attention(q, keq, v, [2, 5, 8], np.arange(S))
    for t, p in enumerate([2, 5, 8]):
        np.testing.assert_allclose(out[t], np.repeat(v[:p + 1].mean(0), 2, 0), rtol=1e-10)
    veq = np.repeat(rng.normal(size=(1, nkv, hd)), S, 0)                 # equal values: that row
    out = model.attention(q, rng.normal(size=(S, nkv, hd)), veq, [2, 5, 8], np.arange(S))
    np.testing.assert_allclose(out, np.repeat(veq[:1], 2, 1).repeat(3, 0), rtol=1e-10)
    # grouped-query == multi-head with repeated key/value heads
    k = rng.normal(size=(S, nkv, hd))
    np.testing.assert_allclose(model.attention(q, k, v, [2, 5, 8], np.arange(S)),
                               model.attention(q, np.repeat(k, 2, 1), np.repeat(v, 2, 1), [2, 5, 8], np.arange(S)),
                               rtol=1e-12)
    # causality: a future key's content is irrelevant
    k2, v2 = k.copy(), v.copy()
    k2[6:], v2[6:] = 99.0, -99.0
    np.testing.assert_allclose(model.attention(q[:2], k, v, [2, 5], np.arange(S)),
                               model.attention(q[:2], k2, v2, [2, 5], np.arange(S)), rtol=1e-12)


def _weights(cfg, seed=0):
    return perturb_norm_weights(make_weights(cfg, seed))


def _kv(cfg, n_layers, cap, seed=7, B=None):
    B = cfg.batch if B is None else B
    table, npages = make_page_tables(np.full(B, cap), cfg.page_size, seed)
    return model.PagedKV(n_layers, cfg.n_kv_heads, cfg.head_dim, table, npages, cfg.page_size)


def test_paged_cache_equals_contiguous_under_any_page_permutation():
    w = _weights(CFG)
    toks = np.random.default_rng(5).integers(0, CFG.vocab, 40)
    outs = []
    for seed in (1, 2, 3):
        kv = _kv(CFG, CFG.n_layers, 64, seed)
        outs.append(model.target_forward(w, toks, np.arange(40), kv, 1, CFG))
        k, v = kv.gather(0, 1, 40)
        outs.append(k)
    ident = model.PagedKV(CFG.n_layers, CFG.n_kv_heads, CFG.head_dim,
                          np.arange(8).reshape(2, 4), 8, CFG.page_size)      # contiguous layout
    ref = model.target_forward(w, toks, np.arange(40), ident, 1, CFG)
    for o in outs[0::2]:
        np.testing.assert_array_equal(o, ref)
    np.testing.assert_array_equal(outs[1], ident.gather(0, 1, 40)[0])
    np.testing.assert_array_equal(outs[1], outs[3])


def test_incremental_forward_equals_full_recompute():
    """The K+1 rows of a cached verify forward == the last K+1 rows of a from-scratch causal
    forward over the whole sequence; also when the chunk overwrites stale entries."""
    w = _weights(CFG)
    rng = np.random.default_rng(6)
    toks = rng.integers(0, CFG.vocab, 37)
    full = model.target_forward(w, toks, np.arange(37), _kv(CFG, CFG.n_layers, 64), 0, CFG)
    kv = _kv(CFG, CFG.n_layers, 64)
    a = model.target_forward(w, toks[:20], np.arange(20), kv, 0, CFG)
    # a rejected chain leaves garbage at 20..23, the next chunk overwrites it
    model.target_forward(w, rng.integers(0, CFG.vocab, 4), np.arange(20, 24), kv, 0, CFG)
    b = model.target_forward(w, toks[20:33], np.arange(20, 33), kv, 0, CFG)
    c = model.target_forward(w, toks[33:], np.arange(33, 37), kv, 0, CFG)
    np.testing.assert_allclose(np.concatenate([a, b, c]), full, rtol=1e-9, atol=1e-11)


def _torch_layer(lw, x, cfg):
    """Third opinion: a full causal layer from library routines only (fp64)."""
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    T = x.shape[0]
    h = F.rms_norm(t(x), (cfg.d_model,), t(lw["ln1"]), eps=cfg.rms_eps)
    bias = lambda n: t(lw[n]) if n in lw else None
    q = F.linear(h, t(lw["wq"]), bias("bq")).view(T, cfg.n_q_heads, cfg.head_dim)
    k = F.linear(h, t(lw["wk"]), bias("bk")).view(T, cfg.n_kv_heads, cfg.head_dim)
    v = F.linear(h, t(lw["wv"]), bias("bv")).view(T, cfg.n_kv_heads, cfg.head_dim)
    if "qnorm" in lw:
        q = F.rms_norm(q, (cfg.head_dim,), t(lw["qnorm"]), eps=cfg.rms_eps)
        k = F.rms_norm(k, (cfg.head_dim,), t(lw["knorm"]), eps=cfg.rms_eps)
    half = cfg.head_dim // 2
    ang = torch.arange(T, dtype=torch.float64)[:, None] * cfg.rope_base ** (
        -torch.arange(half, dtype=torch.float64) * 2 / cfg.head_dim)
    rot = torch.polar(torch.ones_like(ang), ang)[:, None, :]

    def rp(u):
        z = torch.complex(u[..., :half], u[..., half:]) * rot
        return torch.cat([z.real, z.imag], -1)
    q, k = rp(q), rp(k)
    o = F.scaled_dot_product_attention(q.permute(1, 0, 2)[None], k.permute(1, 0, 2)[None],
                                       v.permute(1, 0, 2)[None], is_causal=True, enable_gqa=True)[0]
    x1 = t(x) + o.permute(1, 0, 2).reshape(T, -1) @ t(lw["wo"]).T
    h2 = F.rms_norm(x1, (cfg.d_model,), t(lw["ln2"]), eps=cfg.rms_eps)
    return (x1 + (F.silu(h2 @ t(lw["wg"]).T) * (h2 @ t(lw["wu"]).T)) @ t(lw["wd"]).T).numpy()


def test_decoder_layer_and_logits_against_library_composition():
    w = _weights(CFG)
    rng = np.random.default_rng(7)
    x = rng.normal(size=(13, CFG.d_model))
    out = model.decoder_layer(w["layers"][1], x, np.arange(13), _kv(CFG, CFG.n_layers, 64), 1, 0, CFG)
    np.testing.assert_allclose(out, _torch_layer(w["layers"][1], x, CFG), rtol=1e-9, atol=1e-11)
    lg = model.target_logits(w, x, CFG)
    ref = F.rms_norm(torch.from_numpy(x), (CFG.d_model,), torch.from_numpy(w["final_norm"].astype(np.float64)),
                     eps=CFG.rms_eps) @ torch.from_numpy(w["lm_head"].astype(np.float64)).T
    np.testing.assert_allclose(lg, ref.numpy(), rtol=1e-10, atol=1e-12)


def test_head_forward_structure():
    """The head = projection of [norm(embedding) ; norm(hidden)] followed by one decoder layer with
    its own cache; it must react to both inputs and use its own norms and weights."""
    w = _weights(CFG)
    rng = np.random.default_rng(8)
    hid = rng.normal(size=(5, CFG.d_model))
    toks = rng.integers(0, CFG.vocab, 5)
    hkv = _kv(CFG, 1, 64)
    g = model.head_forward(w, hid, toks, np.arange(5), hkv, 0, CFG)
    # independent composition through the (already pinned) layer
    e = w["embed"].astype(np.float64)[toks]
    z = np.concatenate([model.rmsnorm(e, w["head"]["enorm"], CFG.rms_eps),
                        model.rmsnorm(hid, w["head"]["hnorm"], CFG.rms_eps)], -1) @ w["head"]["proj"].astype(np.float64).T
    np.testing.assert_allclose(g, _torch_layer(w["head"]["layer"], z, CFG), rtol=1e-9, atol=1e-11)
    # scale invariance of each input (each has its own RMSNorm in front)
    g2 = model.head_forward(w, 3.0 * hid, toks, np.arange(5), _kv(CFG, 1, 64), 0, CFG)
    np.testing.assert_allclose(g2, g, rtol=1e-3, atol=1e-6)   # up to eps
    g3 = model.head_forward(w, hid, (toks + 1) % CFG.vocab, np.arange(5), _kv(CFG, 1, 64), 0, CFG)
    assert np.abs(g3 - g).max() > 1e-3
    lg = model.head_logits(w, g, CFG)
    assert lg.shape == (5, CFG.vocab)
    np.testing.assert_allclose(lg, model.rmsnorm(g, w["head"]["final_norm"], CFG.rms_eps)
                               @ w["lm_head"].astype(np.float64).T, rtol=1e-12)


# ---- decoder-layer families and the head's concatenation order (App. B.1) ---------------------------

@pytest.mark.parametrize("bias,qkn", [(True, False), (False, True), (True, True)])
def test_family_layers_against_library_composition(bias, qkn):
    cfg = dataclasses.replace(CFG, qkv_bias=bias, qk_norm=qkn)
    w = _weights(cfg)
    lw = w["layers"][1]
    assert ("bq" in lw) == bias and ("qnorm" in lw) == qkn
    rng = np.random.default_rng(17)
    x = rng.normal(size=(11, cfg.d_model))
    out = model.decoder_layer(lw, x, np.arange(11), _kv(cfg, cfg.n_layers, 64), 1, 0, cfg)
    np.testing.assert_allclose(out, _torch_layer(lw, x, cfg), rtol=1e-9, atol=1e-11)
    # and the extras matter: dropping them changes the output
    plain = {k: v for k, v in lw.items() if k not in ("bq", "bk", "bv", "qnorm", "knorm")}
    out0 = model.decoder_layer(plain, x, np.arange(11), _kv(cfg, cfg.n_layers, 64), 1, 0, cfg)
    assert np.abs(out0 - out).max() > 1e-3


def test_projection_bias_is_an_extra_input_column():
    """h W^T + b == [h, 1] [W, b]^T; a zero bias changes nothing."""
    cfg = dataclasses.replace(CFG, qkv_bias=True)
    lw = _weights(cfg)["layers"][0]
    rng = np.random.default_rng(18)
    h = rng.normal(size=(7, cfg.d_model))
    q, k, v = model.project_qkv(lw, h, cfg)
    h1 = np.concatenate([h, np.ones((7, 1))], 1)
    for got, wn, bn in ((q, "wq", "bq"), (k, "wk", "bk"), (v, "wv", "bv")):
        aug = np.concatenate([lw[wn].astype(np.float64), lw[bn].astype(np.float64)[:, None]], 1)
        np.testing.assert_allclose(got.reshape(7, -1), h1 @ aug.T, rtol=1e-12, atol=1e-14)
    zero = dict(lw, bq=np.zeros_like(lw["bq"]), bk=np.zeros_like(lw["bk"]), bv=np.zeros_like(lw["bv"]))
    plain = {k_: v_ for k_, v_ in lw.items() if k_ not in ("bq", "bk", "bv")}
    for a, b in zip(model.project_qkv(zero, h, cfg), model.project_qkv(plain, h, cfg)):
        np.testing.assert_array_equal(a, b)


def test_query_key_norm_properties():
    """With unit weights every query and key head has mean square 1 (up to eps), whatever the scale of
    the projection; values are not normalised; the weight multiplies element-wise after the division."""
    cfg = dataclasses.replace(CFG, qk_norm=True)
    lw = make_weights(cfg, seed=3)["layers"][0]            # norm weights are one
    rng = np.random.default_rng(19)
    h = rng.normal(size=(9, cfg.d_model))
    q, k, v = model.project_qkv(lw, h, cfg)
    np.testing.assert_allclose((q * q).mean(-1), 1.0, rtol=1e-3)
    np.testing.assert_allclose((k * k).mean(-1), 1.0, rtol=1e-3)
    assert abs((v * v).mean() - 1.0) > 0.1
    big = dict(lw, wq=lw["wq"] * 8.0, wv=lw["wv"] * 8.0)
    q8, k8, v8 = model.project_qkv(big, h, cfg)
    np.testing.assert_allclose(q8, q, rtol=1e-3, atol=1e-6)
    np.testing.assert_allclose(v8, 8.0 * v, rtol=1e-12)
    g = rng.uniform(0.5, 1.5, cfg.head_dim)
    qg, _, _ = model.project_qkv(dict(lw, qnorm=g), h, cfg)
    np.testing.assert_allclose(qg, q * g, rtol=1e-12)
    # the norm comes before the rotary embedding: rotating afterwards keeps the head's mean square
    qr = model.rope(q, np.arange(9), cfg.rope_base)
    np.testing.assert_allclose((qr * qr).mean(-1), 1.0, rtol=1e-3)


def test_opposite_concatenation_order_is_a_swap_of_the_projection_halves():
    w = _weights(CFG)
    rng = np.random.default_rng(20)
    hid = rng.normal(size=(5, CFG.d_model))
    toks = rng.integers(0, CFG.vocab, 5)
    g = model.head_forward(w, hid, toks, np.arange(5), _kv(CFG, 1, 64), 0, CFG)
    d = CFG.d_model
    proj = w["head"]["proj"]
    w2 = dict(w, head=dict(w["head"], concat="hidden_first", proj=np.concatenate([proj[:, d:], proj[:, :d]], 1)))
    g2 = model.head_forward(w2, hid, toks, np.arange(5), _kv(CFG, 1, 64), 0, CFG)
    np.testing.assert_allclose(g2, g, rtol=1e-10, atol=1e-12)
    w3 = dict(w, head=dict(w["head"], concat="hidden_first"))      # same matrix, other order: a different function
    g3 = model.head_forward(w3, hid, toks, np.arange(5), _kv(CFG, 1, 64), 0, CFG)
    assert np.abs(g3 - g).max() > 1e-3
