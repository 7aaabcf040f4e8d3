"""Pins for the oracle's head-update forward: draft-path reconstruction (Eq. 4) and the DCA / VGM objective
(Eq. 5-9)."""
import numpy as np
import pytest

from oracle import model, record, sampler, step, update
from synth_inputs import ModelConfig, make_weights, make_page_tables, random_prompts
from synth_inputs.weights import perturb_norm_weights

T = 0.02        # random-init logits are almost flat; a low temperature makes head and target disagree
CFG = ModelConfig("t", 2, 64, 4, 2, 16, 96, 50, batch=3, k=3, kv_len_min=0, kv_len_max=0,
                  length_law="prompt", prompt_len=9)


def _rollout_with_records(rounding, n_steps=5, K=3):
    w = perturb_norm_weights(make_weights(CFG, 0))
    prompts = random_prompts(CFG.batch, CFG.prompt_len, CFG.vocab, seed=1)
    pt, npg = make_page_tables(np.full(CFG.batch, 96), CFG.page_size, seed=7)
    hpt, hnpg = make_page_tables(np.full(CFG.batch, 96), CFG.page_size, seed=8)
    st = step.prefill(w, CFG, prompts, pt, npg, hpt, hnpg, temperature=T, seed=5, round_interface=rounding)
    cycles = []
    for it in range(n_steps):
        lens = [len(s.tokens) for s in st.seqs]
        start_h = [s.pending_hidden[-1].copy() for s in st.seqs]
        out = step.spec_step(w, CFG, st, K, T, seed=5, round_interface=rounding)
        for b in range(CFG.batch):
            rec = record.cycle_record(start_h[b], out["draft_tok"][b], out["target_logits"][b], out["accept_len"][b], lens[b], T)
            cycles.append((b, rec, out["q"][b], out["p"][b]))
    return w, st, cycles


def _sequence_features(w, st, rounding):
    seqs = []
    for s in st.seqs:
        kv = model.PagedKV(CFG.n_layers, CFG.n_kv_heads, CFG.head_dim, np.arange(16)[None, :], 16)
        H = model.target_forward(w, s.tokens[:-1], np.arange(len(s.tokens) - 1), kv, 0, CFG)
        seqs.append((model.round_bf16(H).astype(np.float64) if rounding else H, list(s.tokens)))
    return seqs


def test_reconstruction_reproduces_the_rollouts_head_distributions():
    """Eq. 4 on recorded inputs recomputes exactly the states drafting ran: every q_k of every cycle of a rollout,
    although the rollout's head cache was written incrementally and partly overwritten by rejected chains."""
    w, st, cycles = _rollout_with_records(rounding=False)
    seqs = _sequence_features(w, st, rounding=False)
    assert any(rec["accepted"] <= 3 for _, rec, _, _ in cycles)          # some chains were cut short
    for b, rec, q_roll, _ in cycles:
        q, _ = update.reconstruct_chain(w, CFG, seqs[b][0], seqs[b][1], rec["start_pos"], rec["drafts"], T,
                                        round_interface=False)
        np.testing.assert_allclose(q, q_roll, rtol=1e-6, atol=1e-12)
        # the start hidden of the record is the feature the chain starts from
        np.testing.assert_allclose(rec["start_hidden"], seqs[b][0][rec["start_pos"] - 2], rtol=1e-9, atol=1e-12)


def test_reconstruction_depends_on_the_recorded_drafts_not_on_the_committed_path():
    w, st, cycles = _rollout_with_records(rounding=False)
    seqs = _sequence_features(w, st, rounding=False)
    b, rec, q_roll, _ = next(c for c in cycles if c[1]["accepted"] == 1)   # first draft rejected
    other = (rec["drafts"] + 1) % CFG.vocab
    q2, _ = update.reconstruct_chain(w, CFG, seqs[b][0], seqs[b][1], rec["start_pos"], other, T, round_interface=False)
    np.testing.assert_allclose(q2[0], q_roll[0], rtol=1e-6)                # depth 1 sees no draft
    assert np.abs(q2[1] - q_roll[1]).max() > 1e-4                          # depth 2 is conditioned on d_1
    # feeding the committed continuation instead of the recorded (rejected) draft gives another state
    committed = np.array(seqs[b][1][rec["start_pos"]:rec["start_pos"] + 3])
    assert committed[0] != rec["drafts"][0]
    q3, _ = update.reconstruct_chain(w, CFG, seqs[b][0], seqs[b][1], rec["start_pos"], committed, T, round_interface=False)
    assert np.abs(q3[1] - q_roll[1]).max() > 1e-4


def test_alpha_from_the_record_is_close_to_the_full_overlap_and_bounds_it():
    w, st, cycles = _rollout_with_records(rounding=True)
    for b, rec, q, p in cycles[:6]:
        a = update.chain_alphas(rec, q)
        full = np.array([sampler.acceptance_probability(p[k], q[k]) for k in range(3)])
        # vocabulary 50 < 64 retained entries: the residual bin is empty and the estimate is the overlap itself
        np.testing.assert_allclose(a, full, atol=4e-3)                      # bf16 log-probabilities
        assert (a > 0).all() and (a <= 1 + 1e-3).all()


def test_chain_losses_closed_forms():
    a = np.array([0.9, 0.5, 0.25])
    assert update.tv_chain_loss(a) == pytest.approx(-(0.9 + 0.45 + 0.1125))
    assert update.dca_loss(a) == pytest.approx(-np.log(0.9 + 0.45 + 0.1125))
    assert update.dca_loss(a) == pytest.approx(-np.log(-update.tv_chain_loss(a)))          # Eq. 7 = -log(-L_TV)
    assert update.dca_loss(np.ones(5)) == pytest.approx(-np.log(5.0))
    assert update.dca_loss([0.3]) == pytest.approx(-np.log(0.3))
    # verify-gated masking: chain sum cut at min(j, K); j = 1 keeps the first position only
    assert update.dca_loss(a, j=1) == pytest.approx(-np.log(0.9))
    assert update.dca_loss(a, j=2) == pytest.approx(-np.log(0.9 + 0.45))
    assert update.dca_loss(a, j=3) == update.dca_loss(a, j=4) == update.dca_loss(a)
    assert update.dca_loss([0.0, 0.5]) == float("inf")
    assert np.isfinite(update.dca_loss([0.5, 0.0, 0.7]))


def test_gradient_weights_of_eq8_match_finite_differences():
    rng = np.random.default_rng(4)
    for K in (1, 2, 5, 7):
        a = rng.uniform(0.05, 0.95, K)
        w = update.dca_position_weights(a)
        for k in range(K):
            e = np.zeros(K)
            e[k] = 1e-6
            fd = -(update.dca_loss(a + e) - update.dca_loss(a - e)) / 2e-6
            assert w[k] == pytest.approx(fd, rel=1e-5)
        # the tail term lies in [1, K-k+1] (k counted from 1)
        D = w * (-update.tv_chain_loss(a)) / np.concatenate([[1.0], np.cumprod(a)[:-1]])
        assert (D >= 1 - 1e-12).all() and (D <= K - np.arange(K) + 1e-12).all()
        # gradient of the logarithmic form = gradient of the chain form / M
        for k in range(K):
            e = np.zeros(K)
            e[k] = 1e-6
            fd_tv = -(update.tv_chain_loss(a + e) - update.tv_chain_loss(a - e)) / 2e-6
            assert w[k] == pytest.approx(fd_tv / (-update.tv_chain_loss(a)), rel=1e-5)


def test_head_update_loss_is_the_mean_over_cycles():
    w, st, cycles = _rollout_with_records(rounding=True, n_steps=3)
    seqs = _sequence_features(w, st, rounding=True)
    recs = [(b, rec) for b, rec, _, _ in cycles]
    loss, alphas = update.head_update_loss(w, CFG, seqs, recs, T)
    assert alphas.shape == (len(recs), 3)
    per = [update.dca_loss(alphas[i], recs[i][1]["accepted"]) for i in range(len(recs))]
    assert loss == pytest.approx(np.mean(per))
    # a perfect head (q = p) would give alpha = 1 everywhere and loss -log(min(j, K)) per cycle: the bound
    assert loss >= -np.mean([np.log(min(r["accepted"], 3)) for _, r in recs]) - 1e-9


def _toy_records(rng, n, K, V, kept, T):
    """Records over a small vocabulary: `kept` retained target tokens per position (padded with -1 to 64), the
    rest of the target mass in the residual bin."""
    recs = []
    for _ in range(n):
        p = update.softmax64(rng.normal(0, 2.0, (K + 1, V)), T)
        idx = np.full((K + 1, 64), -1, np.int64)
        lp = np.full((K + 1, 64), -np.inf)
        for k in range(K + 1):
            top = np.argsort(-p[k])[:kept]
            idx[k, :kept], lp[k, :kept] = top, np.log(p[k, top])
        recs.append({"top_index": idx, "top_logprob": lp, "accepted": int(rng.integers(1, K + 2))})
    return recs


def _mean_loss(logits, recs, T):
    per = []
    for r, rec in enumerate(recs):
        a = update.chain_alphas(rec, update.softmax64(logits[r], T))
        per.append(update.dca_loss(a, rec["accepted"]))
    return float(np.mean(per))


def test_truncated_alpha_gradient_matches_finite_differences_and_eq8():
    rng = np.random.default_rng(9)
    for K in (1, 3, 7):
        a = rng.uniform(0.05, 0.95, K)
        np.testing.assert_allclose(update.dca_loss_grad_alpha(a), -update.dca_position_weights(a), rtol=1e-12)
        for j in range(1, K + 2):
            g = update.dca_loss_grad_alpha(a, j)
            for k in range(K):
                e = np.zeros(K)
                e[k] = 1e-6
                fd = (update.dca_loss(a + e, j) - update.dca_loss(a - e, j)) / 2e-6
                assert g[k] == pytest.approx(fd, rel=1e-5, abs=1e-9)
            assert (g[min(j, K):] == 0).all() and (g[:min(j, K)] < 0).all()      # larger overlap, smaller loss


def test_logit_gradient_matches_finite_differences_of_the_objective():
    """The whole chain record -> overlap with residual bin -> truncated log-domain loss -> mean, differentiated
    numerically with respect to every reconstructed logit."""
    rng = np.random.default_rng(3)
    n, K, V, T = 4, 3, 14, 0.7
    for kept in (5, 14):                                     # with a residual bin, and with the whole vocabulary retained
        recs = _toy_records(rng, n, K, V, kept, T)
        logits = rng.normal(0, 2.0, (n, K, V))
        g = update.head_update_grad_logits(logits, recs, T)
        assert np.abs(g.sum(-1)).max() < 1e-12               # softmax: the gradient of a row sums to zero
        fd = np.zeros_like(g)
        for i in np.ndindex(n, K, V):
            e = np.zeros_like(logits)
            e[i] = 1e-6
            fd[i] = (_mean_loss(logits + e, recs, T) - _mean_loss(logits - e, recs, T)) / 2e-6
        np.testing.assert_allclose(g, fd, rtol=2e-5, atol=1e-9)
        for r, rec in enumerate(recs):                       # positions after the first rejection get no gradient
            assert (g[r, min(rec["accepted"], K):] == 0).all() and np.abs(g[r, 0]).max() > 0


def test_rmsnorm_gradient_matches_finite_differences():
    rng = np.random.default_rng(11)
    x, w, dy = rng.normal(0, 1.5, (3, 12)), rng.uniform(0.5, 1.5, 12), rng.normal(0, 1, (3, 12))
    eps = 1e-3                                                 # large enough to matter
    f = lambda xx: float((model.rmsnorm(xx, w, eps) * dy).sum())
    g = update.rmsnorm_grad(dy, x, w, eps)
    for i in np.ndindex(*x.shape):
        e = np.zeros_like(x)
        e[i] = 1e-6
        assert g[i] == pytest.approx((f(x + e) - f(x - e)) / 2e-6, rel=1e-6, abs=1e-9)
    # a row scaled by c has the same normed output (eps aside): the gradient is orthogonal to x when eps = 0
    g0 = update.rmsnorm_grad(dy, x, w, 0.0)
    assert np.abs((g0 * x).sum(-1)).max() < 1e-12


def test_head_state_gradient_matches_finite_differences_of_the_objective():
    """state -> head norm -> shared LM head -> softmax -> overlap with residual bin -> truncated loss -> mean,
    differentiated numerically with respect to every coordinate of every head state."""
    rng = np.random.default_rng(5)
    n, K, V, d, T = 3, 3, 14, 6, 0.8
    cfg = CFG.with_(d_model=d, vocab=V, rms_eps=1e-4)
    w = {"lm_head": rng.normal(0, 0.8, (V, d)), "head": {"final_norm": rng.uniform(0.6, 1.4, d)}}
    for kept in (5, 14):
        recs = _toy_records(rng, n, K, V, kept, T)
        states = rng.normal(0, 1.0, (n, K, d))
        g, gy, logits = update.head_update_grad_state(w, cfg, states, recs, T)
        np.testing.assert_allclose(logits, model.head_logits(w, states.reshape(-1, d), cfg).reshape(n, K, V))
        loss = lambda st: _mean_loss(model.head_logits(w, st.reshape(-1, d), cfg).reshape(n, K, V), recs, T)
        fd = np.zeros_like(g)
        for i in np.ndindex(n, K, d):
            e = np.zeros_like(states)
            e[i] = 1e-6
            fd[i] = (loss(states + e) - loss(states - e)) / 2e-6
        np.testing.assert_allclose(g, fd, rtol=5e-5, atol=1e-9)
        # the LM-head step alone: a matrix product with the untransposed weight (row of logits gradient times W_lm)
        gl = update.head_update_grad_logits(logits, recs, T)
        np.testing.assert_allclose(gy, np.einsum("nkv,vd->nkd", gl, w["lm_head"]), rtol=1e-12)
        for r, rec in enumerate(recs):                       # positions after the first rejection get no gradient
            assert (g[r, min(rec["accepted"], K):] == 0).all()


def test_ffn_block_gradient_matches_finite_differences():
    """L = sum(C * ffn_block(x)) for a random C: every input coordinate and every entry of the four parameter tensors,
    against central differences of the forward function the decoder layer itself calls."""
    rng = np.random.default_rng(21)
    T_, d, F = 3, 6, 5
    cfg = CFG.with_(d_model=d, d_ffn=F, rms_eps=1e-3)
    lw = {"ln2": rng.uniform(0.6, 1.4, d), "wg": rng.normal(0, 0.7, (F, d)), "wu": rng.normal(0, 0.7, (F, d)),
          "wd": rng.normal(0, 0.7, (d, F))}
    x, C = rng.normal(0, 1.2, (T_, d)), rng.normal(0, 1, (T_, d))
    g = update.ffn_block_grad(C, x, lw, cfg.rms_eps)

    def fd(get, put, shape):
        out = np.zeros(shape)
        for i in np.ndindex(*shape):
            v = get()[i]
            put(i, v + 1e-6); hi = float((model.ffn_block(lw, x, cfg) * C).sum())
            put(i, v - 1e-6); lo = float((model.ffn_block(lw, x, cfg) * C).sum())
            put(i, v)
            out[i] = (hi - lo) / 2e-6
        return out

    def setter(arr):
        def put(i, v):
            arr[i] = v
        return put

    np.testing.assert_allclose(g["dx"], fd(lambda: x, setter(x), x.shape), rtol=2e-6, atol=1e-8)
    for name, key in (("dln2", "ln2"), ("dwg", "wg"), ("dwu", "wu"), ("dwd", "wd")):
        np.testing.assert_allclose(g[name], fd(lambda: lw[key], setter(lw[key]), lw[key].shape), rtol=2e-6, atol=1e-8)
    # the residual path alone: with a zero down projection the block is the identity and so is its backward
    lw0 = dict(lw, wd=np.zeros((d, F)))
    g0 = update.ffn_block_grad(C, x, lw0, cfg.rms_eps)
    np.testing.assert_array_equal(g0["dx"], C)
    assert np.abs(g0["dwg"]).max() == 0 and np.abs(g0["dln2"]).max() == 0 and np.abs(g0["dwd"]).max() > 0


def test_adamw_step_matches_the_library_optimizer_and_its_closed_forms():
    import torch
    rng = np.random.default_rng(8)
    p0 = rng.normal(0, 1, 37)
    grads = [rng.normal(0, 0.3, 37) for _ in range(6)]
    lr, wd = 3e-4, 0.01
    tp = torch.nn.Parameter(torch.tensor(p0, dtype=torch.float64))
    opt = torch.optim.AdamW([tp], lr=lr, betas=(0.9, 0.999), eps=1e-8, weight_decay=wd)
    p, m, v = p0.copy(), np.zeros(37), np.zeros(37)
    for t, g in enumerate(grads, start=1):
        tp.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        p, m, v = update.adamw_step(p, g, m, v, t, lr, weight_decay=wd)
        np.testing.assert_allclose(p, tp.detach().numpy(), rtol=1e-13, atol=1e-15)
    # first step from zero moments: the bias corrections give m_hat = g, v_hat = g^2, so the move is lr g / (|g| + eps)
    g = grads[0]
    p1, _, _ = update.adamw_step(p0, g, np.zeros(37), np.zeros(37), 1, lr, weight_decay=0.0)
    np.testing.assert_allclose(p0 - p1, lr * g / (np.abs(g) + 1e-8), rtol=1e-12)
    # weight decay alone (zero gradient, zero moments): a plain shrink of the parameter
    p2, m2, v2 = update.adamw_step(p0, np.zeros(37), np.zeros(37), np.zeros(37), 1, lr, weight_decay=wd)
    np.testing.assert_allclose(p2, p0 * (1 - lr * wd), rtol=1e-15)
    assert not m2.any() and not v2.any()
    # a common positive factor on the whole gradient history leaves the step unchanged up to eps (App. on SGD vs Adam)
    pa, ma, va = p0.copy(), np.zeros(37), np.zeros(37)
    pb, mb, vb = p0.copy(), np.zeros(37), np.zeros(37)
    for t, g in enumerate(grads, start=1):
        pa, ma, va = update.adamw_step(pa, g, ma, va, t, lr, eps=0.0, weight_decay=0.0)
        pb, mb, vb = update.adamw_step(pb, 7.5 * g, mb, vb, t, lr, eps=0.0, weight_decay=0.0)
    np.testing.assert_allclose(pa, pb, rtol=1e-12)


def test_head_learning_rate_schedule():
    peak, total = 3e-4, 200
    lrs = np.array([update.head_lr(s, peak, total) for s in range(total + 5)])
    assert lrs[0] == pytest.approx(peak / 10) and lrs[9] == pytest.approx(peak)          # warm-up over 10 steps
    assert np.all(np.diff(lrs[:10]) > 0) and np.allclose(np.diff(lrs[:10]), peak / 10)
    assert lrs[10] == pytest.approx(peak) and np.all(np.diff(lrs[10:total + 1]) <= 1e-18)  # then it only decays
    assert lrs[total] == pytest.approx(peak / 10) and lrs[total + 4] == pytest.approx(peak / 10)   # to a tenth of the peak
    mid = (10 + total) // 2
    assert lrs[mid] == pytest.approx(peak * 0.55, rel=1e-9)                               # half-way down the cosine


@pytest.mark.parametrize("concat", ["embedding_first", "hidden_first"])
def test_head_input_gradient_matches_finite_differences(concat):
    """L = sum(C * head_input(hidden, tokens)): every coordinate of the hidden states, every entry of the projection and of
    the two norm weights, against central differences of the function head_forward itself calls; both concatenation orders."""
    rng = np.random.default_rng(31)
    T_, d, V = 4, 5, 9
    cfg = CFG.with_(d_model=d, vocab=V, rms_eps=1e-3)
    w = {"embed": rng.normal(0, 1, (V, d)),
         "head": {"enorm": rng.uniform(0.6, 1.4, d), "hnorm": rng.uniform(0.6, 1.4, d), "proj": rng.normal(0, 0.6, (d, 2 * d)),
                  "concat": concat}}
    hidden, tokens, C = rng.normal(0, 1.3, (T_, d)), np.array([3, 0, 8, 3]), rng.normal(0, 1, (T_, d))
    g = update.head_input_grad(C, w, hidden, tokens, cfg)
    L = lambda: float((model.head_input(w, hidden, tokens, cfg) * C).sum())

    def fd(arr):
        out = np.zeros(arr.shape)
        for i in np.ndindex(*arr.shape):
            v = arr[i]
            arr[i] = v + 1e-6; hi = L()
            arr[i] = v - 1e-6; lo = L()
            arr[i] = v
            out[i] = (hi - lo) / 2e-6
        return out

    np.testing.assert_allclose(g["dhidden"], fd(hidden), rtol=2e-6, atol=1e-8)
    np.testing.assert_allclose(g["dproj"], fd(w["head"]["proj"]), rtol=2e-6, atol=1e-8)
    np.testing.assert_allclose(g["denorm"], fd(w["head"]["enorm"]), rtol=2e-6, atol=1e-8)
    np.testing.assert_allclose(g["dhnorm"], fd(w["head"]["hnorm"]), rtol=2e-6, atol=1e-8)
    # the embedding half of the projection sees the token, the hidden half does not: swapping two tokens' rows of C and of
    # the embedding-side inputs only permutes contributions - checked through the column halves of dproj
    half = slice(d, 2 * d) if concat == "hidden_first" else slice(0, d)
    e_n = model.rmsnorm(w["embed"][tokens], w["head"]["enorm"], cfg.rms_eps)
    np.testing.assert_allclose(g["dproj"][:, half], C.T @ e_n, rtol=1e-12)


def test_attention_gradient_matches_finite_differences():
    """L = sum(C * attention(q, k, v)) with a ragged causal mask (queries in the middle of the key range, a key nobody sees):
    every coordinate of q, k and v against central differences of the forward the decoder layer calls."""
    rng = np.random.default_rng(41)
    T_, S, n_q, n_kv, hd = 3, 7, 4, 2, 6
    q, k, v = rng.normal(0, 1, (T_, n_q, hd)), rng.normal(0, 1, (S, n_kv, hd)), rng.normal(0, 1, (S, n_kv, hd))
    q_pos, k_pos = np.array([2, 4, 5]), np.array([0, 1, 2, 3, 4, 5, 9])          # key 6 (position 9) is visible to nobody
    C = rng.normal(0, 1, (T_, n_q, hd))
    dq, dk, dv = update.attention_grad(C, q, k, v, q_pos, k_pos)
    L = lambda: float((model.attention(q, k, v, q_pos, k_pos) * C).sum())

    def fd(arr):
        out = np.zeros(arr.shape)
        for i in np.ndindex(*arr.shape):
            x = arr[i]
            arr[i] = x + 1e-6; hi = L()
            arr[i] = x - 1e-6; lo = L()
            arr[i] = x
            out[i] = (hi - lo) / 2e-6
        return out

    np.testing.assert_allclose(dq, fd(q), rtol=2e-6, atol=1e-8)
    np.testing.assert_allclose(dk, fd(k), rtol=2e-6, atol=1e-8)
    np.testing.assert_allclose(dv, fd(v), rtol=2e-6, atol=1e-8)
    assert not dk[6].any() and not dv[6].any()                       # the invisible key gets nothing
    # a row's score gradients sum to zero over its keys (softmax ignores a common shift), and dk_j = dS_j q / sqrt(hd):
    # the key gradients of a KV head sum to zero over the keys
    assert np.abs(dk.sum(axis=0)).max() < 1e-12
    # values enter linearly: dv is the attention-weighted sum of the output gradients, so it sums to the sum of dout per group
    np.testing.assert_allclose(dv.sum(axis=0), C.reshape(T_, n_kv, n_q // n_kv, hd).sum(axis=(0, 2)), rtol=1e-12)


def test_rope_gradient_is_the_inverse_rotation():
    rng = np.random.default_rng(43)
    x, C = rng.normal(0, 1, (3, 2, 8)), rng.normal(0, 1, (3, 2, 8))
    pos = np.array([0, 5, 17])
    g = update.rope_grad(C, pos, 1.0e4)
    for i in [(0, 0, 1), (1, 1, 2), (2, 0, 6), (1, 0, 7)]:
        e = np.zeros(x.shape)
        e[i] = 1e-6
        fd = ((model.rope(x + e, pos, 1.0e4) - model.rope(x - e, pos, 1.0e4)) * C).sum() / 2e-6
        assert g[i] == pytest.approx(fd, rel=1e-7, abs=1e-10)
    np.testing.assert_allclose(update.rope_grad(model.rope(x, pos, 1.0e4), pos, 1.0e4), x, atol=1e-12)   # orthogonal
    np.testing.assert_allclose(g[0], C[0], atol=1e-15)                                                    # position 0: identity


def _flat_params(w):
    """(name, array) of every head parameter, views into w (float64 copies installed in place)."""
    hw = w["head"]
    out = []
    for name in ("proj", "enorm", "hnorm", "final_norm"):
        hw[name] = np.array(hw[name], np.float64)
        out.append((name, hw[name]))
    for name in sorted(hw["layer"]):
        hw["layer"][name] = np.array(hw["layer"][name], np.float64)
        out.append(("layer." + name, hw["layer"][name]))
    return out


@pytest.mark.parametrize("family", ["plain", "qkv_bias", "qk_norm"])
def test_head_update_gradient_matches_finite_differences_of_the_objective(family):
    """Every parameter tensor of the head: sampled coordinates and one random direction over all of them against
    central differences of head_update_loss - which goes through the prefix pass, the recurrence over the drafts, the
    shared cache entries, the logits and Eq. 9; any missing path (a state's second term, a cache entry's later readers,
    a norm's weight) changes these numbers."""
    import dataclasses
    global CFG
    keep = CFG
    CFG = dataclasses.replace(CFG, qkv_bias=family == "qkv_bias", qk_norm=family == "qk_norm")
    try:
        w, st, cycles = _rollout_with_records(rounding=False, n_steps=2)
        seqs = _sequence_features(w, st, rounding=False)
        cfg = CFG
    finally:
        CFG = keep
    recs = [(b, dict(rec, accepted=i % 4 + 1)) for i, (b, rec, _, _) in enumerate(cycles)]   # every cut of Eq. 9: j = 1 .. K + 1
    params = _flat_params(w)
    grad = update.head_update_grad(w, cfg, seqs, recs, T)

    def loss():
        """head_update_loss without the fp32 rounding of q (which would drown a 1e-6 step): same states, same logits,
        same objective, every step in float64."""
        per = []
        for s_, rec in recs:
            g = update.reconstruct_states(w, cfg, seqs[s_][0], seqs[s_][1], rec["start_pos"], rec["drafts"])
            q = update.softmax64(model.head_logits(w, g, cfg), T)
            per.append(update.dca_loss(update.chain_alphas(rec, q), rec["accepted"]))
        return float(np.mean(per))

    assert loss() == pytest.approx(update.head_update_loss(w, cfg, seqs, recs, T, round_interface=False)[0], rel=1e-5)
    names = {n for n, _ in params}
    assert {"layer." + n for n in grad["layer"]} | (set(grad) - {"layer"}) == names
    rng = np.random.default_rng(47)
    for name, arr in params:
        g = grad["layer"][name[6:]] if name.startswith("layer.") else grad[name]
        assert g.shape == arr.shape
        scale = np.abs(g).max()
        assert scale > 0
        for _ in range(3):
            i = tuple(rng.integers(0, n) for n in arr.shape)
            x = arr[i]
            h = 1e-4 * max(1.0, abs(x))                 # the loss carries ~1e-12 of rounding noise: not smaller
            arr[i] = x + h; hi = loss()
            arr[i] = x - h; lo = loss()
            arr[i] = x
            assert g[i] == pytest.approx((hi - lo) / (2 * h), rel=5e-4, abs=1e-5 * scale), (name, i)
    # one random direction over all parameters at once
    dirs = [rng.normal(0, 1, a.shape) * np.abs(a).mean() for _, a in params]
    expect = sum(float(((grad["layer"][n[6:]] if n.startswith("layer.") else grad[n]) * d).sum()) for (n, _), d in zip(params, dirs))
    h = 1e-6
    for (_, a), d in zip(params, dirs):
        a += h * d
    hi = loss()
    for (_, a), d in zip(params, dirs):
        a -= 2 * h * d
    lo = loss()
    for (_, a), d in zip(params, dirs):
        a += h * d
    assert expect == pytest.approx((hi - lo) / (2 * h), rel=2e-4)


def test_head_update_gradient_with_given_logit_gradients_is_the_same_chain():
    """Handing head_update_grad the objective's own logit gradients reproduces the default; the result is linear in them."""
    w, st, cycles = _rollout_with_records(rounding=False, n_steps=2)
    seqs = _sequence_features(w, st, rounding=False)
    recs = [(b, dict(rec, accepted=i % 4 + 1)) for i, (b, rec, _, _) in enumerate(cycles)]
    base = update.head_update_grad(w, CFG, seqs, recs, T)
    lgs = np.array([update.reconstruct_chain(w, CFG, seqs[b][0], seqs[b][1], r["start_pos"], r["drafts"], T, False)[1] for b, r in recs])
    gl = update.head_update_grad_logits(lgs, [r for _, r in recs], T)
    same = update.head_update_grad(w, CFG, seqs, recs, T, grad_logits=gl)
    twice = update.head_update_grad(w, CFG, seqs, recs, T, grad_logits=2 * gl)
    for name in ("proj", "final_norm"):
        np.testing.assert_allclose(same[name], base[name], rtol=1e-9, atol=1e-14)
        np.testing.assert_allclose(twice[name], 2 * base[name], rtol=1e-9, atol=1e-14)
    for name in base["layer"]:
        np.testing.assert_allclose(same["layer"][name], base["layer"][name], rtol=1e-9, atol=1e-14)
