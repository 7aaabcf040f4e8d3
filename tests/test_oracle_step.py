"""Pins for the oracle's draft-then-verify cycle (Sec. 2.2; App. E restart equations)."""
import numpy as np
import pytest
from scipy import stats

from oracle import model, philox, sampler, step
from synth_inputs import ModelConfig, make_weights, make_page_tables, random_prompts
from synth_inputs.weights import perturb_norm_weights

CFG = ModelConfig("t", 2, 64, 4, 2, 16, 96, 50, batch=3, k=3, kv_len_min=0, kv_len_max=0,
                  length_law="prompt", prompt_len=9)


def _setup(cfg=CFG, seed=0, cap=96, rounding=False):
    w = perturb_norm_weights(make_weights(cfg, seed))
    prompts = random_prompts(cfg.batch, cfg.prompt_len, cfg.vocab, seed=1)
    pt, npg = make_page_tables(np.full(cfg.batch, cap), cfg.page_size, seed=7)
    hpt, hnpg = make_page_tables(np.full(cfg.batch, cap), cfg.page_size, seed=8)
    st = step.prefill(w, cfg, prompts, pt, npg, hpt, hnpg, seed=5, round_interface=rounding)
    return w, st, prompts


def test_prefill_state():
    w, st, prompts = _setup()
    for b, s in enumerate(st.seqs):
        assert s.tokens[:-1] == list(prompts[b]) and len(s.pending_tok) == 1
        assert s.kv_len == CFG.prompt_len and s.pending_tok[0] == s.tokens[-1]
    assert st.step == 1


def test_ragged_prefill_equals_each_sequence_alone():
    """Prompts of different lengths: every sequence ends in the state it reaches when prefilled on its own
    (own first token, own pending pair, own cache rows), and the head cache holds pairs 1..P-1 at positions 0..P-2."""
    w = perturb_norm_weights(make_weights(CFG, 0))
    rng = np.random.default_rng(3)
    prompts = [rng.integers(0, CFG.vocab, n) for n in (1, 7, 20)]
    pt, npg = make_page_tables(np.full(3, 64), CFG.page_size, seed=7)
    hpt, hnpg = make_page_tables(np.full(3, 64), CFG.page_size, seed=8)
    st = step.prefill(w, CFG, prompts, pt, npg, hpt, hnpg, seed=5, round_interface=False)
    for b, pr in enumerate(prompts):
        s = st.seqs[b]
        assert s.tokens[:-1] == [int(t) for t in pr] and s.kv_len == len(pr) and len(s.pending_tok) == 1
        kv1 = model.PagedKV(CFG.n_layers, CFG.n_kv_heads, CFG.head_dim, pt[b:b + 1], npg)
        H = model.target_forward(w, pr, np.arange(len(pr)), kv1, 0, CFG)
        np.testing.assert_allclose(s.pending_hidden[0], H[-1], rtol=1e-12)
        p = sampler.softmax_probs(model.target_logits(w, H[-1:], CFG)[0])
        assert s.tokens[-1] == sampler.draw_token(p, philox.u24(5, 0, b, philox.SLOT_FINAL))[0]
        for l in range(CFG.n_layers):
            for a, c in zip(st.kv.gather(l, b, len(pr)), kv1.gather(l, 0, len(pr))):
                np.testing.assert_allclose(a, c, rtol=1e-12)
        if len(pr) > 1:
            hk1 = model.PagedKV(1, CFG.n_kv_heads, CFG.head_dim, hpt[b:b + 1], hnpg)
            model.head_forward(w, H[:-1], pr[1:], np.arange(len(pr) - 1), hk1, 0, CFG)
            for a, c in zip(st.hkv.gather(0, b, len(pr) - 1), hk1.gather(0, 0, len(pr) - 1)):
                np.testing.assert_allclose(a, c, rtol=1e-12)


def test_cycle_invariants_and_restart_cache_composition():
    """After several cycles: every cycle commits between 1 and K+1 tokens; the target cache and the
    head cache BEHIND the boundary equal those of a fresh pass over the committed sequence that
    feeds the head target features only (the restart replaces head-recursive entries)."""
    w, st, _ = _setup()
    K = 3
    lens0 = [len(s.tokens) for s in st.seqs]
    total = 0
    for it in range(6):
        before = [len(s.tokens) for s in st.seqs]
        out = step.spec_step(w, CFG, st, K, seed=5, round_interface=False)
        for b, s in enumerate(st.seqs):
            grown = len(s.tokens) - before[b]
            assert grown == out["accept_len"][b] + 1 and 1 <= grown <= K + 1
            assert s.tokens[before[b]:before[b] + out["accept_len"][b]] == list(out["draft_tok"][b][:out["accept_len"][b]])
            assert s.tokens[-1] == out["next_token"][b] == s.pending_tok[-1]
            assert len(s.pending_tok) == grown and s.pending_hidden.shape == (grown, CFG.d_model)
            total += grown
    assert st.step == 7
    for b, s in enumerate(st.seqs):
        L1 = s.kv_len
        n = len(s.pending_tok)
        pt, npg = make_page_tables(np.full(CFG.batch, 96), CFG.page_size, seed=21)
        kv = model.PagedKV(CFG.n_layers, CFG.n_kv_heads, CFG.head_dim, pt, npg, CFG.page_size)
        hkv = model.PagedKV(1, CFG.n_kv_heads, CFG.head_dim, pt, npg, CFG.page_size)
        H = model.target_forward(w, s.tokens[:L1], np.arange(L1), kv, b, CFG)
        for l in range(CFG.n_layers):
            for x, y in zip(st.kv.gather(l, b, L1), kv.gather(l, b, L1)):
                np.testing.assert_allclose(x, y, rtol=1e-8, atol=1e-10)
        # pending hidden states are the target's features of the last n inputs
        np.testing.assert_allclose(s.pending_hidden, H[L1 - n:], rtol=1e-8, atol=1e-10)
        # head entries 0 .. L1-n-1 come from pairs (H_{i-1}, x_i)
        m = L1 - n
        model.head_forward(w, H[:m], s.tokens[1:m + 1], np.arange(m), hkv, b, CFG)
        for x, y in zip(st.hkv.gather(0, b, m), hkv.gather(0, b, m)):
            np.testing.assert_allclose(x, y, rtol=1e-8, atol=1e-10)


def test_full_acceptance_grows_by_k_plus_one():
    """u = 0 accepts every draft with p > 0: the boundary moves by K+1 and the last token is the
    bonus draw from p_{K+1}."""
    w, st, _ = _setup()
    K, B = 3, CFG.batch
    ua = np.zeros((B, K + 1), np.uint32)
    ua[:, K] = 12345
    before = [len(s.tokens) for s in st.seqs]
    out = step.spec_step(w, CFG, st, K, seed=5, u24_accept=ua, round_interface=False)
    for b, s in enumerate(st.seqs):
        assert out["accept_len"][b] == K and len(s.tokens) == before[b] + K + 1
        assert out["next_token"][b] == sampler.draw_token(out["p"][b][K], 12345)[0]


def test_verify_distributions_condition_on_the_drafts():
    """p_{k+1} of the cycle == the target's next-token distribution after the context extended by
    d_1..d_k, recomputed from scratch (Eq. 2)."""
    w, st, _ = _setup()
    K = 3
    ctx = [list(s.tokens) for s in st.seqs]
    out = step.spec_step(w, CFG, st, K, seed=5, do_commit=False, round_interface=False)
    for b in range(CFG.batch):
        for k in range(K + 1):
            seq = ctx[b] + list(out["draft_tok"][b][:k])
            pt, npg = make_page_tables(np.full(CFG.batch, 96), CFG.page_size, seed=3)
            kv = model.PagedKV(CFG.n_layers, CFG.n_kv_heads, CFG.head_dim, pt, npg, CFG.page_size)
            H = model.target_forward(w, seq, np.arange(len(seq)), kv, b, CFG)
            p = sampler.softmax_probs(model.target_logits(w, H[-1:], CFG)[0])
            np.testing.assert_allclose(out["p"][b][k], p, rtol=1e-5, atol=1e-9)


def test_draft_chain_is_recurrent_on_its_own_state():
    """q_k of the cycle == the head applied k times: first on the target feature, then on its own
    output with the previous draft's embedding (restart equations, first and second line)."""
    w, st, _ = _setup()
    K = 3
    s = st.seqs[1]
    L1 = s.kv_len
    hid, tok = s.pending_hidden.copy(), list(s.pending_tok)
    out = step.spec_step(w, CFG, st, K, seed=5, do_commit=False, round_interface=False)
    d = out["draft_tok"][1]
    # rebuild with a scratch copy of the head cache
    import copy
    hkv = copy.deepcopy(st.hkv)
    g = model.head_forward(w, hid, tok, np.arange(L1 - 1, L1), hkv, 1, CFG)[-1:]
    for k in range(K):
        if k > 0:
            g = model.head_forward(w, g, [d[k - 1]], np.array([L1 + k - 1]), hkv, 1, CFG)
        q = sampler.softmax_probs(model.head_logits(w, g, CFG)[0])
        np.testing.assert_allclose(out["q"][1][k], q, rtol=1e-5, atol=1e-9)
        assert d[k] == sampler.draw_token(q, philox.u24(5, 1, 1, philox.SLOT_DRAFT + k))[0]


def test_uniforms_come_from_the_documented_slots():
    w, st, _ = _setup()
    K = 2
    out_a = step.spec_step(w, CFG, st, K, seed=9, do_commit=False, round_interface=False)
    out_b = step.spec_step(w, CFG, st, K, seed=9, do_commit=False, round_interface=False,
                           u24_draft=philox.u24_draft(9, st.step, CFG.batch, K),
                           u24_accept=philox.u24_accept(9, st.step, CFG.batch, K))
    for key in ("draft_tok", "accept_len", "next_token"):
        np.testing.assert_array_equal(out_a[key], out_b[key])


def test_committed_tokens_follow_the_target_autoregressive_law():
    """End to end on a tiny model (vocab 6): over many seeds the first two tokens committed after
    the prompt are distributed as the target's own autoregressive samples."""
    cfg = ModelConfig("m", 1, 16, 2, 1, 8, 24, 6, batch=1, k=2, kv_len_min=0, kv_len_max=0,
                      length_law="prompt", prompt_len=3)
    w = make_weights(cfg, 3)
    for name in ("embed", "lm_head"):
        w[name] = w[name] * 40.0          # make the distributions far from uniform
    w["head"]["layer"]["wd"] = w["head"]["layer"]["wd"] * 30.0
    prompts = np.array([[1, 4, 2]], np.int32)
    pt, npg = make_page_tables(np.array([32]), cfg.page_size, seed=1)
    N = 6000
    counts = np.zeros((cfg.vocab, cfg.vocab))
    acc = 0
    for seed in range(N):
        st = step.prefill(w, cfg, prompts, pt, npg, pt, npg, seed=seed, round_interface=False)
        st.seqs[0].tokens = st.seqs[0].tokens      # first token drawn from the prefill logits
        while len(st.seqs[0].tokens) < 3 + 3:
            out = step.spec_step(w, cfg, st, 2, seed=seed, round_interface=False)
            acc += out["accept_len"][0]
        t = st.seqs[0].tokens
        counts[t[4], t[5]] += 1                     # two tokens produced by speculative cycles
    # the law of (x4, x5) given the prompt, marginalised over x3 ~ p(.|prompt)
    def nxt(seq):
        kv = model.PagedKV(cfg.n_layers, cfg.n_kv_heads, cfg.head_dim, pt, npg, cfg.page_size)
        H = model.target_forward(w, seq, np.arange(len(seq)), kv, 0, cfg)
        return sampler.softmax_probs(model.target_logits(w, H[-1:], cfg)[0]).astype(np.float64)
    expect = np.zeros_like(counts)
    p3 = nxt([1, 4, 2])
    for x3 in range(cfg.vocab):
        p4 = nxt([1, 4, 2, x3])
        for x4 in range(cfg.vocab):
            expect[x4] += p3[x3] * p4[x4] * nxt([1, 4, 2, x3, x4])
    expect *= N / expect.sum()
    keep = expect.ravel() > 5
    chi, pv = stats.chisquare(counts.ravel()[keep], expect.ravel()[keep] * counts.ravel()[keep].sum() / expect.ravel()[keep].sum())
    assert pv > 1e-4, (chi, pv)
    assert acc > 0.05 * N                          # drafts do get accepted, so the test exercises both branches


def test_forced_drafts_replay_the_recorded_path():
    """Feeding a cycle's own drafts back reproduces it exactly (Eq. 4: the reconstruction consumes the
    recorded drafts and samples nothing); other drafts change q_2.. and p_2.. but not q_1, p_1."""
    w, st, _ = _setup()
    K = 3
    free = step.spec_step(w, CFG, st, K, seed=5, do_commit=False, round_interface=False)
    same = step.spec_step(w, CFG, st, K, seed=5, do_commit=False, round_interface=False,
                          forced_draft=free["draft_tok"])
    for key in ("draft_tok", "accept_len", "next_token"):
        np.testing.assert_array_equal(free[key], same[key])
    np.testing.assert_allclose(free["q"], same["q"], rtol=1e-12)
    other = (free["draft_tok"] + 1) % CFG.vocab
    alt = step.spec_step(w, CFG, st, K, seed=5, do_commit=False, round_interface=False, forced_draft=other)
    np.testing.assert_array_equal(alt["draft_tok"], other)
    np.testing.assert_allclose(alt["q"][:, 0], free["q"][:, 0], rtol=1e-12)
    np.testing.assert_allclose(alt["p"][:, 0], free["p"][:, 0], rtol=1e-12)
    assert np.abs(alt["q"][:, 1] - free["q"][:, 1]).max() > 1e-7
    assert np.abs(alt["p"][:, 1] - free["p"][:, 1]).max() > 1e-7


# ---- whole rollouts: stopping rules -----------------------------------------------------------------------

def test_append_committed_rules():
    r = [5]
    assert step.append_committed(r, [1, 2, 3], eos=9, max_new=10) == step.RUNNING and r == [5, 1, 2, 3]
    assert step.append_committed(r, [4, 9, 7, 7], eos=9, max_new=10) == step.HIT_EOS and r == [5, 1, 2, 3, 4, 9]
    r = [5, 1]
    assert step.append_committed(r, [2, 3, 4], eos=9, max_new=4) == step.HIT_CAP and r == [5, 1, 2, 3]
    assert step.append_committed(r, [8], eos=9, max_new=4) == step.HIT_CAP and r == [5, 1, 2, 3]
    r = []
    assert step.append_committed(r, [9], eos=9, max_new=1) == step.HIT_EOS and r == [9]      # EOS wins on the last slot
    r = []
    assert step.append_committed(r, [3], eos=-1, max_new=1) == step.HIT_CAP and r == [3]


def test_rollout_is_the_concatenation_of_its_cycles_and_rows_are_independent():
    """(a) With no stopping rule a rollout's responses are the committed tokens of plain cycles; (b) with a cap and
    an end-of-sequence token each response is that stream cut by the rules; (c) a row's response does not depend
    on when the other rows stop (rolled out alone it gives the same tokens)."""
    w, st, _ = _setup(cap=160)
    w2, st2, _ = _setup(cap=160)
    resp, status, n = step.rollout(w, CFG, st, 3, seed=5, max_steps=6, eos=-1, max_new=1000, round_interface=False)
    assert n == 6 and status == [step.RUNNING] * CFG.batch
    for b, s in enumerate(st.seqs):
        assert resp[b] == s.tokens[CFG.prompt_len:]
    stream = [list(r) for r in resp]
    eos = stream[0][4]                                   # a token row 0 emits early
    resp2, status2, n2 = step.rollout(w2, CFG, st2, 3, seed=5, max_steps=6, eos=eos, max_new=11, round_interface=False)
    for b in range(CFG.batch):
        want = []
        code = step.append_committed(want, stream[b], eos, 11)
        assert resp2[b] == want and status2[b] == code
    assert status2[0] == step.HIT_EOS and resp2[0][-1] == eos
    assert n2 <= 6 and all(len(r) <= 11 for r in resp2)
    # frozen state of a finished row: its committed tokens stop where its response stopped (up to the dropped tail)
    for b, s in enumerate(st2.seqs):
        assert s.tokens[CFG.prompt_len:CFG.prompt_len + len(resp2[b])] == resp2[b]
