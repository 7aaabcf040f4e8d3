"""Whole speculative step on the Tiny configuration: CUDA library vs the oracle, from a common state."""
import numpy as np
import pytest
import torch

from oracle import philox, sampler as osampler, step as ostep
from synth_inputs import get_config

from helpers import (accept_bit_is_threshold_case, band, draw_is_threshold_case, push_state, rel_err, softmax64,
                     tiny_setup)

pytestmark = pytest.mark.gpu

TOL = 2e-2      # per-tensor normalised max error for bf16-path logits and hidden states


def _bufs(B, K, V, d):
    dev = "cuda"
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=dev)
    return dict(draft_tok=z((B, K), torch.int32), draft_logits=z((B, K, V), torch.bfloat16),
                tgt_logits=z((B, K + 1, V), torch.bfloat16), tgt_hidden=z((B, K + 1, d), torch.bfloat16),
                dbg_q=z((B, K, V), torch.float32), dbg_p=z((B, K + 1, V), torch.float32),
                dbg_q2=z((B, K, V), torch.float32), a=z((B,), torch.int32), t=z((B,), torch.int32))


def _run_phases(gmb, ctx, gst, K, seed, step, bufs, commit=False):
    B = gst.batch
    gmb.gm_draft(ctx, gst, K, 1.0, None, seed, step, bufs["draft_tok"], bufs["draft_logits"], bufs["dbg_q"])
    gmb.gm_verify(ctx, gst, K, bufs["draft_tok"], bufs["tgt_logits"], bufs["tgt_hidden"])
    gmb.gm_accept(ctx, gst, B, K, 1.0, bufs["tgt_logits"], bufs["draft_logits"], bufs["draft_tok"], None, seed, step,
                  bufs["a"], bufs["t"], bufs["dbg_p"], bufs["dbg_q2"], bufs["tgt_hidden"], commit_state=commit)
    assert gmb.gm_last_status(ctx) == 0


def _parity_from_common_state(cfg, flags, n_steps, concat=None, top_p=1.0):
    import paper_2609_16648_b200 as gmb
    K, B, V, d = cfg.k, cfg.batch, cfg.vocab, cfg.d_model
    w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=cfg.prompt_len + n_steps * (K + 1) + 8, flags=flags, concat=concat)
    gmb.gm_set_top_p(ctx, top_p)
    bufs = _bufs(B, K, V, d)
    seed = 5
    bit_agree = bit_total = tok_same = tok_total = fin_same = fin_total = explained = 0
    worst = 0.0
    for it in range(n_steps):
        push_state(ost, gst, ctx)
        step = ost.step
        _run_phases(gmb, ctx, gst, K, seed, step, bufs)
        g_dtok = bufs["draft_tok"].cpu().numpy()
        g_q = bufs["dbg_q"].cpu().numpy()
        ud, ua = philox.u24_draft(seed, step, B, K), philox.u24_accept(seed, step, B, K)
        for b in range(B):
            for k in range(K):
                assert g_dtok[b, k] == osampler.draw_token(g_q[b, k], ud[b, k])[0]
        assert torch.equal(bufs["dbg_q"], bufs["dbg_q2"])
        p, q = bufs["dbg_p"].cpu().numpy(), bufs["dbg_q2"].cpu().numpy()
        ga, gt = bufs["a"].cpu().numpy(), bufs["t"].cpu().numpy()
        for b in range(B):
            ea, et, _ = osampler.decide(p[b], q[b], g_dtok[b], ua[b])
            assert (ea, et) == (int(ga[b]), int(gt[b]))
        # (2) replay of the device's drafts through the oracle
        ref = ostep.spec_step(w, cfg, ost, K, 1.0, seed=seed, do_commit=False, forced_draft=g_dtok, top_p=top_p)
        worst = max(worst,
                    rel_err(bufs["draft_logits"].float().cpu().numpy(), ref["draft_logits"]),
                    rel_err(bufs["tgt_logits"].float().cpu().numpy(), ref["target_logits"]),
                    rel_err(bufs["tgt_hidden"].float().cpu().numpy(), ref["target_hidden"]))
        for j in range(K + 1):
            worst = max(worst, rel_err(bufs["tgt_logits"][:, j].float().cpu().numpy(), ref["target_logits"][:, j]))
        dev_dl = bufs["draft_logits"].float().cpu().numpy().astype(np.float64)
        dev_tl = bufs["tgt_logits"].float().cpu().numpy().astype(np.float64)
        for b in range(B):
            both = min(ga[b], ref["accept_len"][b])                 # positions 0..both-1 accepted by both
            n_eval = min(both + 1, K)                                # ... and the next one is evaluated by both
            bit_total += n_eval
            bit_agree += both + (1 if (both < K and ga[b] == ref["accept_len"][b]) else 0)
            if ga[b] != ref["accept_len"][b] and top_p >= 1.0:
                # the first position where the bits differ: the oracle's margin must lie inside the band its logit
                # rows' measured errors allow
                k = int(both)
                eps_p = np.abs(dev_tl[b, k] - ref["target_logits"][b, k]).max()
                eps_q = np.abs(dev_dl[b, k] - ref["draft_logits"][b, k]).max()
                d = int(g_dtok[b, k])
                assert accept_bit_is_threshold_case(softmax64(ref["target_logits"][b, k])[d],
                                                    softmax64(ref["draft_logits"][b, k])[d], int(ua[b, k]), eps_p, eps_q), \
                    ("accept bit differs outside the rounding band", it, b, k)
                explained += 1
            if ga[b] == ref["accept_len"][b]:
                fin_total += 1
                fin_same += int(gt[b] == ref["next_token"][b])
                if gt[b] != ref["next_token"][b] and top_p >= 1.0:
                    a_ = int(ga[b])
                    p_or = softmax64(ref["target_logits"][b, a_])
                    eps_p = np.abs(dev_tl[b, a_] - ref["target_logits"][b, a_]).max()
                    if a_ < K:                               # residual max(0, p - q), normalised by its own mass
                        q_or = softmax64(ref["draft_logits"][b, a_])
                        eps_q = np.abs(dev_dl[b, a_] - ref["draft_logits"][b, a_]).max()
                        w_or = np.maximum(p_or - q_or, 0.0)
                        delta = 2.0 * (band(eps_p) + band(eps_q)) / w_or.sum()
                    else:                                    # all drafts accepted: the extra token comes from p
                        w_or, delta = p_or, band(eps_p)
                    assert draw_is_threshold_case(w_or, int(ua[b, K]), int(gt[b]), int(ref["next_token"][b]), delta), \
                        ("final token differs outside the rounding band", it, b, a_)
                    explained += 1
        # (3) free-running oracle from the same state and uniforms
        free = ostep.spec_step(w, cfg, ost, K, 1.0, seed=seed, do_commit=True, top_p=top_p)
        tok_total += B
        tok_same += int((g_dtok[:, 0] == free["draft_tok"][:, 0]).sum())
        for b in range(B):
            if g_dtok[b, 0] != free["draft_tok"][b, 0]:       # same state, same uniform, different first draft
                eps_q = np.abs(dev_dl[b, 0] - free["draft_logits"][b, 0]).max()
                assert draw_is_threshold_case(softmax64(free["draft_logits"][b, 0]), int(ud[b, 0]), int(g_dtok[b, 0]),
                                              int(free["draft_tok"][b, 0]), band(eps_q)), \
                    ("first draft token differs outside the rounding band", it, b)
                explained += 1
    ctx.close()
    print(f"worst rel err {worst:.3e}; accept bits {bit_agree}/{bit_total}; first draft token {tok_same}/{tok_total}; "
          f"final token {fin_same}/{fin_total}; disagreements shown to be threshold cases: {explained}")
    return worst, (bit_agree, bit_total), (tok_same, tok_total), (fin_same, fin_total)


@pytest.mark.parametrize("flags,chain", [(1, None), (0, "0"), (0, "1"), (0, "2")],
                         ids=["mma_sync_gemm", "tcgen05_gemm_separate_launches", "tcgen05_gemm", "tcgen05_gemm_whole_chain"])
def test_tiny_step_parity_from_common_state(flags, chain, monkeypatch):
    """Every step starts from the oracle's state.
    (1) the device's draft draws and accept/resample decisions equal the oracle's decision function on the
        device's own probabilities, bit for bit;
    (2) with the device's drafts fed back to the oracle (the recorded-path replay of Eq. 4), every logit row
        and hidden state agrees within 2e-2 and the accept bits agree on >= 99.5 % of the positions both
        sides evaluate;
    (3) free-running (each side sampling its own drafts from the same uniforms) the sampled tokens agree on
        most positions (an inverse-CDF draw turns a relative logit error e into a disagreement probability of
        order e * sqrt(V)), and EVERY disagreement - a first draft token, an accept bit, a final token - must be a
        threshold case: the oracle's own quantile / margin lies within the band that the measured error of that
        logit row allows (helpers.band).  A wrong index or a swapped row does not fit that band; rounding does.
    The tcgen05 path is run three ways (GM_CHAIN_MODE, read when the context is created): every projection a launch of
    its own; the default (the wide gate/up projection on the persistent-pair kernel); and a layer's output projection,
    gate/up, down and the next QKV projection as one persistent launch with the norms folded in."""
    if chain is not None:
        monkeypatch.setenv("GM_CHAIN_MODE", chain)
    cfg = get_config("tiny").with_(prompt_len=40)
    worst, bits, toks, fins = _parity_from_common_state(cfg, flags, n_steps=24)
    assert worst < TOL, worst
    assert bits[0] / bits[1] >= 0.995, bits
    assert toks[0] / toks[1] >= 0.85, toks
    assert fins[0] / max(fins[1], 1) >= 0.85, fins


@pytest.mark.parametrize("extras", [dict(qkv_bias=True), dict(qk_norm=True),
                                    dict(qkv_bias=True, qk_norm=True, concat="hidden_first"),
                                    dict(qkv_bias=True, qk_norm=True, n_q_heads=2, n_kv_heads=1, head_dim=128),
                                    dict(k=7), dict(k=1), dict(top_p=0.7),
                                    dict(k=5, n_q_heads=8, n_kv_heads=2, head_dim=128),
                                    dict(k=7, n_q_heads=8, n_kv_heads=2, head_dim=128),
                                    dict(qkv_bias=True, qk_norm=True, fused_rope=True),
                                    dict(qkv_bias=True, qk_norm=True, n_q_heads=2, n_kv_heads=1, head_dim=128, fused_rope=True)],
                         ids=["qkv_bias", "qk_norm", "bias_norm_hidden_first", "bias_norm_head128", "depth7", "depth1",
                              "top_p_0.7", "depth5_group4_24_rows", "depth7_group4_32_rows", "fused_rope_head64",
                              "fused_rope_head128"])
def test_tiny_step_parity_variants(extras, monkeypatch):
    """The same bars for the other operating points of the cycle: the decoder-layer families of App. B.1
    (projection bias; query/key head norms), a head that concatenates [hidden ; embedding], and the
    smallest and largest drafting depth, the evaluation's nucleus sampling of the target, and the fused QKV epilogue."""
    extras = dict(extras)
    concat = extras.pop("concat", None)
    top_p = extras.pop("top_p", 1.0)
    if extras.pop("fused_rope", False):       # the option that runs the rotary embedding and the KV append in the QKV epilogue
        monkeypatch.setenv("GM_FUSED_ROPE", "1")
    cfg = get_config("tiny").with_(prompt_len=40, **extras)
    worst, bits, toks, fins = _parity_from_common_state(cfg, 0, n_steps=10, concat=concat, top_p=top_p)
    assert worst < TOL, worst
    assert bits[0] / bits[1] >= 0.995, bits
    assert toks[0] / toks[1] >= 0.8, toks


def test_spec_step_equals_three_calls_and_commits_state():
    """gm_spec_step == gm_draft; gm_verify; gm_accept(commit) bit for bit, and the committed state follows
    the cycle's rules (kv_len += a+1, pending pairs = accepted drafts + final token with their hiddens)."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(prompt_len=33)
    K, B, V, d = cfg.k, cfg.batch, cfg.vocab, cfg.d_model
    w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=160)
    bufs = _bufs(B, K, V, d)
    seed = 11
    push_state(ost, gst, ctx)
    snap = {n: getattr(gst, n).clone() for n in ("kv_len", "pending_n", "pending_tok", "pending_hidden", "kv_pool",
                                                   "head_kv_pool")}
    hist_a = []
    for it in range(6):
        _run_phases(gmb, ctx, gst, K, seed, 100 + it, bufs, commit=True)
        a, t = bufs["a"].cpu().numpy(), bufs["t"].cpu().numpy()
        hist_a.append((a.copy(), t.copy(), bufs["draft_tok"].cpu().numpy().copy()))
        kv_prev = snap["kv_len"].cpu().numpy() if it == 0 else kv_after
        kv_after = gst.kv_len.cpu().numpy()
        np.testing.assert_array_equal(kv_after, kv_prev + a + 1)
        np.testing.assert_array_equal(gst.pending_n.cpu().numpy(), a + 1)
        pt, ph = gst.pending_tok.cpu().numpy(), gst.pending_hidden.float().cpu().numpy()
        th = bufs["tgt_hidden"].float().cpu().numpy()
        for b in range(B):
            np.testing.assert_array_equal(pt[b, :a[b]], hist_a[-1][2][b, :a[b]])
            assert pt[b, a[b]] == t[b]
            np.testing.assert_array_equal(ph[b, :a[b] + 1], th[b, :a[b] + 1])
    final = {n: getattr(gst, n).clone() for n in snap}
    # replay with the fused call
    for n, v in snap.items():
        getattr(gst, n).copy_(v)
    a2, t2 = torch.zeros_like(bufs["a"]), torch.zeros_like(bufs["t"])
    dt2 = torch.zeros_like(bufs["draft_tok"])
    for it in range(6):
        gmb.gm_spec_step(ctx, gst, K, 1.0, seed, 100 + it, a2, t2, dt2)
        np.testing.assert_array_equal(a2.cpu().numpy(), hist_a[it][0])
        np.testing.assert_array_equal(t2.cpu().numpy(), hist_a[it][1])
        np.testing.assert_array_equal(dt2.cpu().numpy(), hist_a[it][2])
    assert gmb.gm_last_status(ctx) == 0
    for n, v in final.items():
        assert torch.equal(getattr(gst, n), v), n
    # host-buffer form
    for n, v in snap.items():
        getattr(gst, n).copy_(v)
    ah = torch.zeros(B, dtype=torch.int32).pin_memory()
    th_ = torch.zeros(B, dtype=torch.int32).pin_memory()
    gmb.gm_spec_step_host(ctx, gst, K, 1.0, seed, 100, ah, th_)
    np.testing.assert_array_equal(ah.numpy(), hist_a[0][0])
    np.testing.assert_array_equal(th_.numpy(), hist_a[0][1])
    ctx.close()


def test_free_running_rollout_keeps_caches_consistent():
    """Let the device run many committed cycles on its own, then check its caches against an oracle
    recomputation of the committed sequence: target KV everywhere, head KV behind the boundary."""
    import paper_2609_16648_b200 as gmb
    from oracle import model as omodel
    cfg = get_config("tiny").with_(prompt_len=20)
    K, B = cfg.k, cfg.batch
    w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=200)
    push_state(ost, gst, ctx)
    a = torch.zeros(B, dtype=torch.int32, device="cuda")
    t = torch.zeros(B, dtype=torch.int32, device="cuda")
    dt = torch.zeros((B, K), dtype=torch.int32, device="cuda")
    seqs = [list(s.tokens) for s in ost.seqs]
    n_acc = 0
    for it in range(30):
        gmb.gm_spec_step(ctx, gst, K, 1.0, 77, it, a, t, dt)
        an, tn, dn = a.cpu().numpy(), t.cpu().numpy(), dt.cpu().numpy()
        for b in range(B):
            seqs[b] += [int(x) for x in dn[b, :an[b]]] + [int(tn[b])]
            n_acc += an[b]
    assert gmb.gm_last_status(ctx) == 0
    kv_len = gst.kv_len.cpu().numpy()
    pool = gst.kv_pool.float().cpu().numpy()
    hpool = gst.head_kv_pool.float().cpu().numpy()
    pn = gst.pending_n.cpu().numpy()
    assert n_acc > 0
    for b in range(B):
        assert kv_len[b] == len(seqs[b]) - 1
        L1 = int(kv_len[b])
        kv = omodel.PagedKV(cfg.n_layers, cfg.n_kv_heads, cfg.head_dim, ost.kv.table, ost.kv.pool.shape[2])
        H = omodel.target_forward(w, seqs[b][:L1], np.arange(L1), kv, b, cfg)
        dev_kv = omodel.PagedKV(cfg.n_layers, cfg.n_kv_heads, cfg.head_dim, ost.kv.table, ost.kv.pool.shape[2])
        dev_kv.pool = pool.astype(np.float64)
        for l in range(cfg.n_layers):
            for x, y in zip(dev_kv.gather(l, b, L1), kv.gather(l, b, L1)):
                assert rel_err(x, y) < TOL
        m = L1 - int(pn[b])
        hkv = omodel.PagedKV(1, cfg.n_kv_heads, cfg.head_dim, ost.hkv.table, ost.hkv.pool.shape[2])
        omodel.head_forward(w, H[:m], seqs[b][1:m + 1], np.arange(m), hkv, b, cfg)
        dev_h = omodel.PagedKV(1, cfg.n_kv_heads, cfg.head_dim, ost.hkv.table, ost.hkv.pool.shape[2])
        dev_h.pool = hpool.astype(np.float64)
        for x, y in zip(dev_h.gather(0, b, m), hkv.gather(0, b, m)):
            assert rel_err(x, y) < TOL
    ctx.close()


def test_an_expired_device_side_wait_is_reported_and_the_context_stays_usable():
    """Failure detection without a GPU fault: a bounded wait that runs out (a barrier nothing arrives on, 1024 polls)
    sets the status word, the kernel returns normally, the host reads GM_ERR_DEVICE_TIMEOUT once, and the next cycle
    on the same context is clean and equals the cycle of a context that never saw the timeout."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(prompt_len=24)
    K, B = cfg.k, cfg.batch
    outs = []
    for inject in (True, False):
        w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=64)
        push_state(ost, gst, ctx)
        a = torch.zeros(B, dtype=torch.int32, device="cuda")
        t = torch.zeros(B, dtype=torch.int32, device="cuda")
        d = torch.zeros((B, K), dtype=torch.int32, device="cuda")
        if inject:
            gmb.gm_selftest_wait_expiry(ctx)
            assert gmb.gm_last_status(ctx) == gmb.GM_ERR_DEVICE_TIMEOUT
            assert gmb.gm_strerror(gmb.GM_ERR_DEVICE_TIMEOUT) == "a bounded device-side wait expired"
            assert gmb.gm_last_status(ctx) == 0                      # sticky until read, then cleared
        gmb.gm_spec_step(ctx, gst, K, 1.0, 7, 0, a, t, d)
        assert gmb.gm_last_status(ctx) == 0
        outs.append((a.clone(), t.clone(), d.clone(), gst.kv_len.clone()))
        ctx.close()
    for x, y in zip(*outs):
        assert torch.equal(x, y)


def test_device_seen_errors_and_host_validation():
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(prompt_len=20)
    K, B = cfg.k, cfg.batch
    w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=32)       # 2 pages per row only
    push_state(ost, gst, ctx)
    a = torch.zeros(B, dtype=torch.int32, device="cuda")
    t = torch.zeros(B, dtype=torch.int32, device="cuda")
    with pytest.raises(gmb.GmError) as e:
        gmb.gm_spec_step(ctx, gst, K + 1, 1.0, 0, 0, a, t)
    assert e.value.code == gmb.GM_ERR_UNSUPPORTED
    with pytest.raises(gmb.GmError) as e:
        gmb.gm_spec_step(ctx, gst, K, -1.0, 0, 0, a, t)
    assert e.value.code == gmb.GM_ERR_UNSUPPORTED
    with pytest.raises(gmb.GmError) as e:
        gmb.gm_spec_step(ctx, gst, K, 1.0, 0, 0, None, t)
    assert e.value.code == gmb.GM_ERR_INVALID_ARG
    # run until a row outgrows its two pages: the device reports it, nothing faults
    code = 0
    for it in range(12):
        gmb.gm_spec_step(ctx, gst, K, 1.0, 3, it, a, t)
        code = gmb.gm_last_status(ctx)
        if code:
            break
    assert code == gmb.GM_ERR_KV_CAPACITY
    # a page id outside the pool is reported too
    w2, ost2, ctx2, gst2 = tiny_setup(cfg, cap_tokens=96)
    push_state(ost2, gst2, ctx2)
    gst2.page_table[1, 1] = 10 ** 6
    gmb.gm_spec_step(ctx2, gst2, K, 1.0, 3, 0, a, t)
    assert gmb.gm_last_status(ctx2) == gmb.GM_ERR_BAD_PAGE
    ctx.close()
    ctx2.close()


def test_rerun_is_bit_identical_and_resume_equals_uninterrupted():
    """Counter-based uniforms and fixed-order reductions: the same state and (seed, step) give bit-identical
    tokens and state on a second run, and a rollout that is stopped, copied to the host, restored into fresh
    buffers and continued equals the uninterrupted one."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(prompt_len=25)
    K, B = cfg.k, cfg.batch
    w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=200)
    push_state(ost, gst, ctx)
    names = ("kv_len", "pending_n", "pending_tok", "pending_hidden", "kv_pool", "head_kv_pool")
    snap = {n: getattr(gst, n).clone() for n in names}
    a = torch.zeros(B, dtype=torch.int32, device="cuda")
    t = torch.zeros(B, dtype=torch.int32, device="cuda")
    d = torch.zeros((B, K), dtype=torch.int32, device="cuda")

    def rollout(state, first, n):
        out = []
        for it in range(first, first + n):
            gmb.gm_spec_step(ctx, state, K, 1.0, 21, it, a, t, d)
            out.append((a.cpu().clone(), t.cpu().clone(), d.cpu().clone()))
        return out

    ref = rollout(gst, 0, 12)
    end = {n: getattr(gst, n).clone() for n in names}
    for n, v in snap.items():
        getattr(gst, n).copy_(v)
    again = rollout(gst, 0, 12)
    for x, y in zip(ref, again):
        assert all(torch.equal(p, q) for p, q in zip(x, y))
    for n in names:
        assert torch.equal(getattr(gst, n), end[n]), n
    # stop after 5 steps, checkpoint to the host, restore into a new state object, continue
    for n, v in snap.items():
        getattr(gst, n).copy_(v)
    first = rollout(gst, 0, 5)
    ckpt = {n: getattr(gst, n).cpu() for n in names}
    gst2 = gmb.State(ctx, B, gst.page_table.cpu().numpy(), gst.head_page_table.cpu().numpy())
    for n, v in ckpt.items():
        getattr(gst2, n).copy_(v)
    rest = rollout(gst2, 5, 7)
    for x, y in zip(ref, first + rest):
        assert all(torch.equal(p, q) for p, q in zip(x, y))
    for n in names:
        assert torch.equal(getattr(gst2, n), end[n]), n
    assert gmb.gm_last_status(ctx) == 0
    ctx.close()


@pytest.mark.parametrize("sampler_flag", [0, 16], ids=["sampler_by_batch", "sampler_slice_per_cta"])
def test_graph_replayed_cycle_equals_host_launched_cycle(sampler_flag):
    """GM_FLAG_GRAPH on a stream of its own: gm_spec_step and gm_spec_step_host replay a captured cycle; accept
    lengths, tokens, drafts and the final state are bit-identical to the host-launched cycle, across re-captures
    (other output buffers) and with the step index changing every call.  With the sliced sampler the replayed launches
    find their epoch and their clean counters in device memory, not in captured arguments."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(prompt_len=33)
    K, B = cfg.k, cfg.batch
    out = {}
    side = torch.cuda.Stream()
    for flags in (0, gmb.GM_FLAG_GRAPH):
        with torch.cuda.stream(side):
            w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=160, flags=flags | sampler_flag)
            push_state(ost, gst, ctx)
            z = lambda *shape: torch.zeros(shape, dtype=torch.int32, device="cuda")
            a, t, d, a2, t2 = z(B), z(B), z(B, K), z(B), z(B)
            hist = []
            l0 = gmb.gm_launch_count(ctx)
            for it in range(6):
                gmb.gm_spec_step(ctx, gst, K, 1.0, 11, 100 + 7 * it, a, t, d)
                hist.append((a.cpu().numpy().copy(), t.cpu().numpy().copy(), d.cpu().numpy().copy()))
            for it in range(3):                                   # other output pointers: a second capture
                gmb.gm_spec_step(ctx, gst, K, 1.0, 11, 200 + it, a2, t2)
                hist.append((a2.cpu().numpy().copy(), t2.cpu().numpy().copy()))
            ud = torch.randint(0, 1 << 24, (B, K), dtype=torch.int32).pin_memory()
            ua = torch.randint(0, 1 << 24, (B, K + 1), dtype=torch.int32, generator=torch.Generator().manual_seed(3)).pin_memory()
            ah, th = torch.zeros(B, dtype=torch.int32).pin_memory(), torch.zeros(B, dtype=torch.int32).pin_memory()
            dh = torch.zeros((B, K), dtype=torch.int32).pin_memory()
            torch.manual_seed(5)
            for it in range(3):
                ud.copy_(torch.randint(0, 1 << 24, (B, K), dtype=torch.int32))
                gmb.gm_spec_step_host(ctx, gst, K, 1.0, 11, 300 + it, ah, th, dh, ud, ua)
                hist.append((ah.numpy().copy(), th.numpy().copy(), dh.numpy().copy()))
            assert gmb.gm_last_status(ctx) == 0
            out[flags] = (hist, gst.kv_len.cpu().numpy().copy(), gst.pending_hidden.clone().cpu(), gst.kv_pool.clone().cpu(),
                          gmb.gm_launch_count(ctx) - l0)
            ctx.close()
        side.synchronize()
    h0, h1 = out[0], out[gmb.GM_FLAG_GRAPH]
    for x, y in zip(h0[0], h1[0]):
        for u, v in zip(x, y):
            np.testing.assert_array_equal(u, v)
    np.testing.assert_array_equal(h0[1], h1[1])
    assert torch.equal(h0[2], h1[2]) and torch.equal(h0[3], h1[3])
    assert h1[4] == h0[4] + 12                                     # the same kernels + one step-index store per replay


def test_guard_words_behind_the_workspaces_stay_intact(monkeypatch):
    """With GM_CANARY set the library checks the 256 guard bytes behind each of its workspaces whenever the status is
    read: prefill, cycles at the largest depth, top-p, record and rollout bookkeeping leave all of them untouched."""
    import paper_2609_16648_b200 as gmb
    monkeypatch.setenv("GM_CANARY", "1")
    cfg = get_config("tiny").with_(k=7, prompt_len=30)
    K, B = cfg.k, cfg.batch
    w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=30 + 8 * (K + 1) + 8)
    assert gmb.gm_last_status(ctx) == 0
    prompts = np.array([s.tokens[:30] for s in ost.seqs], np.int32)
    gmb.gm_prefill(ctx, gst, torch.from_numpy(prompts).cuda(), torch.full((B,), 30, dtype=torch.int32, device="cuda"), 30, 1.0,
                   None, 5)
    assert gmb.gm_last_status(ctx) == 0
    gmb.gm_set_top_p(ctx, 0.8)
    rec = gmb.Record(B, K, cfg.d_model)
    a = torch.zeros(B, dtype=torch.int32, device="cuda")
    t = torch.zeros(B, dtype=torch.int32, device="cuda")
    d = torch.zeros((B, K), dtype=torch.int32, device="cuda")
    for it in range(3):
        gmb.gm_spec_step_rec(ctx, gst, K, 1.0, 5, 1 + it, a, t, d, rec)
    ro = gmb.Rollout(B, 12, -1)
    gmb.gm_rollout_begin(ctx, gst, ro)
    gmb.gm_rollout_run(ctx, gst, ro, K, 1.0, 5, 10, 3, 1)
    assert gmb.gm_last_status(ctx) == 0
    ctx.close()
