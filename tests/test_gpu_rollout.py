"""Whole rollouts on the device: stopping rules, rows that sit out, and the page allocator."""
import numpy as np
import pytest
import torch

from oracle import step as ostep
from synth_inputs import get_config, make_page_tables, make_weights
from synth_inputs.weights import perturb_norm_weights

from helpers import push_state, tiny_setup

pytestmark = pytest.mark.gpu

STATE_FIELDS = ("kv_len", "pending_n", "pending_tok", "pending_hidden", "kv_pool", "head_kv_pool")


def _free_running_streams(gmb, ctx, gst, K, seed, n_steps):
    """Committed tokens per row of n_steps plain cycles: [first token] + accepted drafts + final token of each."""
    B = gst.batch
    a = torch.zeros(B, dtype=torch.int32, device="cuda")
    t = torch.zeros(B, dtype=torch.int32, device="cuda")
    d = torch.zeros((B, K), dtype=torch.int32, device="cuda")
    streams = [[int(x)] for x in gst.pending_tok[:, 0].cpu().numpy()]
    per_step = []
    for it in range(n_steps):
        gmb.gm_spec_step(ctx, gst, K, 1.0, seed, 1 + it, a, t, d)
        an, tn, dn = a.cpu().numpy(), t.cpu().numpy(), d.cpu().numpy()
        for b in range(B):
            streams[b] += [int(x) for x in dn[b, :an[b]]] + [int(tn[b])]
        per_step.append(an.copy())
    return streams, per_step


@pytest.mark.parametrize("sampler", [None, "flow"], ids=["sampler_by_batch", "sampler_slice_per_cta"])
def test_rollout_equals_plain_cycles_cut_by_the_stopping_rules(sampler, monkeypatch):
    """The rollout driver's responses are the streams of plain cycles cut by the oracle's stopping rule; rows
    that have ended sit out and leave the others unchanged (here every attention segment is a single page, so
    the running rows' arithmetic does not depend on who else is running).  Both with the sampler mapping the batch
    size selects and with the sliced mapping forced (rows that sit out, state commit)."""
    import paper_2609_16648_b200 as gmb
    if sampler:
        monkeypatch.setenv("GM_SAMPLER", sampler)
    cfg = get_config("tiny").with_(prompt_len=20)
    K, B = cfg.k, cfg.batch
    n_steps, cap = 10, 13
    w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=20 + n_steps * (K + 1) + 8)
    push_state(ost, gst, ctx)
    snap = {n: getattr(gst, n).clone() for n in STATE_FIELDS}
    streams, _ = _free_running_streams(gmb, ctx, gst, K, 5, n_steps)
    assert gmb.gm_last_status(ctx) == 0
    eos = streams[0][5]
    for eos_token, max_new in ((eos, cap), (-1, cap), (eos, 1000), (streams[1][0], 7)):
        for n, v in snap.items():
            getattr(gst, n).copy_(v)
        ro = gmb.Rollout(B, max_new, eos_token)
        gmb.gm_rollout_begin(ctx, gst, ro)
        steps, running = gmb.gm_rollout_run(ctx, gst, ro, K, 1.0, 5, 1, n_steps, check_every=3)
        assert gmb.gm_last_status(ctx) == 0
        resp, fin = ro.responses(), ro.finished.cpu().numpy()
        for b in range(B):
            want = []
            code = ostep.append_committed(want, streams[b], eos_token, max_new)
            assert resp[b] == want, (eos_token, max_new, b)
            assert fin[b] == code
        assert running == int((fin == 0).sum()) == int(ro.n_running[0])
        assert steps <= n_steps and (running > 0 or steps < n_steps or max_new >= 1000)
        # a finished row's state is frozen where it stopped: its cache length never passes the tokens it kept
        # by more than one cycle
        kv = gst.kv_len.cpu().numpy()
        for b in range(B):
            if fin[b]:
                assert kv[b] <= 20 + len(resp[b]) + K
    ctx.close()


def test_row_that_sits_out_is_left_untouched():
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(prompt_len=20)
    K, B = cfg.k, cfg.batch
    w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=80)
    push_state(ost, gst, ctx)
    ro = gmb.Rollout(B, 50, -1)
    gmb.gm_rollout_begin(ctx, gst, ro)
    ro.finished[2] = 2                                      # row 2 sits out from the start
    before = {n: getattr(gst, n).clone() for n in STATE_FIELDS}
    for it in range(4):
        gmb.gm_rollout_step(ctx, gst, ro, K, 1.0, 5, 1 + it)
    assert gmb.gm_last_status(ctx) == 0
    assert int(gst.kv_len[2]) == int(before["kv_len"][2]) and int(ro.out_len[2]) == 1
    assert torch.equal(gst.pending_tok[2], before["pending_tok"][2])
    assert torch.equal(gst.pending_hidden[2], before["pending_hidden"][2])
    pt = gst.page_table.cpu().numpy()
    for name, table in (("kv_pool", pt), ("head_kv_pool", gst.head_page_table.cpu().numpy())):
        pages = torch.as_tensor(table[2][table[2] >= 0], device="cuda", dtype=torch.long)
        assert torch.equal(getattr(gst, name)[:, :, pages], before[name][:, :, pages])
    assert (gst.kv_len.cpu().numpy()[[0, 1, 3]] >= before["kv_len"].cpu().numpy()[[0, 1, 3]] + 4).all()
    assert int(ro.n_running[0]) == 3
    ctx.close()


def test_page_allocator_rollout_equals_static_tables_and_returns_pages():
    """Prefill + rollout with pages handed out on demand gives the same responses as with page tables laid
    out in advance; no page is ever held twice; finished rows hand their pages back; exhaustion is reported."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny")
    K, B, V = cfg.k, cfg.batch, cfg.vocab
    w = perturb_norm_weights(make_weights(cfg, 0))
    lengths = [7, 30, 18, 1]
    rng = np.random.default_rng(3)
    tok = np.zeros((B, 32), np.int32)
    for b, n in enumerate(lengths):
        tok[b, :n] = rng.integers(0, V, n)
    tok_d = torch.from_numpy(tok).cuda()
    len_d = torch.tensor(lengths, dtype=torch.int32, device="cuda")
    max_new, n_steps = 24, 12
    cap = 30 + max_new + 2 * (K + 1)
    pt, npg = make_page_tables(np.full(B, cap), cfg.page_size, seed=7)
    ctx = gmb.Context(cfg, gmb.pack_weights(w), B, K, pt.shape[1], npg, npg)

    def run(allocator):
        st = gmb.State(ctx, B, np.full_like(pt, -1) if allocator else pt, np.full_like(pt, -1) if allocator else pt)
        if allocator:
            gmb.gm_pages_reset(ctx, st)
            assert gmb.gm_pages_free_count(ctx) == (npg, npg)
            gmb.gm_pages_reserve(ctx, st, len_d, K + 1)
        gmb.gm_prefill(ctx, st, tok_d, len_d, max(lengths), 1.0, None, 9)
        ro = gmb.Rollout(B, max_new, -1)
        gmb.gm_rollout_begin(ctx, st, ro)
        held_seen = []
        for it in range(n_steps):
            gmb.gm_rollout_step(ctx, st, ro, K, 1.0, 9, 1 + it)
            if allocator:
                t = st.page_table.cpu().numpy()
                ids = t[t >= 0]
                assert len(ids) == len(set(ids.tolist()))                    # no page held twice
                kv, fin = st.kv_len.cpu().numpy(), ro.finished.cpu().numpy()
                for b in range(B):
                    held = int((t[b] >= 0).sum())
                    assert held == 0 if fin[b] else held * 16 >= kv[b]
                held_seen.append(len(ids))
                assert gmb.gm_pages_free_count(ctx)[0] == npg - len(ids)
        assert gmb.gm_last_status(ctx) == 0
        return ro.responses(), ro.finished.cpu().numpy(), held_seen

    r0, f0, _ = run(False)
    r1, f1, held = run(True)
    assert r0 == r1 and (f0 == f1).all()
    assert (f1 == 2).all() and held[-1] == 0                                 # everyone reached the cap: all pages back
    assert gmb.gm_pages_free_count(ctx) == (npg, npg)
    # a pool that is too small: reported, nothing written out of range
    st = gmb.State(ctx, B, np.full_like(pt, -1), np.full_like(pt, -1))
    gmb.gm_pages_reset(ctx, st)
    gmb.gm_pages_reserve(ctx, st, torch.full((B,), 16 * npg, dtype=torch.int32, device="cuda"), 1)
    torch.cuda.synchronize()
    assert gmb.gm_last_status(ctx) != 0
    t = st.page_table.cpu().numpy()
    assert t.max() < npg and len(set(t[t >= 0].tolist())) == (t >= 0).sum()
    ctx.close()


def _two_rollouts(gmb, cfg, n_steps, flags):
    K, B = cfg.k, cfg.batch
    w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=20 + n_steps * (K + 1) + 8, flags=flags)
    push_state(ost, gst, ctx)
    snap = {n: getattr(gst, n).clone() for n in STATE_FIELDS}
    ro = gmb.Rollout(B, 17, -1)
    runs = []
    for rep in range(2):
        for n, v in snap.items():
            getattr(gst, n).copy_(v)
        gmb.gm_rollout_begin(ctx, gst, ro)
        l0 = gmb.gm_launch_count(ctx)
        steps, running = gmb.gm_rollout_run(ctx, gst, ro, K, 1.0, 5, 1 + 100 * rep, n_steps, check_every=2)
        assert gmb.gm_last_status(ctx) == 0
        runs.append((steps, running, ro.responses(), ro.finished.cpu().numpy().copy(), gst.kv_len.cpu().numpy().copy(),
                     gst.pending_hidden.clone().cpu(), gmb.gm_launch_count(ctx) - l0))
    ctx.close()
    return runs


def test_graph_replayed_rollout_equals_host_launched_rollout():
    """One captured cycle replayed per step (step index on the device) gives the same responses, stop codes and
    final state as the host-launched loop; a second rollout through the same buffers reuses the graph."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(prompt_len=20)
    K, B = cfg.k, cfg.batch
    n_steps = 9
    results = {}
    side = torch.cuda.Stream()                                   # the default stream cannot be captured
    for flags in (0, 8):
        with torch.cuda.stream(side):
            runs = _two_rollouts(gmb, cfg, n_steps, flags)
        side.synchronize()
        results[flags] = runs
    for rep in range(2):
        h, g = results[0][rep], results[8][rep]
        assert h[0] == g[0] and h[1] == g[1] and h[2] == g[2]
        np.testing.assert_array_equal(h[3], g[3])
        np.testing.assert_array_equal(h[4], g[4])
        assert torch.equal(h[5], g[5])
        assert g[6] == h[6] + 1 > 1                              # the replayed kernels are counted, plus one store of the first step index
    assert results[0][0][2] != results[0][1][2]                  # different step indices: different uniforms


def test_graph_replay_with_on_demand_pages_and_stopping():
    """The captured cycle includes the page reserve / release kernels and the finished mask: a graph-replayed rollout
    with on-demand pages, an end-of-sequence token and a cap equals the host-launched one, and every page comes back."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny")
    K, B, V = cfg.k, cfg.batch, cfg.vocab
    w = perturb_norm_weights(make_weights(cfg, 0))
    lengths = [5, 21, 12, 30]
    rng = np.random.default_rng(4)
    tok = np.zeros((B, 32), np.int32)
    for b, n in enumerate(lengths):
        tok[b, :n] = rng.integers(0, V, n)
    max_new, n_steps = 20, 12
    pt, npg = make_page_tables(np.full(B, 30 + max_new + 2 * (K + 1)), cfg.page_size, seed=7)
    out = {}
    side = torch.cuda.Stream()
    for flags in (0, gmb.GM_FLAG_GRAPH):
        with torch.cuda.stream(side):
            ctx = gmb.Context(cfg, gmb.pack_weights(w), B, K, pt.shape[1], npg, npg, flags=flags)
            st = gmb.State(ctx, B, np.full_like(pt, -1), np.full_like(pt, -1))
            tok_d = torch.from_numpy(tok).cuda()
            len_d = torch.tensor(lengths, dtype=torch.int32, device="cuda")
            gmb.gm_pages_reset(ctx, st)
            gmb.gm_pages_reserve(ctx, st, len_d, K + 1)
            gmb.gm_prefill(ctx, st, tok_d, len_d, max(lengths), 1.0, None, 9)
            eos = int(st.pending_tok[1, 0])                      # row 1 ends at once; the others run on
            ro = gmb.Rollout(B, max_new, eos)
            gmb.gm_rollout_begin(ctx, st, ro)
            steps, running = gmb.gm_rollout_run(ctx, st, ro, K, 1.0, 9, 1, n_steps, check_every=4)
            assert gmb.gm_last_status(ctx) == 0
            out[flags] = (steps, running, ro.responses(), ro.finished.cpu().numpy().copy(), gmb.gm_pages_free_count(ctx),
                          st.kv_len.cpu().numpy().copy())
            ctx.close()
        side.synchronize()
    h, g = out[0], out[gmb.GM_FLAG_GRAPH]
    assert h[2] == g[2] and (h[3] == g[3]).all() and (h[5] == g[5]).all() and h[1] == g[1]
    assert h[3][1] == 1 and len(h[2][1]) == 1                    # ended on its first token
    assert g[0] >= h[0] and g[0] - h[0] < 4                      # the replayed loop may run up to check_every - 1 idle cycles
    assert h[4] == g[4]
    if h[1] == 0:
        assert h[4] == (npg, npg)
