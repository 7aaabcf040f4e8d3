"""Prompt prefill on the device (chunks of max_k + 1 positions through the verify / draft kernels) against the
oracle's full causal prefill: caches of the backbone and of the draft head, pending pair, first response token."""
import numpy as np
import pytest
import torch

from oracle import model as omodel, philox, sampler as osampler, step as ostep
from synth_inputs import get_config, make_page_tables, make_weights
from synth_inputs.weights import perturb_norm_weights

from helpers import rel_err

pytestmark = pytest.mark.gpu

TOL = 2e-2


def _cache_view(cfg, n_layers, pool_tensor, page_table, num_pages):
    kv = omodel.PagedKV(n_layers, cfg.n_kv_heads, cfg.head_dim, page_table, num_pages, cfg.page_size)
    kv.pool = pool_tensor.float().cpu().numpy().astype(np.float64)
    return kv


@pytest.mark.parametrize("lengths,k", [((1, 5, 40, 17), 3), ((33, 2, 64, 8), 7), ((9, 9, 9, 9), 1)])
def test_prefill_matches_the_oracle(lengths, k):
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(k=k, batch=len(lengths))
    B, V, d = cfg.batch, cfg.vocab, cfg.d_model
    w = perturb_norm_weights(make_weights(cfg, 0))
    rng = np.random.default_rng(12)
    prompts = [rng.integers(0, V, n) for n in lengths]
    cap = max(lengths) + 4 * (k + 1) + 16
    pt, npg = make_page_tables(np.full(B, cap), cfg.page_size, seed=7, slack_pages=3)
    hpt, hnpg = make_page_tables(np.full(B, cap), cfg.page_size, seed=8, slack_pages=2)
    seed = 5
    ost = ostep.prefill(w, cfg, prompts, pt, npg, hpt, hnpg, temperature=1.0, seed=seed)
    ctx = gmb.Context(cfg, gmb.pack_weights(w), B, k, pt.shape[1], npg, hnpg)
    gst = gmb.State(ctx, B, pt, hpt)
    stride = max(lengths) + 3
    tok = np.zeros((B, stride), np.int32)
    for b, pr in enumerate(prompts):
        tok[b, :len(pr)] = pr
    first = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    dbg_p = torch.zeros((B, V), dtype=torch.float32, device="cuda")
    gmb.gm_prefill(ctx, gst, torch.from_numpy(tok).cuda(), torch.tensor(lengths, dtype=torch.int32, device="cuda"),
                   max(lengths), 1.0, None, seed, first, dbg_p)
    torch.cuda.synchronize()
    assert gmb.gm_last_status(ctx) == 0
    np.testing.assert_array_equal(gst.kv_len.cpu().numpy(), lengths)
    np.testing.assert_array_equal(gst.pending_n.cpu().numpy(), 1)
    np.testing.assert_array_equal(gst.pending_tok.cpu().numpy()[:, 0], first.cpu().numpy())
    p = dbg_p.cpu().numpy()
    kv = _cache_view(cfg, cfg.n_layers, gst.kv_pool, pt, npg)
    hkv = _cache_view(cfg, 1, gst.head_kv_pool, hpt, hnpg)
    same_first = 0
    for b, L in enumerate(lengths):
        s = ost.seqs[b]
        # the first token is the integer inverse-CDF draw from the device's own distribution
        assert int(first[b]) == osampler.draw_token(p[b], philox.u24(seed, 0, b, philox.SLOT_FINAL))[0]
        same_first += int(first[b]) == s.tokens[-1]
        H_last = omodel.round_bf16(s.pending_hidden[0])
        ref_p = osampler.softmax_probs(omodel.round_bf16(omodel.target_logits(w, H_last[None], cfg))[0])
        assert np.abs(p[b] - ref_p).max() <= 0.05 * ref_p.max()
        assert rel_err(gst.pending_hidden[b, 0].float().cpu().numpy(), s.pending_hidden[0]) < TOL
        for l in range(cfg.n_layers):
            for got, ref in zip(kv.gather(l, b, L), ost.kv.gather(l, b, L)):
                assert rel_err(got, ref) < TOL, (b, l)
        if L > 1:
            for got, ref in zip(hkv.gather(0, b, L - 1), ost.hkv.gather(0, b, L - 1)):
                assert rel_err(got, ref) < TOL, b
    assert same_first >= B - 1
    # a cycle runs from the prefilled state
    a = torch.zeros(B, dtype=torch.int32, device="cuda")
    t = torch.zeros(B, dtype=torch.int32, device="cuda")
    for it in range(3):
        gmb.gm_spec_step(ctx, gst, k, 1.0, seed, 1 + it, a, t)
    assert gmb.gm_last_status(ctx) == 0
    assert (gst.kv_len.cpu().numpy() >= np.array(lengths) + 3).all()
    ctx.close()


def test_prefill_rejects_bad_lengths():
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(batch=2)
    w = make_weights(cfg, 0)
    pt, npg = make_page_tables(np.full(2, 64), cfg.page_size, seed=7)
    ctx = gmb.Context(cfg, gmb.pack_weights(w), 2, cfg.k, pt.shape[1], npg, npg)
    gst = gmb.State(ctx, 2, pt, pt)
    tok = torch.zeros((2, 16), dtype=torch.int32, device="cuda")
    with pytest.raises(RuntimeError):                      # stride shorter than the longest prompt
        gmb.gm_prefill(ctx, gst, tok, torch.tensor([4, 4], dtype=torch.int32, device="cuda"), 32, 1.0, None, 0)
    with pytest.raises(RuntimeError):                      # page tables cannot hold the prompt
        big = torch.zeros((2, 4096), dtype=torch.int32, device="cuda")
        gmb.gm_prefill(ctx, gst, big, torch.tensor([4, 4], dtype=torch.int32, device="cuda"), 4096, 1.0, None, 0)
    gmb.gm_prefill(ctx, gst, tok, torch.tensor([0, 9], dtype=torch.int32, device="cuda"), 8, 1.0, None, 0)
    torch.cuda.synchronize()
    assert gmb.gm_last_status(ctx) != 0                    # an empty prompt and one longer than max_prompt_len: reported
    ctx.close()
