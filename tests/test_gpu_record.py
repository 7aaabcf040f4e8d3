"""Cycle record (gm_record_begin / gm_record_end / gm_spec_step_rec) against the oracle (App. D.2)."""
import numpy as np
import pytest
import torch

from oracle import record as orecord
from synth_inputs import ModelConfig, get_config, sampler_only_logits, bf16_round

from helpers import push_state, tiny_setup

pytestmark = pytest.mark.gpu


def _ctx(vocab, max_batch, max_k=3):
    import paper_2609_16648_b200 as gmb
    cfg = ModelConfig("r", 1, 64, 1, 1, 64, 64, vocab, batch=max_batch, k=max_k, kv_len_min=0, kv_len_max=0,
                      length_law="uniform")
    return gmb, gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), max_batch, max_k, 4, 8, 8)


def _run_end(gmb, ctx, tgt, K, temp=1.0):
    B, _, V = tgt.shape
    rec = gmb.Record(B, K, 64)
    dt = torch.arange(B * K, dtype=torch.int32, device="cuda").reshape(B, K)
    al = torch.arange(B, dtype=torch.int32, device="cuda") % (K + 1)
    gmb.gm_record_end(ctx, B, K, temp, torch.from_numpy(tgt).to(device="cuda", dtype=torch.bfloat16), dt, al, rec)
    assert gmb.gm_last_status(ctx) == 0
    assert torch.equal(rec.drafts, dt) and torch.equal(rec.accepted, al + 1)
    return rec.top_index.cpu().numpy(), rec.top_logprob.float().cpu().numpy()


def _check(tgt, K, idx, lp, temp=1.0):
    B = tgt.shape[0]
    for b in range(B):
        for k in range(K):
            ei, el = orecord.top_logprobs(tgt[b, k], temp)
            np.testing.assert_array_equal(idx[b, k], ei)
            fin = np.isfinite(el)
            # bf16 log-probabilities: one ulp (2^-8 relative) of slack for the fp32 vs fp64 log-sum-exp
            assert np.all(np.abs(lp[b, k][fin] - el[fin]) <= 2.0 ** -7 * np.abs(el[fin]) + 1e-6)
            assert np.all(np.isneginf(lp[b, k][~fin]))


@pytest.mark.parametrize("B,K,V,temp", [(3, 3, 4096, 1.0), (2, 1, 520, 0.7), (5, 5, 8200, 1.0), (4, 3, 151936, 1.0)])
def test_top64_matches_the_oracle(B, K, V, temp):
    gmb, ctx = _ctx(V, B, max_k=K)
    tgt, _ = sampler_only_logits(B, K, V, seed=70 + K)
    idx, lp = _run_end(gmb, ctx, tgt, K, temp)
    _check(tgt, K, idx, lp, temp)
    ctx.close()


def test_ties_and_short_rows():
    """bf16 logits tie often: the cut must fall inside a run of equal values and take the lowest token ids, also
    across the eight vocabulary slices; a row shorter than 64 is padded."""
    gmb, ctx = _ctx(1024, 3)
    K, V = 2, 1024
    tgt = np.zeros((3, K + 1, V), np.float32)
    tgt[0, 0, [5, 700, 1023]] = 2.0
    tgt[0, 0, 100:400] = 1.0                           # 300 ties for 61 places, spanning three slices
    tgt[0, 1] = bf16_round(np.linspace(-3, 3, V).astype(np.float32))
    tgt[1, 0] = -1.5                                   # everything ties
    tgt[1, 1, ::2] = 0.25
    tgt[1, 1, 1::2] = -0.0                             # -0 and +0 mixed with a positive class
    tgt[2, 0] = bf16_round(np.random.default_rng(3).normal(0, 0.05, V).astype(np.float32))   # few distinct values
    tgt[2, 1] = tgt[2, 0][::-1]
    idx, lp = _run_end(gmb, ctx, tgt, K)
    _check(tgt, K, idx, lp)
    ctx.close()
    # peaked rows: fewer than 64 entries within 256 key steps of the maximum (the selection's full-range levels)
    gmb, ctx = _ctx(4096, 2)
    tgt = np.full((2, 3, 4096), -30.0, np.float32)
    tgt[0, 0, 77] = 30.0                               # one-hot-like: the other 63 places are ties far below
    tgt[0, 1, 5:25] = bf16_round(np.linspace(8, 20, 20).astype(np.float32))
    tgt[1, 0] = bf16_round(np.random.default_rng(4).normal(0, 1, 4096).astype(np.float32))
    tgt[1, 0, 1000:1040] = 500.0                       # 40 large ties, then the bulk of the row far below
    tgt[1, 1] = bf16_round((np.arange(4096) % 97).astype(np.float32) * -0.5)
    idx, lp = _run_end(gmb, ctx, tgt, 2)
    _check(tgt, 2, idx, lp)
    ctx.close()
    gmb, ctx = _ctx(40, 2)
    tgt, _ = sampler_only_logits(2, 1, 40, seed=9)
    idx, lp = _run_end(gmb, ctx, tgt, 1)
    _check(tgt, 1, idx, lp)
    assert np.all(idx[:, :, 40:] == -1)
    ctx.close()


def test_spec_step_rec_records_the_cycle_and_leaves_it_unchanged():
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(prompt_len=30)
    K, B, V, d = cfg.k, cfg.batch, cfg.vocab, cfg.d_model
    w, ost, ctx, gst = tiny_setup(cfg, cap_tokens=120)
    push_state(ost, gst, ctx)
    snap = {n: getattr(gst, n).clone() for n in ("kv_len", "pending_n", "pending_tok", "pending_hidden", "kv_pool",
                                                   "head_kv_pool")}
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device="cuda")
    a, t, dt = z((B,), torch.int32), z((B,), torch.int32), z((B, K), torch.int32)
    rec = gmb.Record(B, K, d)
    start_h = torch.stack([gst.pending_hidden[b, int(gst.pending_n[b]) - 1] for b in range(B)]).clone()
    start_len = gst.kv_len.clone() + 1
    gmb.gm_spec_step_rec(ctx, gst, K, 1.0, 9, 3, a, t, dt, rec)
    assert gmb.gm_last_status(ctx) == 0
    assert torch.equal(rec.start_hidden, start_h) and torch.equal(rec.start_pos, start_len)
    assert torch.equal(rec.drafts, dt) and torch.equal(rec.accepted, a + 1)
    after = {n: getattr(gst, n).clone() for n in snap}
    # the same cycle without the record, from the same state: identical outputs and state
    for n, v in snap.items():
        getattr(gst, n).copy_(v)
    a2, t2, dt2 = z((B,), torch.int32), z((B,), torch.int32), z((B, K), torch.int32)
    tl, th, dl = z((B, K + 1, V), torch.bfloat16), z((B, K + 1, d), torch.bfloat16), z((B, K, V), torch.bfloat16)
    gmb.gm_draft(ctx, gst, K, 1.0, None, 9, 3, dt2, dl)
    gmb.gm_verify(ctx, gst, K, dt2, tl, th)
    gmb.gm_accept(ctx, gst, B, K, 1.0, tl, dl, dt2, None, 9, 3, a2, t2, None, None, th, commit_state=True)
    assert torch.equal(a, a2) and torch.equal(t, t2) and torch.equal(dt, dt2)
    for n, v in after.items():
        assert torch.equal(getattr(gst, n), v), n
    # the recorded distributions are the top-64 of this cycle's verification logits
    tln = tl.float().cpu().numpy()
    _check(tln, K, rec.top_index.cpu().numpy(), rec.top_logprob.float().cpu().numpy())
    ctx.close()
