"""CUDA sampler (gm_accept / gm_draw) against the oracle's decision function."""
import numpy as np
import pytest
import torch

from oracle import philox, sampler as osampler
from synth_inputs import ModelConfig, sampler_only_logits
from synth_inputs.workload import random_u24

pytestmark = pytest.mark.gpu


MAPPING = {"flags": 0}


@pytest.fixture(autouse=True, params=[2, 4], ids=["cluster_per_sequence", "cta_per_sequence"])
def _mapping(request):
    """Every test of this file runs with both mappings of the sampler kernel."""
    MAPPING["flags"] = request.param
    yield


def _ctx(vocab, max_batch=256, max_k=7):
    import paper_2609_16648_b200 as gmb
    cfg = ModelConfig("s", 1, 64, 1, 1, 64, 64, vocab, batch=max_batch, k=max_k, kv_len_min=0, kv_len_max=0,
                      length_law="uniform")
    packed = gmb.random_packed_weights(cfg, "cuda")      # the sampler itself reads no weights
    return gmb, gmb.Context(cfg, packed, max_batch, max_k, 4, 8, 8, flags=MAPPING["flags"])


def _bf16(x):
    return torch.from_numpy(x).to(device="cuda", dtype=torch.bfloat16)


def _draft_tokens(drf, seed):
    B, K, V = drf.shape
    us = random_u24((B, K), seed=seed)
    return np.array([[osampler.draw_token(osampler.softmax_probs(drf[b, k]), us[b, k])[0] for k in range(K)]
                     for b in range(B)], np.int32)


@pytest.mark.parametrize("B,K,V,sigma,temp", [(5, 3, 4096, 0.9, 1.0), (3, 1, 4104, 0.5, 1.0), (4, 5, 8200, 1.4, 0.7),
                                              (2, 7, 151936, 0.908, 1.0), (6, 3, 151936, 0.908, 1.3)])
def test_accept_decisions_bit_exact_on_dumped_probabilities(B, K, V, sigma, temp):
    gmb, ctx = _ctx(V)
    tgt, drf = sampler_only_logits(B, K, V, sigma=sigma, seed=40 + K)
    dtok = _draft_tokens(drf, seed=50 + K)
    u24 = random_u24((B, K + 1), seed=60 + K)
    u24[0, :K] = 0                      # u = 0: accepts whenever p > 0
    u24[1 % B, 0] = (1 << 24) - 1
    a = torch.zeros(B, dtype=torch.int32, device="cuda")
    t = torch.zeros(B, dtype=torch.int32, device="cuda")
    dp = torch.zeros((B, K + 1, V), dtype=torch.float32, device="cuda")
    dq = torch.zeros((B, K, V), dtype=torch.float32, device="cuda")
    gmb.gm_accept(ctx, None, B, K, temp, _bf16(tgt), _bf16(drf), torch.from_numpy(dtok).cuda(),
                  torch.from_numpy(u24.astype(np.int32)).cuda(), 0, 0, a, t, dp, dq)
    assert gmb.gm_last_status(ctx) == 0
    p, q = dp.cpu().numpy(), dq.cpu().numpy()
    for b in range(B):
        ea, et, warn = osampler.decide(p[b], q[b], dtok[b], u24[b])
        assert warn == 0
        assert (int(a[b]), int(t[b])) == (ea, et), (b, int(a[b]), int(t[b]), ea, et)
    # the dumped probabilities are the softmax of the logits (fp32 arithmetic on the device)
    ref_p = osampler.softmax_probs(tgt, temp)
    ref_q = osampler.softmax_probs(drf, temp)
    # exponent arguments reach 2^5, so each of their three roundings (c of the thread, of the merge, of the row) moves p by <= 1.3e-6
    assert np.abs(p - ref_p).max() <= 5e-6 * ref_p.max() + 1e-9
    assert np.abs(q - ref_q).max() <= 5e-6 * ref_q.max() + 1e-9
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=2e-5)
    # end to end (oracle softmax in fp64 instead of the device's): decisions agree on almost every row
    ea, et, _ = osampler.accept_batch(tgt, drf, dtok, u24, temp)
    assert (ea == a.cpu().numpy()).mean() >= 0.8 or B < 5
    # without the dump buffers the result is the same
    a2, t2 = torch.zeros_like(a), torch.zeros_like(t)
    gmb.gm_accept(ctx, None, B, K, temp, _bf16(tgt), _bf16(drf), torch.from_numpy(dtok).cuda(),
                  torch.from_numpy(u24.astype(np.int32)).cuda(), 0, 0, a2, t2)
    assert torch.equal(a, a2) and torch.equal(t, t2)
    ctx.close()


def test_accept_with_device_philox_matches_oracle_slots():
    gmb, ctx = _ctx(4096)
    B, K, V = 7, 3, 4096
    tgt, drf = sampler_only_logits(B, K, V, sigma=1.0, seed=3)
    dtok = _draft_tokens(drf, seed=4)
    seed, step = 0x1234567_89ABCDEF, (1 << 32) + 17
    a = torch.zeros(B, dtype=torch.int32, device="cuda")
    t = torch.zeros(B, dtype=torch.int32, device="cuda")
    dp = torch.zeros((B, K + 1, V), dtype=torch.float32, device="cuda")
    dq = torch.zeros((B, K, V), dtype=torch.float32, device="cuda")
    gmb.gm_accept(ctx, None, B, K, 1.0, _bf16(tgt), _bf16(drf), torch.from_numpy(dtok).cuda(), None, seed, step, a, t,
                  dp, dq)
    ua = philox.u24_accept(seed, step, B, K)
    p, q = dp.cpu().numpy(), dq.cpu().numpy()
    for b in range(B):
        ea, et, _ = osampler.decide(p[b], q[b], dtok[b], ua[b])
        assert (int(a[b]), int(t[b])) == (ea, et)
    ctx.close()


@pytest.mark.parametrize("rows,V", [(9, 4096), (3, 151936), (1, 8)])
def test_draw_matches_integer_inverse_cdf(rows, V):
    gmb, ctx = _ctx(V)
    tgt, _ = sampler_only_logits(rows, 0, V, seed=9)
    logits = tgt[:, 0]
    u = random_u24((rows,), seed=10)
    u[0] = 0
    u[-1] = (1 << 24) - 1
    out = torch.zeros(rows, dtype=torch.int32, device="cuda")
    dbg = torch.zeros((rows, V), dtype=torch.float32, device="cuda")
    gmb.gm_draw(ctx, _bf16(logits), rows, 1.0, torch.from_numpy(u.astype(np.int32)).cuda(), out, dbg)
    pr = dbg.cpu().numpy()
    for r in range(rows):
        assert int(out[r]) == osampler.draw_token(pr[r], u[r])[0]
    ctx.close()


def test_identical_logits_accept_everything_and_peaked_rows():
    """q == p accepts all K drafts whatever the uniforms; a one-hot-like row still draws correctly."""
    gmb, ctx = _ctx(4096)
    B, K, V = 4, 3, 4096
    tgt, _ = sampler_only_logits(B, K, V, seed=11)
    tgt[2, :, :] = -30.0
    tgt[2, :, 77] = 30.0                     # a peaked row: p(77) = 1 to fp32 precision
    drf = tgt[:, :K].copy()
    dtok = _draft_tokens(drf, seed=12)
    u24 = np.full((B, K + 1), (1 << 24) - 1, np.uint32)
    a = torch.zeros(B, dtype=torch.int32, device="cuda")
    t = torch.zeros(B, dtype=torch.int32, device="cuda")
    dp = torch.zeros((B, K + 1, V), dtype=torch.float32, device="cuda")
    gmb.gm_accept(ctx, None, B, K, 1.0, _bf16(tgt), _bf16(drf), torch.from_numpy(dtok).cuda(),
                  torch.from_numpy(u24.astype(np.int32)).cuda(), 0, 0, a, t, dp, None)
    assert a.tolist() == [K] * B
    p = dp.cpu().numpy()
    for b in range(B):
        assert int(t[b]) == osampler.draw_token(p[b, K], u24[b, K])[0]
    assert int(t[2]) == 77
    ctx.close()


def test_argument_validation():
    gmb, ctx = _ctx(4096, max_batch=4, max_k=3)
    z = torch.zeros(8, dtype=torch.int32, device="cuda")
    lg = torch.zeros((4, 4, 4096), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(gmb.GmError) as e:
        gmb.gm_accept(ctx, None, 4, 3, 0.0, lg, lg, z, None, 0, 0, z, z)
    assert e.value.code == gmb.GM_ERR_UNSUPPORTED
    with pytest.raises(gmb.GmError) as e:
        gmb.gm_accept(ctx, None, 4, 3, 1.0, None, lg, z, None, 0, 0, z, z)
    assert e.value.code == gmb.GM_ERR_INVALID_ARG
    with pytest.raises(gmb.GmError) as e:
        gmb.gm_accept(ctx, None, 4, 9, 1.0, lg, lg, z, None, 0, 0, z, z)
    assert e.value.code == gmb.GM_ERR_UNSUPPORTED
    ctx.close()


def test_sampler_only_workload_full_size_all_rows():
    """The sampler-only configuration at full size (256 sequences x 4 positions, vocabulary 151936, draft =
    target + N(0, 0.908) noise): the device's decisions equal the oracle's decision function on the device's
    probabilities for ALL 256 rows, and the mean acceptance is near the closed form 0.65."""
    gmb, ctx = _ctx(151936, max_batch=256, max_k=3)
    B, K, V = 256, 3, 151936
    tgt, drf = sampler_only_logits(B, K, V, sigma=0.908, seed=4)
    t_dev, d_dev = _bf16(tgt), _bf16(drf)
    us = random_u24((B, K), seed=5)
    dtok = torch.zeros((B, K), dtype=torch.int32, device="cuda")
    for k in range(K):                                            # drafts drawn on the device from q_k
        col = torch.zeros(B, dtype=torch.int32, device="cuda")
        gmb.gm_draw(ctx, d_dev[:, k].contiguous(), B, 1.0, torch.from_numpy(us[:, k].astype(np.int32)).cuda(), col)
        dtok[:, k] = col
    u24 = random_u24((B, K + 1), seed=6)
    a = torch.zeros(B, dtype=torch.int32, device="cuda")
    t = torch.zeros(B, dtype=torch.int32, device="cuda")
    dp = torch.zeros((B, K + 1, V), dtype=torch.float32, device="cuda")
    dq = torch.zeros((B, K, V), dtype=torch.float32, device="cuda")
    gmb.gm_accept(ctx, None, B, K, 1.0, t_dev, d_dev, dtok, torch.from_numpy(u24.astype(np.int32)).cuda(), 0, 0, a, t, dp, dq)
    assert gmb.gm_last_status(ctx) == 0
    p, q, dt = dp.cpu().numpy(), dq.cpu().numpy(), dtok.cpu().numpy()
    an, tn = a.cpu().numpy(), t.cpu().numpy()
    for b in range(B):
        for k in range(K):
            assert dt[b, k] == osampler.draw_token(q[b, k], us[b, k])[0]
        ea, et, warn = osampler.decide(p[b], q[b], dt[b], u24[b])
        assert (ea, et, warn) == (an[b], tn[b], 0), b
    first = (an >= 1).mean()
    assert 0.5 < first < 0.8, first                               # per-token acceptance ~ 0.65 (+- sampling noise)
    ctx.close()
