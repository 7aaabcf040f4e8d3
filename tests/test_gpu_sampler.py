"""CUDA sampler (gm_accept / gm_draw) against the oracle's decision function."""
import numpy as np
import pytest
import torch

from oracle import philox, sampler as osampler
from synth_inputs import ModelConfig, sampler_only_logits
from synth_inputs.workload import random_u24

pytestmark = pytest.mark.gpu


MAPPING = {"flags": 0}


@pytest.fixture(autouse=True, params=[2, 4, 16], ids=["cluster_per_sequence", "cta_per_sequence", "slice_per_cta"])
def _mapping(request):
    """Every test of this file runs with all three mappings of the sampler kernel."""
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
    ga = a.cpu().numpy()
    print(f"accepted lengths equal to the fp64 softmax path on {(ea == ga).sum()} of {B} rows")
    for b in np.nonzero(ea != ga)[0]:
        # same logits on both sides, so only the softmax arithmetic differs (<= 5e-6 relative, asserted above): a
        # different accept bit must sit that close to its threshold u q = p
        k = int(min(ea[b], ga[b]))
        pk, qk = ref_p[b, k, dtok[b, k]], ref_q[b, k, dtok[b, k]]
        u = float(u24[b, k]) / 2.0 ** 24
        assert abs(pk - u * qk) <= 1e-5 * (pk + u * qk) + 1e-12, ("accept bit differs away from its threshold", b, k)
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


# ---- nucleus (top-p) truncation of the target rows ----------------------------------------------------------

@pytest.mark.parametrize("rows,V,temp,top_p", [(6, 4096, 1.0, 0.7), (3, 4104, 0.6, 0.3), (4, 151936, 1.0, 0.7),
                                               (2, 151936, 1.5, 0.95), (2, 8, 1.0, 0.5)])
def test_nucleus_set_is_the_oracles_on_the_device_weights(rows, V, temp, top_p):
    gmb, ctx = _ctx(V)
    rng = np.random.default_rng(70 + rows)
    x = (rng.standard_normal((rows, V)) * 3.0).astype(np.float32)
    x[0, : V // 2] = x[0, V // 2: 2 * (V // 2)]          # plenty of exact ties in the first row
    xin = _bf16(x)
    out = torch.zeros_like(xin)
    e = torch.zeros((rows, V), dtype=torch.float32, device="cuda")
    gmb.gm_nucleus(ctx, xin, rows, temp, top_p, out, e)
    assert gmb.gm_last_status(ctx) == 0
    xb, ob, ev = xin.float().cpu().numpy(), out.float().cpu().numpy(), e.cpu().numpy()
    kept = np.isfinite(ob)
    np.testing.assert_array_equal(ob[kept], xb[kept])                        # kept entries pass through unchanged
    assert np.isneginf(ob[~kept]).all()
    ref_e = np.exp2((xb.astype(np.float64) - xb.max(1, keepdims=True)) * (np.log2(np.e) / temp))
    assert np.abs(ev - ref_e).max() <= 5e-6
    for r in range(rows):
        want = osampler.nucleus_keep(ev[r], top_p)
        diff = np.nonzero(want != kept[r])[0]
        # distinct logits whose weights round to the same fp32 value may fall on either side of the cut
        assert len(diff) == 0 or (len(np.unique(ev[r][diff])) == 1 and ev[r][diff[0]] == ev[r][kept[r]].min()), (r, diff[:8])
        assert len(diff) <= 4
        lo = xb[r][kept[r]].min()
        assert (xb[r][~kept[r]] < lo).all() or len(diff)                      # a threshold on the logit
    # without the weight dump the result is the same
    out2 = torch.zeros_like(xin)
    gmb.gm_nucleus(ctx, xin, rows, temp, top_p, out2)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    ctx.close()


def test_accept_with_top_p_truncates_the_target_only():
    gmb, ctx = _ctx(8200, max_batch=8, max_k=3)
    B, K, V, top_p = 8, 3, 8200, 0.7
    tgt, drf = sampler_only_logits(B, K, V, sigma=0.9, seed=81)
    dtok = _draft_tokens(drf, seed=82)
    u24 = random_u24((B, K + 1), seed=83)
    args = (_bf16(tgt), _bf16(drf), torch.from_numpy(dtok).cuda(), torch.from_numpy(u24.astype(np.int32)).cuda(), 0, 0)

    def run():
        a = torch.zeros(B, dtype=torch.int32, device="cuda")
        t = torch.zeros(B, dtype=torch.int32, device="cuda")
        dp = torch.zeros((B, K + 1, V), dtype=torch.float32, device="cuda")
        dq = torch.zeros((B, K, V), dtype=torch.float32, device="cuda")
        gmb.gm_accept(ctx, None, B, K, 1.0, *args, a, t, dp, dq)
        assert gmb.gm_last_status(ctx) == 0
        return a.cpu().numpy(), t.cpu().numpy(), dp.cpu().numpy(), dq.cpu().numpy()

    a0, t0, p0, q0 = run()
    gmb.gm_set_top_p(ctx, top_p)
    a1, t1, p1, q1 = run()
    np.testing.assert_array_equal(q1, q0)                                    # the head's rows are untouched
    ref = osampler.nucleus_filter(osampler.softmax_probs(_bf16(tgt).float().cpu().numpy()), top_p)
    support_diff = ((p1 > 0) != (ref > 0)).sum()
    assert support_diff <= 2, support_diff                                   # a cut within rounding of a token's mass
    if support_diff == 0:
        assert np.abs(p1 - ref).max() <= 1e-5 * ref.max()
    np.testing.assert_allclose(p1.sum(-1), 1.0, atol=2e-5)
    assert ((p1 > 0).sum(-1) < (p0 > 0).sum(-1)).all()
    for b in range(B):                                                       # decisions: the oracle on the dumped rows
        ea, et, _ = osampler.decide(p1[b], q1[b], dtok[b], u24[b])
        assert (int(a1[b]), int(t1[b])) == (ea, et)
        assert p1[b, a1[b], t1[b]] > 0                                       # the final token lies in the nucleus
    gmb.gm_set_top_p(ctx, 1.0)
    a2, t2, p2, _ = run()
    np.testing.assert_array_equal(a2, a0)
    np.testing.assert_array_equal(t2, t0)
    np.testing.assert_array_equal(p2, p0)
    with pytest.raises(RuntimeError):
        gmb.gm_set_top_p(ctx, 0.0)
    ctx.close()


def test_nucleus_flat_negative_constant_and_peaked_rows():
    """Rows whose cut lies far below the maximum in key space (the kernel's key window has to slide), below zero,
    on a tie that spans the row, or right at the mode."""
    V, top_p = 8192, 0.9
    gmb, ctx = _ctx(V)
    rng = np.random.default_rng(91)
    x = np.zeros((6, V), np.float32)
    x[0] = rng.standard_normal(V) * 0.02                   # flat around zero: the cut is a small negative logit
    x[1] = -np.abs(rng.standard_normal(V)) * 4.0 - 1.0     # all negative
    x[2] = 1.25                                            # constant: one tie, everything kept
    x[3] = rng.standard_normal(V)
    x[3, 77] = 40.0                                        # one token holds all the mass
    x[4] = rng.standard_normal(V) * 1e-3 - 5.0             # flat, negative
    x[5] = np.where(rng.random(V) < 0.5, 3.0, -3.0)        # two ties
    xin = _bf16(x)
    out = torch.zeros_like(xin)
    e = torch.zeros((6, V), dtype=torch.float32, device="cuda")
    gmb.gm_nucleus(ctx, xin, 6, 1.0, top_p, out, e)
    assert gmb.gm_last_status(ctx) == 0
    kept, ev = np.isfinite(out.float().cpu().numpy()), e.cpu().numpy()
    for r in range(6):
        want = osampler.nucleus_keep(ev[r], top_p)
        diff = np.nonzero(want != kept[r])[0]
        assert len(diff) == 0 or len(np.unique(ev[r][diff])) == 1, (r, len(diff))
    assert kept[2].all() and kept[3].sum() == 1 and kept[3, 77]
    assert (xin[0].float().cpu().numpy()[kept[0]] < 0).any() and 0.85 * V < kept[0].sum() < 0.95 * V
    np.testing.assert_array_equal(kept[5], xin[5].float().cpu().numpy() > 0)
    ctx.close()
