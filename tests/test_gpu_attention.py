"""Paged multi-query decode attention (gm_attention) against the oracle's explicit-softmax attention."""
import numpy as np
import pytest
import torch

from oracle import model as omodel
from synth_inputs import ModelConfig, make_page_tables, bf16_round

pytestmark = pytest.mark.gpu


def _case(n_q, n_kv, hd, q_stride, lens, q_counts, seed, layers=2, layer=1):
    import paper_2609_16648_b200 as gmb
    B = len(lens)
    group = n_q // n_kv
    cfg = ModelConfig("a", layers, 64, n_q, n_kv, hd, 64, 8, batch=B, k=q_stride - 1 if q_stride > 1 else 1,
                      kv_len_min=0, kv_len_max=0, length_law="uniform")
    lens = np.asarray(lens)
    q_counts = np.asarray(q_counts, np.int32)
    total = lens + q_counts                                   # positions attended by the last query
    pt, npg = make_page_tables(total, 16, seed=seed, slack_pages=2)
    max_k = max(q_stride - 1, 1)
    packed = gmb.random_packed_weights(cfg, "cuda")
    ctx = gmb.Context(cfg, packed, B, max_k, pt.shape[1], npg, 4)
    rng = np.random.default_rng(seed)
    pool = np.zeros((layers, 2, npg, n_kv, 16, hd), np.float32)
    q_rows = 16 * ((q_stride * group + 15) // 16)
    qbuf = np.zeros((B, n_kv, q_rows, hd), np.float32)
    refs = []
    for b in range(B):
        S, n = int(total[b]), int(q_counts[b])
        k = bf16_round(rng.standard_normal((S, n_kv, hd)).astype(np.float32))
        v = bf16_round(rng.standard_normal((S, n_kv, hd)).astype(np.float32))
        q = bf16_round(rng.standard_normal((n, n_q, hd)).astype(np.float32) * 1.5)
        idx = np.arange(S)
        pool[layer, 0, pt[b, idx // 16], :, idx % 16, :] = k
        pool[layer, 1, pt[b, idx // 16], :, idx % 16, :] = v
        for j in range(n):
            for h in range(n_q):
                qbuf[b, h // group, j * group + h % group] = q[j, h]
        refs.append(omodel.attention(q, k, v, np.arange(lens[b], S), idx))
    out = torch.full((B * q_stride, n_q * hd), 7.0, dtype=torch.bfloat16, device="cuda")
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(device="cuda", dtype=dt)
    gmb.gm_attention(ctx, dev(qbuf, torch.bfloat16), dev(pool, torch.bfloat16), layer, dev(np.where(pt < 0, 0, pt), torch.int32),
                     dev(q_counts, torch.int32), dev(lens.astype(np.int32), torch.int32), B, q_stride, out)
    assert gmb.gm_last_status(ctx) == 0
    got = out.float().cpu().numpy().reshape(B, q_stride, n_q, hd)
    worst = 0.0
    for b in range(B):
        n = int(q_counts[b])
        err = np.abs(got[b, :n] - refs[b]).max() / np.abs(refs[b]).max()
        worst = max(worst, err)
        assert np.all(got[b, n:] == 7.0)                       # rows beyond q_count are untouched
    ctx.close()
    return worst


@pytest.mark.parametrize("n_q,n_kv,hd,q_stride", [(4, 2, 64, 4), (32, 8, 128, 4), (32, 8, 128, 1), (8, 1, 128, 4),
                                                  (32, 16, 64, 2), (32, 8, 128, 6), (16, 8, 128, 8)])
def test_ragged_batches(n_q, n_kv, hd, q_stride):
    lens = [0, 1, 15, 16, 17, 31, 200, 1000, 2500, 33]
    rng = np.random.default_rng(q_stride)
    counts = [int(rng.integers(1, q_stride + 1)) for _ in lens]
    counts[0] = q_stride                                       # empty cache: the queries only see themselves
    assert _case(n_q, n_kv, hd, q_stride, lens, counts, seed=3) < 1.5e-2


def test_one_long_sequence_is_split_over_every_cta():
    assert _case(32, 8, 128, 4, [32768 - 4], [4], seed=5, layers=1, layer=0) < 1.5e-2


def test_many_short_sequences():
    lens = list(np.random.default_rng(0).integers(0, 40, 200))
    assert _case(8, 2, 64, 2, lens, [1 + (i % 2) for i in range(200)], seed=6, layers=1, layer=0) < 1.5e-2


def test_capacity_is_reported_not_faulted():
    import paper_2609_16648_b200 as gmb
    cfg = ModelConfig("a", 1, 64, 4, 2, 64, 64, 8, batch=2, k=3, kv_len_min=0, kv_len_max=0, length_law="uniform")
    ctx = gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), 2, 3, 2, 8, 4)      # 2 pages per row = 32 positions
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device="cuda")
    out = z((8, 256), torch.bfloat16)
    gmb.gm_attention(ctx, z((2, 2, 16, 64), torch.bfloat16), z((1, 2, 8, 2, 16, 64), torch.bfloat16), 0,
                     z((2, 2), torch.int32), torch.tensor([4, 4], dtype=torch.int32, device="cuda"),
                     torch.tensor([10, 30], dtype=torch.int32, device="cuda"), 2, 4, out)
    assert gmb.gm_last_status(ctx) == gmb.GM_ERR_KV_CAPACITY
    with pytest.raises(gmb.GmError):
        gmb.gm_attention(ctx, z((2, 2, 16, 64), torch.bfloat16), z((1, 2, 8, 2, 16, 64), torch.bfloat16), 0,
                         z((2, 2), torch.int32), z((2,), torch.int32), z((2,), torch.int32), 2, 5, out)
    ctx.close()


@pytest.mark.parametrize("qs", [4, 6, 8], ids=["k3_one_tile", "k5_transposed", "k7_two_tiles"])
def test_4b_shape_batch_on_sampled_sequences(qs):
    """The benchmark's attention launch (64 sequences, KV uniform 1k..8k, 32 q / 8 kv heads, head_dim 128,
    4 queries per sequence; also 6 and 8 queries, which take the other two kernels): three sampled sequences
    against the oracle, every row finite."""
    import paper_2609_16648_b200 as gmb
    from synth_inputs import kv_lengths_uniform
    n_q, n_kv, hd, B = 32, 8, 128, 64
    lens = kv_lengths_uniform(B, 1024, 8192, seed=3).astype(np.int64)
    pt, npg = make_page_tables(lens + qs, 16, seed=7)
    cfg = ModelConfig("a", 1, 64, n_q, n_kv, hd, 64, 8, batch=B, k=qs - 1, kv_len_min=0, kv_len_max=0, length_law="uniform")
    ctx = gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), B, qs - 1, pt.shape[1], npg, 4)
    g = torch.Generator(device="cuda").manual_seed(1)
    pool = torch.randn((1, 2, npg, n_kv, 16, hd), device="cuda", generator=g).to(torch.bfloat16)
    q = torch.randn((B, n_kv, 16 * ((qs * 4 + 15) // 16), hd), device="cuda", generator=g).to(torch.bfloat16)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device="cuda", dtype=torch.int32)
    out = torch.zeros((B * qs, n_q * hd), dtype=torch.bfloat16, device="cuda")
    gmb.gm_attention(ctx, q, pool, 0, dev(np.where(pt < 0, 0, pt)), dev(np.full(B, qs)), dev(lens), B, qs, out)
    assert gmb.gm_last_status(ctx) == 0
    got = out.float().cpu().numpy().reshape(B, qs, n_q, hd)
    assert np.isfinite(got).all()
    pool_h, q_h = pool.float().cpu().numpy(), q.float().cpu().numpy()
    for b in (0, int(np.argmax(lens)), int(np.argmin(lens))):
        S = int(lens[b]) + qs
        idx = np.arange(S)
        k = pool_h[0, 0, pt[b, idx // 16], :, idx % 16, :]
        v = pool_h[0, 1, pt[b, idx // 16], :, idx % 16, :]
        qq = np.zeros((qs, n_q, hd))
        for j in range(qs):
            for h in range(n_q):
                qq[j, h] = q_h[b, h // 4, j * 4 + h % 4]
        ref = omodel.attention(qq, k, v, np.arange(lens[b], S), idx)
        assert np.abs(got[b] - ref).max() / np.abs(ref).max() < 1.5e-2
    ctx.close()


@pytest.mark.parametrize("n_q,n_kv,hd,q_stride", [(4, 2, 64, 4), (32, 8, 128, 4), (8, 1, 128, 3), (16, 8, 128, 8)])
def test_attention_backward_matches_the_oracle(n_q, n_kv, hd, q_stride):
    """gm_attention_backward against the oracle's attention_grad, sequence by sequence, on ragged lengths in shuffled pages.
    The last two sequences are chains of one sequence: their page-table rows share the pages of a common prefix and own
    the pages after it, so the prefix entries must collect the key / value gradients of both."""
    import paper_2609_16648_b200 as gmb
    from oracle import update as oupdate
    lens = [0, 15, 16, 40, 333, 77, 77]
    B = len(lens)
    group = n_q // n_kv
    rng = np.random.default_rng(9 + q_stride)
    q_counts = np.array([q_stride] + [int(rng.integers(1, q_stride + 1)) for _ in lens[1:]], np.int32)
    q_counts[-2:] = q_stride
    lens = np.asarray(lens)
    total = lens + q_counts
    layers, layer = 2, 1
    cfg = ModelConfig("a", layers, 64, n_q, n_kv, hd, 64, 8, batch=B, k=max(q_stride - 1, 1), kv_len_min=0, kv_len_max=0,
                      length_law="uniform")
    pt, npg = make_page_tables(total, 16, seed=4, slack_pages=2)
    shared = lens[-1] // 16                                   # whole pages of the common prefix (77 // 16 = 4)
    pt[-1, :shared] = pt[-2, :shared]
    ctx = gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), B, max(q_stride - 1, 1), pt.shape[1], npg, 4)
    pool = np.zeros((layers, 2, npg, n_kv, 16, hd), np.float32)
    q_rows = 16 * ((q_stride * group + 15) // 16)
    qbuf = np.zeros((B, n_kv, q_rows, hd), np.float32)
    dout = np.zeros((B, q_stride, n_q, hd), np.float32)
    qs, ks, vs = [], [], []
    for b in range(B):
        S, n = int(total[b]), int(q_counts[b])
        k = bf16_round(rng.standard_normal((S, n_kv, hd)).astype(np.float32))
        v = bf16_round(rng.standard_normal((S, n_kv, hd)).astype(np.float32))
        if b == B - 1:                                         # the second chain sees the first one's prefix entries
            k[:shared * 16], v[:shared * 16] = ks[-1][:shared * 16], vs[-1][:shared * 16]
        q = bf16_round(rng.standard_normal((n, n_q, hd)).astype(np.float32) * 1.5)
        idx = np.arange(S)
        pool[layer, 0, pt[b, idx // 16], :, idx % 16, :] = k
        pool[layer, 1, pt[b, idx // 16], :, idx % 16, :] = v
        for j in range(n):
            for h in range(n_q):
                qbuf[b, h // group, j * group + h % group] = q[j, h]
        dout[b, :n] = rng.standard_normal((n, n_q, hd)).astype(np.float32)
        dout[b, n:] = 5.0                                      # rows beyond q_count must be ignored
        qs.append(q); ks.append(k); vs.append(v)
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(device="cuda", dtype=dt)
    dq = torch.full((B * q_stride, n_q * hd), 7.0, dtype=torch.float32, device="cuda")
    dkp = torch.zeros((npg, n_kv, 16, hd), dtype=torch.float32, device="cuda")
    dvp = torch.zeros_like(dkp)
    gmb.gm_attention_backward(ctx, dev(qbuf, torch.bfloat16), dev(dout.reshape(B * q_stride, -1), torch.float32),
                              dev(pool, torch.bfloat16), layer, dev(np.where(pt < 0, 0, pt), torch.int32),
                              dev(q_counts, torch.int32), dev(lens.astype(np.int32), torch.int32), B, q_stride, dq, dkp, dvp)
    assert gmb.gm_last_status(ctx) == 0
    got_dq = dq.cpu().numpy().reshape(B, q_stride, n_q, hd)
    got_dk, got_dv = dkp.cpu().numpy().astype(np.float64), dvp.cpu().numpy().astype(np.float64)
    want_dk, want_dv = np.zeros_like(got_dk), np.zeros_like(got_dv)
    worst = 0.0
    for b in range(B):
        S, n = int(total[b]), int(q_counts[b])
        idx = np.arange(S)
        rdq, rdk, rdv = oupdate.attention_grad(dout[b, :n], qs[b], ks[b], vs[b], np.arange(lens[b], S), idx)
        worst = max(worst, np.abs(got_dq[b, :n] - rdq).max() / np.abs(rdq).max())
        assert np.all(got_dq[b, n:] == 0)
        np.add.at(want_dk, (pt[b, idx // 16], slice(None), idx % 16), rdk)
        np.add.at(want_dv, (pt[b, idx // 16], slice(None), idx % 16), rdv)
    assert worst < 2e-4, worst                                 # fp32 arithmetic on exact bf16 inputs
    assert np.abs(got_dk - want_dk).max() < 2e-4 * np.abs(want_dk).max()
    assert np.abs(got_dv - want_dv).max() < 2e-4 * np.abs(want_dv).max()
    prefix_pages = pt[-2, :shared]
    assert np.abs(want_dk[prefix_pages]).max() > 0              # the shared pages did collect terms (from both chains)
    ctx.close()
