"""Forward pass of the head update on the device (head-cache rebuild from recorded pairs, draft-path reconstruction
through virtual page tables, overlaps from the top-64 record, DCA / VGM objective) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import model as omodel, record as orecord, sampler as osampler, step as ostep, update as oupdate
from synth_inputs import get_config, make_page_tables, make_weights, random_prompts
from synth_inputs.weights import perturb_norm_weights

from helpers import rel_err

pytestmark = pytest.mark.gpu

TOL = 2e-2
T = 0.2          # sharpens the nearly flat random-init distributions so that chains get rejected


def _oracle_rollout(cfg, w, n_steps):
    B, K = cfg.batch, cfg.k
    prompts = random_prompts(B, cfg.prompt_len, cfg.vocab, seed=1)
    pt, npg = make_page_tables(np.full(B, 96), cfg.page_size, seed=7)
    hpt, hnpg = make_page_tables(np.full(B, 96), cfg.page_size, seed=8)
    st = ostep.prefill(w, cfg, prompts, pt, npg, hpt, hnpg, temperature=T, seed=5)
    cycles = []
    for it in range(n_steps):
        lens = [len(s.tokens) for s in st.seqs]
        start_h = [s.pending_hidden[-1].copy() for s in st.seqs]
        out = ostep.spec_step(w, cfg, st, K, T, seed=5)
        for b in range(B):
            cycles.append((b, orecord.cycle_record(start_h[b], out["draft_tok"][b], out["target_logits"][b],
                                                   out["accept_len"][b], lens[b], T)))
    seqs = []
    for s in st.seqs:
        kv = omodel.PagedKV(cfg.n_layers, cfg.n_kv_heads, cfg.head_dim, np.arange(16)[None, :], 16)
        H = omodel.target_forward(w, s.tokens[:-1], np.arange(len(s.tokens) - 1), kv, 0, cfg)
        seqs.append((omodel.round_bf16(H).astype(np.float64), list(s.tokens)))
    return st, cycles, seqs, hpt, hnpg


def test_head_update_forward_matches_the_oracle():
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(prompt_len=12)
    B, K, V, d = cfg.batch, cfg.k, cfg.vocab, cfg.d_model
    w = perturb_norm_weights(make_weights(cfg, 0))
    st, cycles, seqs, hpt, hnpg = _oracle_rollout(cfg, w, n_steps=5)
    n = len(cycles)
    assert any(r["accepted"] <= K for _, r in cycles) and any(r["accepted"] == K + 1 for _, r in cycles)

    ctx = gmb.Context(cfg, gmb.pack_weights(w), B, K, hpt.shape[1], hnpg, hnpg + 2 * n)     # spare pages for the chains
    gst = gmb.State(ctx, B, hpt, hpt)
    S = max(len(t) for _, t in seqs)
    seq_tok = np.zeros((B, S), np.int32)
    seq_hid = np.zeros((B, S, d), np.float32)
    seq_len = np.zeros(B, np.int32)
    for b, (H, toks) in enumerate(seqs):
        seq_tok[b, :len(toks)] = toks
        seq_hid[b, :len(toks) - 1] = H
        seq_len[b] = len(toks)
    tok_d = torch.from_numpy(seq_tok).cuda()
    hid_d = torch.from_numpy(seq_hid).to(device="cuda", dtype=torch.bfloat16)
    gmb.gm_head_prefill(ctx, gst, hid_d, tok_d, torch.from_numpy(seq_len).cuda(), int(seq_len.max()))
    assert gmb.gm_last_status(ctx) == 0
    # the rebuilt prefix cache = the oracle's head over the recorded pairs
    hkv = omodel.PagedKV(1, cfg.n_kv_heads, cfg.head_dim, hpt, hnpg + 2 * n, cfg.page_size)
    hkv.pool = gst.head_kv_pool.float().cpu().numpy().astype(np.float64)
    for b, (H, toks) in enumerate(seqs):
        L = len(toks)
        ref = omodel.PagedKV(1, cfg.n_kv_heads, cfg.head_dim, np.arange(8)[None, :], 8, cfg.page_size)
        omodel.head_forward(w, H, toks[1:], np.arange(L - 1), ref, 0, cfg)
        for got, want in zip(hkv.gather(0, b, L - 1), ref.gather(0, 0, L - 1)):
            assert rel_err(got, want) < TOL

    rec = gmb.Record(n, K, d)
    rec.start_hidden.copy_(torch.from_numpy(np.stack([r["start_hidden"] for _, r in cycles])).to(torch.bfloat16))
    rec.start_pos.copy_(torch.tensor([r["start_pos"] for _, r in cycles], dtype=torch.int32))
    rec.drafts.copy_(torch.from_numpy(np.stack([r["drafts"] for _, r in cycles]).astype(np.int32)))
    rec.top_index.copy_(torch.from_numpy(np.stack([r["top_index"] for _, r in cycles]).astype(np.int32)))
    rec.top_logprob.copy_(torch.from_numpy(np.stack([r["top_logprob"] for _, r in cycles])).to(torch.bfloat16))
    rec.accepted.copy_(torch.tensor([r["accepted"] for _, r in cycles], dtype=torch.int32))
    cycle_seq = torch.tensor([b for b, _ in cycles], dtype=torch.int32, device="cuda")
    scratch = torch.arange(hnpg, hnpg + 2 * n, dtype=torch.int32, device="cuda").reshape(n, 2)
    logits = torch.zeros((n, K, V), dtype=torch.bfloat16, device="cuda")
    shared = torch.as_tensor(hpt[hpt >= 0], device="cuda", dtype=torch.long)
    before = gst.head_kv_pool[:, :, shared].clone()
    states = torch.full((n, K, d), 7.0, dtype=torch.float32, device="cuda")
    gmb.gm_reconstruct(ctx, gst, n, K, cycle_seq, rec, tok_d, scratch, logits, head_states=states)   # 20 chains, 4 per pass
    assert gmb.gm_last_status(ctx) == 0
    logits_plain = torch.zeros_like(logits)
    gmb.gm_reconstruct(ctx, gst, n, K, cycle_seq, rec, tok_d, scratch, logits_plain)    # the call without the states: same logits
    assert torch.equal(logits_plain, logits)
    assert torch.equal(gst.head_kv_pool[:, :, shared], before)                         # chains wrote to their own pages only

    lg = logits.float().cpu().numpy()
    worst = 0.0
    ref_alpha = np.zeros((n, K))
    for i, (b, r) in enumerate(cycles):
        q, ref_lg = oupdate.reconstruct_chain(w, cfg, seqs[b][0], seqs[b][1], r["start_pos"], r["drafts"], T)
        worst = max(worst, rel_err(lg[i], ref_lg))
        ref_alpha[i] = oupdate.chain_alphas(r, q)
    assert worst < TOL, worst

    alpha = torch.zeros((n, K), dtype=torch.float32, device="cuda")
    gmb.gm_overlap(ctx, n, K, T, logits, rec, alpha)
    al = alpha.cpu().numpy()
    for i, (b, r) in enumerate(cycles):                     # the kernel itself: the oracle's overlap on the device's logits
        want = oupdate.chain_alphas(r, osampler.softmax_probs(lg[i], T))
        np.testing.assert_allclose(al[i], want, atol=3e-5)
    assert np.abs(al - ref_alpha).max() < 3e-2              # end to end: bf16 forward passes on both sides
    assert al.min() > 0 and al.max() <= 1 + 1e-4 and al.std() > 1e-3

    loss = torch.zeros(n, dtype=torch.float32, device="cuda")
    mean = torch.zeros(1, dtype=torch.float32, device="cuda")
    gmb.gm_dca_loss(ctx, n, K, alpha, rec.accepted, loss, mean)
    want = np.array([oupdate.dca_loss(al[i], cycles[i][1]["accepted"]) for i in range(n)])
    np.testing.assert_allclose(loss.cpu().numpy(), want, rtol=2e-5, atol=2e-6)
    assert float(mean[0]) == pytest.approx(want.mean(), rel=1e-5)
    ref_loss, _ = oupdate.head_update_loss(w, cfg, seqs, cycles, T)
    assert abs(float(mean[0]) - ref_loss) < 3e-2

    # first step of the backward pass: d mean / d logits, against the oracle on the device's logits
    grad = torch.full((n, K, V), 7.0, dtype=torch.bfloat16, device="cuda")
    gmb.gm_dca_grad(ctx, n, K, T, logits, rec, alpha, rec.accepted, grad)
    _check_grad(grad.float().cpu().numpy(), lg, [r for _, r in cycles], T)
    # with the row statistics handed over from the overlap pass: the same numbers
    lse = torch.zeros((n, K), dtype=torch.float32, device="cuda")
    alpha2 = torch.zeros_like(alpha)
    gmb.gm_overlap(ctx, n, K, T, logits, rec, alpha2, lse)
    assert torch.equal(alpha2, alpha)
    y = lg / T
    np.testing.assert_allclose(lse.cpu().numpy(), np.log(np.exp(y - y.max(-1, keepdims=True)).sum(-1)) + y.max(-1), rtol=0, atol=2e-5 * np.abs(y).max())
    grad2 = torch.full_like(grad, 7.0)
    gmb.gm_dca_grad(ctx, n, K, T, logits, rec, alpha, rec.accepted, grad2, lse)
    assert torch.equal(grad2, grad)

    # second step: through the shared LM head and the head's final norm, back to the head states
    st_np = states.cpu().numpy().astype(np.float64)
    # the states the reconstruction returned are the ones its logits came from (up to the bf16 normed state and logits)
    relg = rel_err(omodel.head_logits(w, st_np.reshape(n * K, d), cfg).reshape(n, K, V), lg)
    assert relg < TOL, relg
    gy = torch.full((n * K, d), 7.0, dtype=torch.float32, device="cuda")
    gs = torch.full((n * K, d), 7.0, dtype=torch.float32, device="cuda")
    gmb.gm_head_state_grad(ctx, n * K, grad, gy, states, gs)
    assert gmb.gm_last_status(ctx) == 0
    g_in = grad.float().cpu().numpy().astype(np.float64)                      # the device's own bf16 gradient rows
    want_gy = oupdate.lm_head_input_grad(g_in, omodel.round_bf16(w["lm_head"])).reshape(n * K, d)
    want_gs = oupdate.rmsnorm_grad(want_gy, st_np.reshape(n * K, d), omodel.round_bf16(w["head"]["final_norm"]), cfg.rms_eps)
    assert np.abs(want_gy).max() > 0
    assert rel_err(gy.cpu().numpy(), want_gy) < 2e-4                          # bf16 products, fp32 sums over 4096 terms
    assert rel_err(gs.cpu().numpy(), want_gs) < 2e-4
    live = np.array([[j < min(r["accepted"], K) for j in range(K)] for _, r in cycles]).reshape(-1)
    assert (gs.cpu().numpy()[~live] == 0).all() and (np.abs(gs.cpu().numpy()[live]).max(-1) > 0).all()
    # end to end against the oracle's own chain (its logits, its states): the direction of the update agrees
    ref_states = np.stack([oupdate.reconstruct_states(w, cfg, seqs[b][0], seqs[b][1], r["start_pos"], r["drafts"])
                           for b, r in cycles])
    assert rel_err(st_np, ref_states) < TOL
    ref_gs, _, _ = oupdate.head_update_grad_state(w, cfg, ref_states, [r for _, r in cycles], T)
    cos = (ref_gs.reshape(-1) * gs.cpu().numpy().reshape(-1)).sum() / (np.linalg.norm(ref_gs) * np.linalg.norm(gs.cpu().numpy()))
    assert cos > 0.98, cos
    # the projection alone, and a refreshed weight copy: the same numbers
    gy2 = torch.zeros_like(gy)
    gmb.gm_head_state_grad(ctx, n * K, grad, gy2, refresh_weights=True)
    assert torch.equal(gy2, gy)
    with pytest.raises(gmb.GmError):
        gmb.gm_head_state_grad(ctx, n * K, grad, gy, states, None)
    ctx.close()


def _check_grad(got, lg, recs, T):
    """Element-wise against the oracle's gradient.  A retained token whose q and p agree to fp32 rounding may take
    either slope (the objective has a kink there): such rows are left out, and must be rare."""
    n, K, V = got.shape
    want = oupdate.head_update_grad_logits(lg, recs, T)
    q = oupdate.softmax64(lg, T)
    skipped = 0
    for r, rec in enumerate(recs):
        L = min(rec["accepted"], K)
        assert (got[r, L:] == 0).all()                       # the verify gate: nothing after the first rejection
        for k in range(L):
            keep = rec["top_index"][k] >= 0
            pk = np.exp(rec["top_logprob"][k][keep].astype(np.float64))
            qk = q[r, k][rec["top_index"][k][keep]]
            near = np.abs(pk - qk) <= 1e-5 * np.maximum(pk, qk)
            res_near = abs(max(1 - pk.sum(), 0) - max(1 - qk.sum(), 0)) <= 1e-5
            if near.any() or res_near:
                skipped += 1
                continue
            scale = np.abs(want[r, k]).max()
            assert scale > 0
            # bf16 output: 2^-8 relative per element, on top of fp32 exponentials
            np.testing.assert_allclose(got[r, k], want[r, k], rtol=1.2e-2, atol=1e-3 * scale)
            assert abs(got[r, k].sum()) < 2e-2 * np.abs(got[r, k]).sum()
    assert skipped <= max(2, n * K // 20), skipped
    return skipped


def test_gradient_kernel_full_vocabulary_and_edge_cases():
    """gm_dca_grad alone at the 4B vocabulary (ragged tail of the vector loop: 151936 = 8 * 18992): synthetic head
    logits and records built by the oracle from synthetic target logits; dead chains, gated rows, K = 7."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(vocab=151936)
    n, K, V = 8, 7, cfg.vocab
    ctx = gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), 4, K, 4, 8, 8)
    rng = np.random.default_rng(11)
    Tg = 0.8
    head = omodel.round_bf16(rng.normal(0, 2.5, (n, K, V))).astype(np.float64)
    recs = []
    for r in range(n):
        tgt = omodel.round_bf16(head[r] + rng.normal(0, 1.0, (K, V)))
        full = orecord.cycle_record(np.zeros(cfg.d_model), np.zeros(K, np.int64),
                                    np.concatenate([tgt, tgt[:1]]), int(r % (K + 1)), 5, Tg)
        recs.append({"top_index": full["top_index"][:K], "top_logprob": full["top_logprob"][:K], "accepted": full["accepted"]})
    rec = gmb.Record(n, K, cfg.d_model)
    rec.top_index.copy_(torch.from_numpy(np.stack([r["top_index"] for r in recs]).astype(np.int32)))
    rec.top_logprob.copy_(torch.from_numpy(np.stack([r["top_logprob"] for r in recs])).to(torch.bfloat16))
    rec.accepted.copy_(torch.tensor([r["accepted"] for r in recs], dtype=torch.int32))
    logits = torch.from_numpy(head).to(device="cuda", dtype=torch.bfloat16)
    alpha = torch.zeros((n, K), dtype=torch.float32, device="cuda")
    lse = torch.zeros((n, K), dtype=torch.float32, device="cuda")
    gmb.gm_overlap(ctx, n, K, Tg, logits, rec, alpha, lse)
    grad = torch.full((n, K, V), 7.0, dtype=torch.bfloat16, device="cuda")
    gmb.gm_dca_grad(ctx, n, K, Tg, logits, rec, alpha, rec.accepted, grad, lse)
    assert gmb.gm_last_status(ctx) == 0
    got = grad.float().cpu().numpy()
    _check_grad(got, head, recs, Tg)
    assert any(r["accepted"] == 1 for r in recs) and any(r["accepted"] == K + 1 for r in recs)
    # argument checks of the update entry points: nothing is launched
    for bad in (dict(temperature=0.0), dict(temperature=float("nan")), dict(k=8), dict(n=0)):
        with pytest.raises(gmb.GmError) as e:
            gmb.gm_dca_grad(ctx, bad.get("n", n), bad.get("k", K), bad.get("temperature", Tg), logits, rec, alpha,
                            rec.accepted, grad, lse)
        assert e.value.code == (gmb.GM_ERR_UNSUPPORTED if "temperature" in bad else gmb.GM_ERR_INVALID_ARG)
    with pytest.raises(gmb.GmError) as e:
        gmb.gm_overlap(ctx, n, K, -1.0, logits, rec, alpha)
    assert e.value.code == gmb.GM_ERR_UNSUPPORTED
    with pytest.raises(gmb.GmError) as e:
        gmb.gm_dca_grad(ctx, n, K, Tg, logits, rec, None, rec.accepted, grad)
    assert e.value.code == gmb.GM_ERR_INVALID_ARG
    assert gmb.gm_last_status(ctx) == 0
    # a dead chain (first overlap 0) has no finite objective: its rows are written as zeros
    alpha[2, 0] = 0.0
    gmb.gm_dca_grad(ctx, n, K, Tg, logits, rec, alpha, rec.accepted, grad)
    g2 = grad.float().cpu().numpy()
    assert (g2[2] == 0).all() and np.array_equal(g2[[0, 1, 3, 4, 5, 6, 7]], got[[0, 1, 3, 4, 5, 6, 7]])
    ctx.close()


@pytest.mark.parametrize("rows", [192, 448], ids=["64x3", "two_token_blocks_ragged"])
def test_head_state_gradient_at_the_4b_dimensions(rows):
    """gm_head_state_grad alone at d = 2560, V = 151936: the projection contracts over 2374 K blocks (split along K over
    clusters at 192 rows; two token blocks, the second ragged, at 448).  Synthetic gradient rows with the structure
    gm_dca_grad writes: dense small values, a third of the rows exactly zero.  The oracle computes sampled rows."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(vocab=151936, d_model=2560)
    V, d = cfg.vocab, cfg.d_model
    ctx = gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), 4, 3, 4, 8, 8)
    g = torch.Generator(device="cuda").manual_seed(9)
    ctx.packed["head"]["final_norm"].copy_((1 + (torch.rand(d, device="cuda", generator=g) - 0.5) * 0.5).to(torch.bfloat16))
    grad = (torch.randn((rows, V), device="cuda", generator=g) * 1e-3).to(torch.bfloat16)
    grad[2::3] = 0
    states = torch.randn((rows, d), device="cuda", generator=g) * 3.0
    gy = torch.full((rows, d), 7.0, dtype=torch.float32, device="cuda")
    gs = torch.full((rows, d), 7.0, dtype=torch.float32, device="cuda")
    gmb.gm_head_state_grad(ctx, rows, grad, gy, states, gs)
    assert gmb.gm_last_status(ctx) == 0
    sample = sorted(set(np.random.default_rng(3).choice(rows, 24, replace=False).tolist()) | {0, 2, 255 % rows, rows - 1})
    w_lm = ctx.packed["lm_head"].double().cpu().numpy()
    want_gy = oupdate.lm_head_input_grad(grad[sample].double().cpu().numpy(), w_lm)
    want_gs = oupdate.rmsnorm_grad(want_gy, states[sample].double().cpu().numpy(),
                                   ctx.packed["head"]["final_norm"].double().cpu().numpy(), cfg.rms_eps)
    got_gy, got_gs = gy[sample].cpu().numpy(), gs[sample].cpu().numpy()
    assert rel_err(got_gy, want_gy) < 2e-4 and rel_err(got_gs, want_gs) < 2e-4     # fp32 sums over 151936 exact bf16 products
    zero = [i for i, r in enumerate(sample) if r % 3 == 2]
    assert zero and (got_gy[zero] == 0).all() and (got_gs[zero] == 0).all()
    assert not torch.isnan(gs).any() and float(gs[0::3].abs().max()) > 0
    # timing of the two launches (weights already transposed)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    for _ in range(3):
        gmb.gm_head_state_grad(ctx, rows, grad, gy, states, gs)
    ev[0].record()
    for _ in range(10):
        gmb.gm_head_state_grad(ctx, rows, grad, gy, states, gs)
    ev[1].record()
    torch.cuda.synchronize()
    ms = ev[0].elapsed_time(ev[1]) / 10
    print(f"gm_head_state_grad rows {rows}: {ms:.3f} ms per call, {(d * V * 2 + rows * V * 2) / ms / 1e6:.0f} GB/s of the "
          f"operands, {2.0 * rows * d * V / ms / 1e9:.0f} TFLOP/s")
    ctx.close()


@pytest.mark.parametrize("name,rows", [("tiny", 24), ("tiny", 100), ("4b", 192)], ids=["tiny-24", "tiny-100_ragged", "4b-192"])
def test_head_ffn_backward_matches_the_oracle(name, rows):
    """gm_head_ffn_backward on the head layer's feed-forward block against the oracle's fp64 backward of the same block
    (same bf16 weights, same fp32 inputs).  The device rounds the recomputed activations and the activation gradients
    to bf16 before each product, so tensors are compared by their largest entry; at the 4B dimensions (d 2560, F 9728)
    the weight gradients are compared on sampled rows."""
    import paper_2609_16648_b200 as gmb
    base = get_config("tiny")
    cfg = base if name == "tiny" else base.with_(d_model=2560, d_ffn=9728, vocab=4096)
    d, F = cfg.d_model, cfg.d_ffn
    ctx = gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), 4, 3, 4, 8, 8)
    g = torch.Generator(device="cuda").manual_seed(5)
    hl = ctx.packed["head"]["layer"]
    hl["ln2"].copy_((1 + (torch.rand(d, device="cuda", generator=g) - 0.5) * 0.5).to(torch.bfloat16))
    for key in ("w_gate_up", "w_down"):                       # larger than the init scale, so that the block's path matters
        hl[key].copy_((torch.randn(hl[key].shape, device="cuda", generator=g) * (2.0 / np.sqrt(hl[key].shape[1]))).to(torch.bfloat16))
    x = torch.randn((rows, d), device="cuda", generator=g) * 1.5
    dg = torch.randn((rows, d), device="cuda", generator=g) * 0.1
    dg[1::4] = 0                                               # rows without a gradient (after the first rejection)
    z = lambda *shape: torch.full(shape, 7.0, dtype=torch.float32, device="cuda")
    dx, dwgu, dwd, dln2 = z(rows, d), z(2 * F, d), z(d, F), z(d)
    gmb.gm_head_ffn_backward(ctx, rows, x, dg, dx, dwgu, dwd, dln2)
    assert gmb.gm_last_status(ctx) == 0
    f = lambda t: t.double().cpu().numpy()
    wgu = f(hl["w_gate_up"])
    lw = {"ln2": f(hl["ln2"]), "wg": wgu[0::2], "wu": wgu[1::2], "wd": f(hl["w_down"])}
    want = oupdate.ffn_block_grad(f(dg), f(x), lw, cfg.rms_eps)
    tol = 2.5e-2
    assert rel_err(f(dx), want["dx"]) < tol
    assert rel_err(f(dx) - f(dg), want["dx"] - f(dg)) < tol          # the block's own path, not hidden behind the residual one
    assert (f(dx)[1::4] == 0).all()                                    # no gradient in, none out
    assert rel_err(f(dln2), want["dln2"]) < tol
    rs = np.random.default_rng(2).choice(F, min(F, 64), replace=False)
    assert rel_err(f(dwgu)[0::2][rs], want["dwg"][rs]) < tol and rel_err(f(dwgu)[1::2][rs], want["dwu"][rs]) < tol
    cs = np.random.default_rng(3).choice(d, min(d, 64), replace=False)
    assert rel_err(f(dwd)[cs], want["dwd"][cs]) < tol
    assert np.abs(want["dwd"]).max() > 0 and np.abs(want["dwg"]).max() > 0
    # a second call with fewer rows reuses the scratch: same numbers as a fresh computation of that prefix
    r2 = rows // 2
    dx2, dwgu2, dwd2, dln22 = z(r2, d), z(2 * F, d), z(d, F), z(d)
    gmb.gm_head_ffn_backward(ctx, r2, x[:r2].contiguous(), dg[:r2].contiguous(), dx2, dwgu2, dwd2, dln22, refresh_weights=True)
    want2 = oupdate.ffn_block_grad(f(dg)[:r2], f(x)[:r2], lw, cfg.rms_eps)
    assert torch.equal(dx2, dx[:r2])
    assert rel_err(f(dwd2)[cs], want2["dwd"][cs]) < tol and rel_err(f(dln22), want2["dln2"]) < tol
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    for _ in range(2):
        gmb.gm_head_ffn_backward(ctx, rows, x, dg, dx, dwgu, dwd, dln2)
    ev[0].record()
    for _ in range(5):
        gmb.gm_head_ffn_backward(ctx, rows, x, dg, dx, dwgu, dwd, dln2)
    ev[1].record()
    torch.cuda.synchronize()
    ms = ev[0].elapsed_time(ev[1]) / 5
    print(f"gm_head_ffn_backward {name} rows {rows}: {ms:.3f} ms per call, {16.0 * rows * d * F / ms / 1e9:.0f} TFLOP/s "
          f"over its five products (the recomputed gate/up forward, two input gradients, two weight gradients)")
    ctx.close()


@pytest.mark.parametrize("name,rows,concat", [("tiny", 40, None), ("tiny", 40, "hidden_first"), ("4b", 192, None)],
                         ids=["tiny-40", "tiny-40-hidden_first", "4b-192"])
def test_head_input_backward_matches_the_oracle(name, rows, concat):
    """gm_head_input_backward against the oracle's fp64 backward of the head's input on the same bf16 weights: the hidden
    states' gradient (the recurrence term), the projection's and the two norm weights' gradients; both concatenation
    orders (the packed projection always takes [embedding ; hidden], so dproj comes back with its column halves swapped)."""
    import paper_2609_16648_b200 as gmb
    base = get_config("tiny")
    cfg = base if name == "tiny" else base.with_(d_model=2560, vocab=4096)
    d, V = cfg.d_model, cfg.vocab
    w = perturb_norm_weights(make_weights(cfg, 3))
    w["head"]["proj"] = np.random.default_rng(4).normal(0, 1.0 / np.sqrt(2 * d), (d, 2 * d)).astype(np.float32)
    if concat:
        w["head"]["concat"] = concat
    packed = gmb.pack_weights(w)
    ctx = gmb.Context(cfg, packed, 4, 3, 4, 8, 8)
    rng = np.random.default_rng(6)
    tokens = rng.integers(0, V, rows).astype(np.int32)
    hidden = rng.normal(0, 1.5, (rows, d)).astype(np.float32)
    dz = rng.normal(0, 0.1, (rows, d)).astype(np.float32)
    dz[2::5] = 0
    z = lambda *shape: torch.full(shape, 7.0, dtype=torch.float32, device="cuda")
    dh, dp, de, dhn = z(rows, d), z(d, 2 * d), z(d), z(d)
    cu = lambda a: torch.from_numpy(a).cuda()
    gmb.gm_head_input_backward(ctx, rows, cu(tokens), cu(hidden), cu(dz), dh, dp, de, dhn)
    assert gmb.gm_last_status(ctx) == 0
    r16 = lambda a: omodel.round_bf16(a).astype(np.float64)           # the oracle on the weights the device holds
    wo = {"embed": r16(w["embed"]), "head": {"enorm": r16(w["head"]["enorm"]), "hnorm": r16(w["head"]["hnorm"]),
                                             "proj": r16(w["head"]["proj"]), "concat": concat or "embedding_first"}}
    want = oupdate.head_input_grad(dz, wo, hidden, tokens, cfg)
    f = lambda t: t.double().cpu().numpy()
    tol = 2.5e-2
    assert rel_err(f(dh), want["dhidden"]) < tol and (f(dh)[2::5] == 0).all()
    want_dp = want["dproj"]
    if concat == "hidden_first":                                        # packed order is always [embedding ; hidden]
        want_dp = np.concatenate([want_dp[:, d:], want_dp[:, :d]], axis=1)
    assert rel_err(f(dp), want_dp) < tol
    assert rel_err(f(de), want["denorm"]) < tol and rel_err(f(dhn), want["dhnorm"]) < tol
    assert np.abs(want["denorm"]).max() > 0 and np.abs(want["dproj"]).max() > 0
    # a token id outside the vocabulary is reported, not dereferenced
    bad = cu(tokens.copy())
    bad[1] = V + 5
    gmb.gm_head_input_backward(ctx, rows, bad, cu(hidden), cu(dz), dh, dp, de, dhn)
    assert gmb.gm_last_status(ctx) == gmb.GM_ERR_BAD_PAGE
    ctx.close()


@pytest.mark.parametrize("name,family", [("tiny", "plain"), ("tiny", "qkv_bias"), ("tiny", "qk_norm"), ("4b", "qk_norm")],
                         ids=["tiny-plain", "tiny-qkv_bias", "tiny-qk_norm", "4b_heads-qk_norm"])
def test_head_attn_backward_matches_the_oracle(name, family):
    """gm_head_attn_backward against the oracle's backward of the attention half, sequence by sequence: ragged row counts
    at ragged prefix lengths in shuffled pages, gradient already sitting on every cache entry (the rows of later passes),
    and two chains of one sequence whose page tables share the prefix pages.  The rows' own cache entries are the oracle's
    keys / values of those rows rounded to bf16, on both sides."""
    import paper_2609_16648_b200 as gmb
    base = get_config("tiny").with_(n_layers=1, qkv_bias=family == "qkv_bias", qk_norm=family == "qk_norm")
    cfg = base if name == "tiny" else base.with_(d_model=2560, n_q_heads=32, n_kv_heads=8, head_dim=128)
    d, hd, n_q, n_kv, NQ, NKV = cfg.d_model, cfg.head_dim, cfg.n_q_heads, cfg.n_kv_heads, cfg.q_dim, cfg.kv_dim
    QT = 4
    lens = np.array([0, 15, 40, 333, 77, 77])
    B = len(lens)
    rng = np.random.default_rng(17)
    counts = np.array([QT, 1, 3, 2, QT, QT], np.int32)
    total = lens + counts
    pt, npg = make_page_tables(total, 16, seed=4, slack_pages=2)
    shared = lens[-1] // 16
    pt[-1, :shared] = pt[-2, :shared]
    ctx = gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), B, QT - 1, pt.shape[1], 8, npg)
    g = torch.Generator(device="cuda").manual_seed(5)
    hl = ctx.packed["head"]["layer"]
    pert = lambda n: (1 + (torch.rand(n, device="cuda", generator=g) - 0.5) * 0.5).to(torch.bfloat16)
    hl["ln1"].copy_(pert(d))
    for key in ("wqkv", "wo"):                                   # larger than the init scale, so that the block's path matters
        hl[key].copy_((torch.randn(hl[key].shape, device="cuda", generator=g) * (1.5 / np.sqrt(hl[key].shape[1]))).to(torch.bfloat16))
    if cfg.qkv_bias:
        hl["b_qkv"].copy_((torch.randn(NQ + 2 * NKV, device="cuda", generator=g) * 0.3).to(torch.bfloat16))
    if cfg.qk_norm:
        hl["q_norm"].copy_(pert(hd)); hl["k_norm"].copy_(pert(hd))
    f = lambda t: t.double().cpu().numpy()
    wqkv = f(hl["wqkv"])
    lw = {"ln1": f(hl["ln1"]), "wq": wqkv[:NQ], "wk": wqkv[NQ:NQ + NKV], "wv": wqkv[NQ + NKV:], "wo": f(hl["wo"])}
    if cfg.qkv_bias:
        bq = f(hl["b_qkv"])
        lw.update(bq=bq[:NQ], bk=bq[NQ:NQ + NKV], bv=bq[NQ + NKV:])
    if cfg.qk_norm:
        lw.update(qnorm=f(hl["q_norm"]), knorm=f(hl["k_norm"]))
    x = rng.normal(0, 1.5, (B, QT, d)).astype(np.float32)
    dxmid = rng.normal(0, 0.1, (B, QT, d)).astype(np.float32)
    pool = np.zeros((1, 2, npg, n_kv, 16, hd), np.float32)
    dk0 = np.zeros((npg, n_kv, 16, hd), np.float32)
    dv0 = np.zeros_like(dk0)
    kcs, vcs = [], []
    for b in range(B):
        S, n = int(total[b]), int(counts[b])
        dxmid[b, n:] = 0
        pos = lens[b] + np.arange(n)
        kc = omodel.round_bf16(rng.standard_normal((S, n_kv, hd))).astype(np.float64)
        vc = omodel.round_bf16(rng.standard_normal((S, n_kv, hd))).astype(np.float64)
        if b == B - 1:
            kc[:shared * 16], vc[:shared * 16] = kcs[-1][:shared * 16], vcs[-1][:shared * 16]
        _, k_own, v_own = omodel.project_qkv(lw, omodel.rmsnorm(x[b, :n], lw["ln1"], cfg.rms_eps), cfg)
        kc[pos] = omodel.round_bf16(omodel.rope(k_own, pos, cfg.rope_base))
        vc[pos] = omodel.round_bf16(v_own)
        idx = np.arange(S)
        pool[0, 0, pt[b, idx // 16], :, idx % 16, :] = kc
        pool[0, 1, pt[b, idx // 16], :, idx % 16, :] = vc
        dk0[pt[b, idx // 16], :, idx % 16, :] = rng.normal(0, 0.02, (S, n_kv, hd))
        dv0[pt[b, idx // 16], :, idx % 16, :] = rng.normal(0, 0.02, (S, n_kv, hd))
        kcs.append(kc); vcs.append(vc)
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(device="cuda", dtype=dt)
    z = lambda *shape: torch.full(shape, 7.0, dtype=torch.float32, device="cuda")
    dkp, dvp = dev(dk0, torch.float32), dev(dv0, torch.float32)
    dx, dwqkv, dwo, dln1 = z(B * QT, d), z(NQ + 2 * NKV, d), z(d, NQ), z(d)
    dbias = z(NQ + 2 * NKV) if cfg.qkv_bias else None
    dqkn = z(2 * hd) if cfg.qk_norm else None
    args = (ctx, dev(x.reshape(B * QT, d), torch.float32), dev(dxmid.reshape(B * QT, d), torch.float32), dev(pool, torch.bfloat16),
            dev(np.where(pt < 0, 0, pt), torch.int32), dev(counts, torch.int32), dev(lens.astype(np.int32), torch.int32), B, QT)
    pool_before = args[3].clone()
    gmb.gm_head_attn_backward(*args, dkp, dvp, dx, dwqkv, dwo, dln1, dbias, dqkn)
    assert gmb.gm_last_status(ctx) == 0
    assert torch.equal(args[3], pool_before)                                # the cache is read, not rewritten
    want = {}
    want_dk, want_dv = dk0.astype(np.float64), dv0.astype(np.float64)
    got_dx = f(dx).reshape(B, QT, d)
    tol = 2.5e-2
    for b in range(B):
        S, n = int(total[b]), int(counts[b])
        idx = np.arange(S)
        pg, sl = pt[b, idx // 16], idx % 16
        dkc, dvc = dk0[pg, :, sl, :].astype(np.float64), dv0[pg, :, sl, :].astype(np.float64)
        before_k, before_v = dkc.copy(), dvc.copy()
        out = oupdate.attention_block_grad(dxmid[b, :n], x[b, :n], lw, lens[b] + np.arange(n), kcs[b], vcs[b], dkc, dvc, cfg)
        np.add.at(want_dk, (pg, slice(None), sl), dkc - before_k)
        np.add.at(want_dv, (pg, slice(None), sl), dvc - before_v)
        assert rel_err(got_dx[b, :n], out["dx"]) < tol, b
        assert rel_err(got_dx[b, :n] - dxmid[b, :n], out["dx"] - dxmid[b, :n]) < tol, b       # the attention half's own path
        assert (got_dx[b, n:] == 0).all()
        for key, val in out.items():
            if key != "dx":
                want[key] = want.get(key, 0.0) + val
    # what this pass added to the planes (the device rounds the queries, the attention output's gradient enters in fp32)
    assert rel_err(f(dkp) - dk0, want_dk - dk0) < tol and rel_err(f(dvp) - dv0, want_dv - dv0) < tol
    assert np.abs((want_dk - dk0)[pt[-2, :shared]]).max() > 0                      # the shared prefix pages collected terms
    got_w = f(dwqkv)
    assert rel_err(got_w[:NQ], want["dwq"]) < tol and rel_err(got_w[NQ:NQ + NKV], want["dwk"]) < tol
    assert rel_err(got_w[NQ + NKV:], want["dwv"]) < tol
    assert rel_err(f(dwo), want["dwo"]) < tol and rel_err(f(dln1), want["dln1"]) < tol
    if cfg.qkv_bias:
        assert rel_err(f(dbias), np.concatenate([want["dbq"], want["dbk"], want["dbv"]])) < tol
    if cfg.qk_norm:
        assert rel_err(f(dqkn)[:hd], want["dqnorm"]) < tol and rel_err(f(dqkn)[hd:], want["dknorm"]) < tol
    for key in ("dwq", "dwk", "dwv", "dwo", "dln1"):
        assert np.abs(want[key]).max() > 0
    # a layer's optional outputs must be asked for exactly when the layer has them
    with pytest.raises(RuntimeError):
        gmb.gm_head_attn_backward(*args, dkp, dvp, dx, dwqkv, dwo, dln1, None if cfg.qkv_bias else z(NQ + 2 * NKV), dqkn)
    ctx.close()


def _update_setup(family, n_steps=3, dims="tiny", prompt_len=12, k=3, max_k=None):
    """A short oracle rollout with its records, and a device context / state / record holding the same cycles."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny").with_(prompt_len=prompt_len, qk_norm=family == "qk_norm", qkv_bias=family == "qkv_bias", k=k)
    if dims == "4b":                                     # the 4B head's layer (one backbone layer, a small vocabulary)
        cfg = cfg.with_(n_layers=1, d_model=2560, n_q_heads=32, n_kv_heads=8, head_dim=128, d_ffn=9728)
    B, K, V, d = cfg.batch, cfg.k, cfg.vocab, cfg.d_model
    w = perturb_norm_weights(make_weights(cfg, 0))
    st, cycles, seqs, hpt, hnpg = _oracle_rollout(cfg, w, n_steps=n_steps)
    if not any(r["accepted"] >= 2 for _, r in cycles):
        # random weights of this size reject every first draft; the objective is defined for any first rejected position,
        # so spread it over 1 .. K + 1 for the chains to reach the recurrence
        cycles = [(b_, dict(r, accepted=i % (K + 1) + 1)) for i, (b_, r) in enumerate(cycles)]
    n = len(cycles)
    assert any(r["accepted"] >= 2 for _, r in cycles)                     # some chains reach the recurrence
    ctx = gmb.Context(cfg, gmb.pack_weights(w), B, max_k or K, hpt.shape[1], hnpg, hnpg + 2 * n)
    gst = gmb.State(ctx, B, hpt, hpt)
    S = max(len(t) for _, t in seqs)
    seq_tok, seq_hid, seq_len = np.zeros((B, S), np.int32), np.zeros((B, S, d), np.float32), np.zeros(B, np.int32)
    for b, (H, toks) in enumerate(seqs):
        seq_tok[b, :len(toks)] = toks
        seq_hid[b, :len(toks) - 1] = H
        seq_len[b] = len(toks)
    tok_d, len_d = torch.from_numpy(seq_tok).cuda(), torch.from_numpy(seq_len).cuda()
    hid_d = torch.from_numpy(seq_hid).to(device="cuda", dtype=torch.bfloat16)
    rec = gmb.Record(n, K, d)
    rec.start_hidden.copy_(torch.from_numpy(np.stack([r["start_hidden"] for _, r in cycles])).to(torch.bfloat16))
    rec.start_pos.copy_(torch.tensor([r["start_pos"] for _, r in cycles], dtype=torch.int32))
    rec.drafts.copy_(torch.from_numpy(np.stack([r["drafts"] for _, r in cycles]).astype(np.int32)))
    rec.top_index.copy_(torch.from_numpy(np.stack([r["top_index"] for _, r in cycles]).astype(np.int32)))
    rec.top_logprob.copy_(torch.from_numpy(np.stack([r["top_logprob"] for _, r in cycles])).to(torch.bfloat16))
    rec.accepted.copy_(torch.tensor([r["accepted"] for _, r in cycles], dtype=torch.int32))
    cycle_seq = torch.tensor([b for b, _ in cycles], dtype=torch.int32, device="cuda")
    scratch = torch.arange(hnpg, hnpg + 2 * n, dtype=torch.int32, device="cuda").reshape(n, 2)
    return dict(gmb=gmb, cfg=cfg, w=w, cycles=cycles, seqs=seqs, n=n, ctx=ctx, gst=gst, tok_d=tok_d, len_d=len_d, hid_d=hid_d,
                max_len=int(seq_len.max()), rec=rec, cycle_seq=cycle_seq, scratch=scratch, hnpg=hnpg)


@pytest.mark.parametrize("family,dims,prompt_len,k,max_k",
                         [("plain", "tiny", 12, 3, 3), ("qk_norm", "tiny", 12, 3, 3), ("qkv_bias", "tiny", 12, 3, 3),
                          ("qk_norm", "4b", 12, 3, 3), ("plain", "tiny", 1, 3, 3), ("qk_norm", "tiny", 15, 3, 3),
                          ("plain", "tiny", 12, 2, 4), ("plain", "tiny", 12, 5, 5)],
                         ids=["plain", "qk_norm", "qkv_bias", "qk_norm-4b_head_dimensions", "plain-one_token_prompts",
                              "qk_norm-first_chain_entry_on_a_page_boundary", "plain-k2_in_a_context_of_max_k4", "plain-k5"])
def test_head_update_backward_matches_the_oracle(family, dims, prompt_len, k, max_k):
    """gm_head_update_backward - the whole backward pass over recorded cycles, chains replayed three chunks of max_batch
    at a time - against the oracle's head_update_grad on the weights the device holds, both starting from the device's
    own logit gradients (the piecewise-linear overlap picks its branches from the logits, which differ in rounding).
    Every parameter tensor of the head; the oracle's is pinned by finite differences of the objective."""
    # one-token prompts: the first cycle starts at length 2, its chain's first entry is position 0 and its prefix is empty;
    # 15-token prompts: length 16 + 2 at the second cycle or so puts a chain's first entry at slot 0 of a page (nothing to fold)
    u = _update_setup(family, n_steps=3 if dims == "tiny" else 2, dims=dims, prompt_len=prompt_len, k=k, max_k=max_k)
    gmb, cfg, w, cycles, seqs, n, ctx, gst = (u[k_] for k_ in ("gmb", "cfg", "w", "cycles", "seqs", "n", "ctx", "gst"))
    tok_d, len_d, hid_d, rec, cycle_seq, scratch, hnpg = (u[k_] for k_ in ("tok_d", "len_d", "hid_d", "rec", "cycle_seq", "scratch", "hnpg"))
    B, K, V, d = cfg.batch, cfg.k, cfg.vocab, cfg.d_model
    if prompt_len == 1:
        assert any(r["start_pos"] == 2 for _, r in cycles)
    if prompt_len == 15:
        assert any((r["start_pos"] - 2) % 16 == 0 for _, r in cycles)
    gmb.gm_head_prefill(ctx, gst, hid_d, tok_d, len_d, u["max_len"])
    logits = torch.zeros((n, K, V), dtype=torch.bfloat16, device="cuda")
    gmb.gm_reconstruct(ctx, gst, n, K, cycle_seq, rec, tok_d, scratch, logits)
    alpha = torch.zeros((n, K), dtype=torch.float32, device="cuda")
    gmb.gm_overlap(ctx, n, K, T, logits, rec, alpha)
    grad = torch.zeros((n, K, V), dtype=torch.bfloat16, device="cuda")
    gmb.gm_dca_grad(ctx, n, K, T, logits, rec, alpha, rec.accepted, grad)
    npg_h = hnpg + 2 * n
    dkp = torch.full((npg_h, cfg.n_kv_heads, 16, cfg.head_dim), 7.0, dtype=torch.float32, device="cuda")
    dvp = torch.full_like(dkp, 7.0)
    grads = gmb.head_grad_buffers(cfg)
    for t in grads.values():
        t.fill_(7.0)                                                       # outputs are overwritten, not added to
    pool_before = gst.head_kv_pool.clone()
    gmb.gm_head_update_backward(ctx, gst, n, K, cycle_seq, rec, tok_d, scratch, grad, hid_d, len_d, u["max_len"], dkp, dvp, grads)
    assert gmb.gm_last_status(ctx) == 0
    assert torch.equal(gst.head_kv_pool, pool_before)                      # the replay rewrites the chains' pages with the same values
    # a second call gives the same bits: the cache entries' gradients are summed in fixed point, everything else in a fixed order
    first = {k_: t.clone() for k_, t in grads.items()}
    dk1, dv1 = dkp.clone(), dvp.clone()
    gmb.gm_head_update_backward(ctx, gst, n, K, cycle_seq, rec, tok_d, scratch, grad, hid_d, len_d, u["max_len"], dkp, dvp, grads)
    assert all(torch.equal(grads[k_], first[k_]) for k_ in grads) and torch.equal(dkp, dk1) and torch.equal(dvp, dv1)
    # the oracle on the device's weights and the device's logit gradients
    r16 = lambda a: omodel.round_bf16(a).astype(np.float64)
    w16 = {"embed": r16(w["embed"]), "lm_head": r16(w["lm_head"]),
           "head": {k_: (r16(v_) if k_ != "layer" else {n_: r16(a_) for n_, a_ in v_.items()}) for k_, v_ in w["head"].items() if k_ != "concat"}}
    want = oupdate.head_update_grad(w16, cfg, seqs, cycles, T, grad_logits=grad.double().cpu().numpy())
    f = lambda t: t.double().cpu().numpy()
    NQ, NKV = cfg.q_dim, cfg.kv_dim
    got = {"proj": f(grads["proj"]), "enorm": f(grads["enorm"]), "hnorm": f(grads["hnorm"]), "final_norm": f(grads["final_norm"])}
    gl = {"ln1": f(grads["ln1"]), "ln2": f(grads["ln2"]), "wq": f(grads["wqkv"])[:NQ], "wk": f(grads["wqkv"])[NQ:NQ + NKV],
          "wv": f(grads["wqkv"])[NQ + NKV:], "wo": f(grads["wo"]), "wg": f(grads["w_gate_up"])[0::2], "wu": f(grads["w_gate_up"])[1::2],
          "wd": f(grads["w_down"])}
    if cfg.qkv_bias:
        bq = f(grads["b_qkv"])
        gl.update(bq=bq[:NQ], bk=bq[NQ:NQ + NKV], bv=bq[NQ + NKV:])
    if cfg.qk_norm:
        gl.update(qnorm=f(grads["qk_norm"])[:cfg.head_dim], knorm=f(grads["qk_norm"])[cfg.head_dim:])
    assert set(gl) == set(want["layer"])
    errs = {k_: rel_err(v_, want[k_]) for k_, v_ in got.items()}
    errs.update({"layer." + k_: rel_err(v_, want["layer"][k_]) for k_, v_ in gl.items()})
    print({k_: round(v_, 4) for k_, v_ in errs.items()})
    for k_, e in errs.items():
        assert e < 2e-2, (k_, e)
    ctx.close()


HEAD_TENSORS = ("proj", "enorm", "hnorm", "final_norm")


def _head_params(packed):
    out = {n_: packed["head"][n_] for n_ in HEAD_TENSORS}
    out.update({"layer." + n_: t for n_, t in packed["head"]["layer"].items()})
    return out


@pytest.mark.parametrize("family", ["plain", "qk_norm"])
def test_head_update_steps_lower_the_objective_and_equal_the_calls_made_one_by_one(family):
    """gm_head_update_step (Alg. 1, "update phi" as one call).  (1) Its first update leaves exactly the parameters that the
    public calls it is made of leave when made one by one on a second context (cache rebuild, reconstruction, overlap,
    loss, logit gradients, backward pass, AdamW per tensor from fp32 copies of the bf16 parameters and zero moments).
    (2) Repeated on the same recorded cycles with the head's schedule, it lowers the objective it reports - the mean of
    Eq. 9 before each update - i.e. the head's acceptance on those cycles rises; the backbone's tensors never change."""
    u = _update_setup(family)
    gmb, cfg, n, ctx, gst = u["gmb"], u["cfg"], u["n"], u["ctx"], u["gst"]
    K, V, d = cfg.k, cfg.vocab, cfg.d_model
    common = (u["cycle_seq"], u["rec"], u["tok_d"], u["scratch"])
    frozen = {k_: ctx.packed[k_].clone() for k_ in ("embed", "lm_head", "final_norm")}
    frozen["l0.wqkv"] = ctx.packed["layers"][0]["wqkv"].clone()
    before = {k_: t.clone() for k_, t in _head_params(ctx.packed).items()}
    mean = torch.zeros(1, dtype=torch.float32, device="cuda")
    peak, steps = 2e-3, 8
    f32 = lambda x: float(np.float32(x))
    lr1 = f32(oupdate.head_lr(0, peak, steps, warmup=2))
    with pytest.raises(gmb.GmError):                                      # updates are numbered from 1, in order
        gmb.gm_head_update_step(ctx, gst, n, K, T, *common, u["hid_d"], u["len_d"], u["max_len"], 2, lr1, mean)
    gmb.gm_head_update_step(ctx, gst, n, K, T, *common, u["hid_d"], u["len_d"], u["max_len"], 1, lr1, mean)
    assert gmb.gm_last_status(ctx) == 0
    losses = [float(mean[0])]
    after1 = {k_: t.clone() for k_, t in _head_params(ctx.packed).items()}
    # every matrix moved; a norm weight near 1 has a bf16 spacing of 2^-7, which one step of 1e-3 does not cross - the
    # fp32 master copy carries it
    assert all(not torch.equal(after1[k_], before[k_]) for k_ in after1 if after1[k_].dim() == 2)

    # (1) the same update, call by call, on a second context with its own copy of the weights
    u2 = _update_setup(family)
    c2, g2 = u2["ctx"], u2["gst"]
    gmb.gm_head_prefill(c2, g2, u2["hid_d"], u2["tok_d"], u2["len_d"], u2["max_len"])
    logits = torch.zeros((n, K, V), dtype=torch.bfloat16, device="cuda")
    gmb.gm_reconstruct(c2, g2, n, K, u2["cycle_seq"], u2["rec"], u2["tok_d"], u2["scratch"], logits)
    alpha, lse = torch.zeros((n, K), device="cuda"), torch.zeros((n, K), device="cuda")
    gmb.gm_overlap(c2, n, K, T, logits, u2["rec"], alpha, lse)
    loss, mean2 = torch.zeros(n, device="cuda"), torch.zeros(1, device="cuda")
    gmb.gm_dca_loss(c2, n, K, alpha, u2["rec"].accepted, loss, mean2)
    assert float(mean2[0]) == losses[0]
    grad = torch.zeros((n, K, V), dtype=torch.bfloat16, device="cuda")
    gmb.gm_dca_grad(c2, n, K, T, logits, u2["rec"], alpha, u2["rec"].accepted, grad, lse)
    npg_h = u2["hnpg"] + 2 * n
    dkp = torch.zeros((npg_h, cfg.n_kv_heads, 16, cfg.head_dim), dtype=torch.float32, device="cuda")
    grads = gmb.head_grad_buffers(cfg)
    gmb.gm_head_update_backward(c2, g2, n, K, u2["cycle_seq"], u2["rec"], u2["tok_d"], u2["scratch"], grad, u2["hid_d"], u2["len_d"],
                                u2["max_len"], dkp, torch.zeros_like(dkp), grads)
    hd = cfg.head_dim
    gmap = {"proj": grads["proj"], "enorm": grads["enorm"], "hnorm": grads["hnorm"], "final_norm": grads["final_norm"],
            "layer.ln1": grads["ln1"], "layer.ln2": grads["ln2"], "layer.wqkv": grads["wqkv"], "layer.wo": grads["wo"],
            "layer.w_gate_up": grads["w_gate_up"], "layer.w_down": grads["w_down"]}
    if family == "qk_norm":
        gmap.update({"layer.q_norm": grads["qk_norm"][:hd].contiguous(), "layer.k_norm": grads["qk_norm"][hd:].contiguous()})
    p2 = _head_params(c2.packed)
    assert set(p2) == set(gmap)
    for name, t in p2.items():
        master = t.float().reshape(-1).contiguous()
        gmb.gm_adamw_step(c2, master, gmap[name].reshape(-1), torch.zeros_like(master), torch.zeros_like(master), 1, lr1, param_bf16=t)
        assert torch.equal(t, after1[name]), name
    c2.close()

    # (2) more updates on the same cycles
    for s_ in range(1, steps):
        gmb.gm_head_update_step(ctx, gst, n, K, T, *common, u["hid_d"], u["len_d"], u["max_len"], s_ + 1,
                                f32(oupdate.head_lr(s_, peak, steps, warmup=2)), mean)
        losses.append(float(mean[0]))
    assert gmb.gm_last_status(ctx) == 0
    print("mean objective before each update:", [round(x, 4) for x in losses])
    assert all(np.isfinite(losses))
    assert losses[-1] < losses[0] - 0.02 and min(losses[1:]) < losses[0]
    assert torch.equal(ctx.packed["lm_head"], frozen["lm_head"]) and torch.equal(ctx.packed["embed"], frozen["embed"])
    assert torch.equal(ctx.packed["final_norm"], frozen["final_norm"]) and torch.equal(ctx.packed["layers"][0]["wqkv"], frozen["l0.wqkv"])
    ctx.close()


@pytest.mark.parametrize("n_seq,L,n", [(8, 512, 64), (64, 512, 256)], ids=["8x512_64_cycles", "64x512_256_cycles"])
def test_head_update_step_at_the_4b_head_dimensions_runs_and_is_timed(n_seq, L, n):
    """gm_head_update_step on the 4B head (d 2560, 32/8 heads of 128, FFN 9728, head norms, the full 151936 vocabulary) over
    synthetic records: n cycles spread over n_seq recorded sequences of L positions, k = 3, chains in chunks of 64.  There
    is no oracle at this size (the 4B-dimension parity case of the backward pass runs on a small vocabulary); this checks
    that the call runs clean at the full shapes - status, finite objective, every matrix of the head moved, the backbone's
    tensors untouched - and prints the time per update."""
    import paper_2609_16648_b200 as gmb
    K = 3
    cfg = get_config("4b").with_(n_layers=1, batch=n_seq, qk_norm=True)
    d, V = cfg.d_model, cfg.vocab
    hpt, hnpg = make_page_tables(np.full(n_seq, L + 8), 16, seed=8)
    ctx = gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), 64, K, hpt.shape[1], 8, hnpg + 2 * n)
    gst = gmb.State(ctx, n_seq, hpt, hpt)
    g = torch.Generator(device="cuda").manual_seed(1)
    tok = torch.randint(0, V, (n_seq, L), device="cuda", generator=g, dtype=torch.int32)
    hid = torch.randn((n_seq, L, d), device="cuda", generator=g).to(torch.bfloat16)
    slen = torch.full((n_seq,), L, dtype=torch.int32, device="cuda")
    rng = np.random.default_rng(3)
    seq = rng.integers(0, n_seq, n).astype(np.int32)
    start = rng.integers(L // 2, L - K - 1, n).astype(np.int32)
    rec = gmb.Record(n, K, d)
    rec.start_pos.copy_(torch.from_numpy(start))
    rec.start_hidden.copy_(hid[torch.from_numpy(seq).long().cuda(), torch.from_numpy(start - 2).long().cuda()])
    rec.drafts.copy_(torch.randint(0, V, (n, K), device="cuda", generator=g, dtype=torch.int32))
    order = torch.rand((n * K, V), device="cuda", generator=g).topk(64, dim=-1).indices            # 64 distinct ids per row
    rec.top_index.copy_(order.reshape(n, K, 64).to(torch.int32))
    lp = torch.log_softmax(torch.randn((n, K, 64), device="cuda", generator=g) * 2, -1) - 0.3     # 26 % of the mass in the residual bin
    rec.top_logprob.copy_(lp.sort(dim=-1, descending=True).values.to(torch.bfloat16))
    rec.accepted.copy_(torch.randint(1, K + 2, (n,), device="cuda", generator=g, dtype=torch.int32))
    cyc = torch.from_numpy(seq).cuda()
    scratch = torch.arange(hnpg, hnpg + 2 * n, dtype=torch.int32, device="cuda").reshape(n, 2)
    mean = torch.zeros(1, device="cuda")
    before = {k_: t.clone() for k_, t in _head_params(ctx.packed).items()}
    lm_head = ctx.packed["lm_head"].clone()
    losses, ev = [], [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    for s_ in range(1, 6):
        if s_ == 3:
            ev[0].record()
        gmb.gm_head_update_step(ctx, gst, n, K, 1.0, cyc, rec, tok, scratch, hid, slen, L, s_, 1e-4, mean)
        losses.append(float(mean[0]))
    ev[1].record()
    torch.cuda.synchronize()
    assert gmb.gm_last_status(ctx) == 0
    assert all(np.isfinite(losses)), losses
    after = _head_params(ctx.packed)
    assert all(not torch.equal(after[k_], before[k_]) for k_ in after if after[k_].dim() == 2)
    assert torch.equal(ctx.packed["lm_head"], lm_head)
    print(f"gm_head_update_step, 4B head, {n} cycles over {n_seq} x {L} positions: {ev[0].elapsed_time(ev[1]) / 3:.1f} ms per update; "
          f"objective before each update {[round(x, 4) for x in losses]}")
    ctx.close()


@pytest.mark.parametrize("n", [1003, 49_807_360], ids=["ragged_1003", "gate_up_of_the_4b_head"])
def test_adamw_step_matches_the_oracle(n):
    """gm_adamw_step over several updates with the head's schedule against the oracle's fp64 AdamW (sampled entries at the
    size of the 4B head's gate/up matrix, 19456 x 2560), the rewritten bf16 copy, argument checks, and the pass's bandwidth."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny")
    ctx = gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), 4, 3, 4, 8, 8)
    g = torch.Generator(device="cuda").manual_seed(12)
    p = torch.randn(n, device="cuda", generator=g) * 0.05
    m, v = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    pb = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    idx = torch.from_numpy(np.unique(np.concatenate([np.random.default_rng(1).integers(0, n, 4000), [0, n - 1, n - 2, n - 3]]))).cuda()
    po, mo, vo = (t[idx].double().cpu().numpy() for t in (p, m, v))
    steps, peak = 4, 3e-4
    f32 = lambda x: float(np.float32(x))                               # the C ABI takes the coefficients as floats: same values on both sides
    b1, b2, eps, wd = f32(0.9), f32(0.999), f32(1e-8), f32(0.01)
    for t in range(1, steps + 1):
        grad = torch.randn(n, device="cuda", generator=g) * (0.02 * t)
        grad[::7] = 0                                                  # entries without a gradient still decay
        lr = f32(oupdate.head_lr(t - 1, peak, 100))
        scale = 0.5 if t == 3 else 1.0                                 # a clipped update
        gmb.gm_adamw_step(ctx, p, grad, m, v, t, lr, param_bf16=pb, beta1=b1, beta2=b2, eps=eps, weight_decay=wd, grad_scale=scale)
        po, mo, vo = oupdate.adamw_step(po, scale * grad[idx].double().cpu().numpy(), mo, vo, t, lr, b1, b2, eps, wd)
    assert gmb.gm_last_status(ctx) == 0
    got = p[idx].double().cpu().numpy()
    # fp32 arithmetic: the parameter to an ulp or two, the accumulated movement (about steps * lr) to 1e-5 of itself
    np.testing.assert_allclose(got, po, rtol=3e-7, atol=steps * peak * 1e-5)
    np.testing.assert_allclose(m[idx].double().cpu().numpy(), mo, rtol=1e-5, atol=3e-8)      # gradients of both signs cancel in m
    np.testing.assert_allclose(v[idx].double().cpu().numpy(), vo, rtol=1e-5, atol=1e-12)
    assert torch.equal(pb, p.to(torch.bfloat16))
    for bad in (dict(beta1=1.0), dict(beta2=-0.1), dict(eps=-1.0), dict(lr=float("nan"))):
        with pytest.raises(gmb.GmError) as e:
            gmb.gm_adamw_step(ctx, p, grad, m, v, 1, bad.pop("lr", 1e-4), **bad)
        assert e.value.code == gmb.GM_ERR_UNSUPPORTED
    with pytest.raises(gmb.GmError) as e:
        gmb.gm_adamw_step(ctx, p, grad, m, v, 0, 1e-4)
    assert e.value.code == gmb.GM_ERR_INVALID_ARG
    if n > 1 << 20:
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        for _ in range(3):
            gmb.gm_adamw_step(ctx, p, grad, m, v, 5, 1e-4, param_bf16=pb)
        ev[0].record()
        for _ in range(10):
            gmb.gm_adamw_step(ctx, p, grad, m, v, 5, 1e-4, param_bf16=pb)
        ev[1].record()
        torch.cuda.synchronize()
        ms = ev[0].elapsed_time(ev[1]) / 10
        print(f"gm_adamw_step n {n}: {ms:.3f} ms per call, {30.0 * n / ms / 1e6:.0f} GB/s (16 bytes read, 14 written per element)")
    ctx.close()


def test_loss_kernel_edge_cases():
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny")
    ctx = gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), 4, 7, 4, 8, 8)
    rng = np.random.default_rng(2)
    n, K = 2500, 7
    al = rng.uniform(0.01, 1.0, (n, K)).astype(np.float32)
    acc = rng.integers(1, K + 2, n).astype(np.int32)
    al[0] = 1.0; acc[0] = K + 1                              # perfect head: -log K
    al[1, 0] = 0.0                                           # dead chain: +inf
    al[2, 1] = 0.0; acc[2] = 5                               # dies after the first position: -log alpha_1
    loss = torch.zeros(n, dtype=torch.float32, device="cuda")
    mean = torch.zeros(1, dtype=torch.float32, device="cuda")
    gmb.gm_dca_loss(ctx, n, K, torch.from_numpy(al).cuda(), torch.from_numpy(acc).cuda(), loss, mean)
    got = loss.cpu().numpy()
    want = np.array([oupdate.dca_loss(al[i], acc[i]) for i in range(n)])
    assert got[0] == pytest.approx(-np.log(K), rel=1e-6) and np.isinf(got[1]) and got[2] == pytest.approx(-np.log(al[2, 0]), rel=1e-5)
    fin = np.isfinite(want)
    np.testing.assert_allclose(got[fin], want[fin], rtol=3e-5, atol=3e-6)
    assert np.isinf(float(mean[0]))
    al[1, 0] = 0.5
    gmb.gm_dca_loss(ctx, n, K, torch.from_numpy(al).cuda(), torch.from_numpy(acc).cuda(), loss, mean)
    want = np.array([oupdate.dca_loss(al[i], acc[i]) for i in range(n)])
    assert float(mean[0]) == pytest.approx(want.mean(), rel=1e-5)
    ctx.close()


def test_device_pipeline_reconstruction_reproduces_the_rollouts_draft_logits():
    """Prefill -> cycles with records and hidden capture -> head-cache rebuild in a fresh state -> reconstruction:
    the replayed chains give back the draft logits the rollout itself computed (the property Eq. 4 is built for),
    through the device path alone, with ragged prompts and rejected chains."""
    import paper_2609_16648_b200 as gmb
    cfg = get_config("tiny")
    B, K, V, d = cfg.batch, cfg.k, cfg.vocab, cfg.d_model
    w = perturb_norm_weights(make_weights(cfg, 0))
    lengths = [9, 14, 20, 11]
    n_steps = 6
    n = n_steps * B
    cap = max(lengths) + n_steps * (K + 1) + 8
    pt, npg = make_page_tables(np.full(B, cap), cfg.page_size, seed=7)
    hpt, hnpg = make_page_tables(np.full(B, cap), cfg.page_size, seed=8)
    ctx = gmb.Context(cfg, gmb.pack_weights(w), B, K, pt.shape[1], npg, hnpg + 2 * n)
    st = gmb.State(ctx, B, pt, hpt)
    rng = np.random.default_rng(5)
    S = cap + 4
    seq_tok = np.zeros((B, S), np.int32)
    for b, L in enumerate(lengths):
        seq_tok[b, :L] = rng.integers(0, V, L)
    capture = torch.zeros((B, S, d), dtype=torch.bfloat16, device="cuda")
    gmb.gm_capture_hidden(ctx, capture)
    first = torch.zeros(B, dtype=torch.int32, device="cuda")
    gmb.gm_prefill(ctx, st, torch.from_numpy(seq_tok).cuda(), torch.tensor(lengths, dtype=torch.int32, device="cuda"),
                   max(lengths), T, None, 3, first)
    cur = list(lengths)
    for b in range(B):
        seq_tok[b, cur[b]] = int(first[b]); cur[b] += 1
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device="cuda")
    big = gmb.Record(n, K, d)
    saved_logits, accepted_all = [], []
    for it in range(n_steps):
        rec = gmb.Record(B, K, d)
        dtok, dl = z((B, K), torch.int32), z((B, K, V), torch.bfloat16)
        tl, th = z((B, K + 1, V), torch.bfloat16), z((B, K + 1, d), torch.bfloat16)
        a, t = z((B,), torch.int32), z((B,), torch.int32)
        gmb.gm_record_begin(ctx, st, rec)
        gmb.gm_draft(ctx, st, K, T, None, 3, 1 + it, dtok, dl)
        gmb.gm_verify(ctx, st, K, dtok, tl, th)
        gmb.gm_accept(ctx, st, B, K, T, tl, dl, dtok, None, 3, 1 + it, a, t, None, None, th, commit_state=True)
        gmb.gm_record_end(ctx, B, K, T, tl, dtok, a, rec)
        saved_logits.append(dl.clone())
        an, tn, dn = a.cpu().numpy(), t.cpu().numpy(), dtok.cpu().numpy()
        accepted_all.append(an.copy())
        for b in range(B):
            new = [int(x) for x in dn[b, :an[b]]] + [int(tn[b])]
            seq_tok[b, cur[b]:cur[b] + len(new)] = new
            cur[b] += len(new)
        for name in ("start_hidden", "start_pos", "drafts", "top_logprob", "top_index", "accepted"):
            getattr(big, name)[it * B:(it + 1) * B].copy_(getattr(rec, name))
    assert gmb.gm_last_status(ctx) == 0
    gmb.gm_capture_hidden(ctx, None)
    acc = np.concatenate(accepted_all)
    assert (acc < K).any()                                                   # some chains were cut short
    np.testing.assert_array_equal(st.kv_len.cpu().numpy() + 1, cur)
    # the captured hidden of the position before each cycle's start is that cycle's recorded start hidden
    sp = big.start_pos.cpu().numpy()
    for i in range(n):
        assert torch.equal(capture[i % B, sp[i] - 2], big.start_hidden[i])

    st2 = gmb.State(ctx, B, pt, hpt)                                          # a fresh state: only recorded inputs
    tok_d = torch.from_numpy(seq_tok).cuda()
    gmb.gm_head_prefill(ctx, st2, capture, tok_d, torch.tensor(cur, dtype=torch.int32, device="cuda"), max(cur))
    cycle_seq = torch.arange(n, dtype=torch.int32, device="cuda") % B
    scratch = torch.arange(hnpg, hnpg + 2 * n, dtype=torch.int32, device="cuda").reshape(n, 2)
    logits = z((n, K, V), torch.bfloat16)
    gmb.gm_reconstruct(ctx, st2, n, K, cycle_seq, big, tok_d, scratch, logits)
    assert gmb.gm_last_status(ctx) == 0
    want = torch.cat(saved_logits).float().cpu().numpy()
    got = logits.float().cpu().numpy()
    err = max(rel_err(got[i], want[i]) for i in range(n))
    exact = float((got == want).mean())
    print(f"reconstructed vs rollout-time draft logits: worst rel err {err:.2e}, bit-identical entries {exact:.4f}")
    assert err < 1e-2 and exact > 0.9
    ctx.close()
