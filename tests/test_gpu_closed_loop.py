"""The training loop of Alg. 1 closed on the device: rollout with speculative cycles -> per-cycle records and captured
hidden states -> updates of the draft head on those records -> the next rollout runs with the updated head."""
import numpy as np
import pytest
import torch

from oracle import update as oupdate
from synth_inputs import get_config, make_page_tables, make_weights
from synth_inputs.weights import perturb_norm_weights

pytestmark = pytest.mark.gpu

T = 0.2          # sharpens the nearly flat random-init distributions so that there is something to learn


def test_rollout_record_update_laps_raise_the_acceptance():
    """Four laps of (rollout of 12 cycles on 16 sequences with records, 20 updates on those 192 cycles).  The head starts
    at random initialisation, independent of the target, so few drafts are accepted; every lap's updates lower the
    objective (mean of Eq. 9) on its own records, and the accepted drafts per cycle of the NEXT rollout - same prompts, new
    random draws, the updated head - rise well above the first lap's.  On other prompts the gain is small (a
    192-cycle training set on a toy model; measured 0.30 -> 0.38 / 0.45 / 0.43 on the default kernels) and within the
    sampling noise of 192 cycles under other kernel choices, so it is printed and only loosely bounded.  Everything goes through the C ABI: prefill,
    draft / verify / accept with gm_record_begin / gm_record_end and gm_capture_hidden, then gm_head_update_step."""
    import paper_2609_16648_b200 as gmb
    B, n_steps, K, epochs, peak = 16, 12, 3, 20, 1e-3
    cfg = get_config("tiny").with_(batch=B)
    V, d = cfg.vocab, cfg.d_model
    w = perturb_norm_weights(make_weights(cfg, 0))
    n = n_steps * B
    lengths = [8 + (3 * b) % 9 for b in range(B)]
    cap = max(lengths) + n_steps * (K + 1) + 8
    pt, npg = make_page_tables(np.full(B, cap), cfg.page_size, seed=7)
    hpt, hnpg = make_page_tables(np.full(B, cap), cfg.page_size, seed=8)
    ctx = gmb.Context(cfg, gmb.pack_weights(w), B, K, pt.shape[1], npg, hnpg + 2 * n)
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device="cuda")

    def rollout(seed, prompt_seed):
        st = gmb.State(ctx, B, pt, hpt)
        rng = np.random.default_rng(prompt_seed)
        S = cap + 4
        seq_tok = np.zeros((B, S), np.int32)
        for b, L in enumerate(lengths):
            seq_tok[b, :L] = rng.integers(0, V, L)
        capture = z((B, S, d), torch.bfloat16)
        gmb.gm_capture_hidden(ctx, capture)
        first = z((B,), torch.int32)
        gmb.gm_prefill(ctx, st, torch.from_numpy(seq_tok).cuda(), torch.tensor(lengths, dtype=torch.int32, device="cuda"),
                       max(lengths), T, None, seed, first)
        cur = list(lengths)
        for b in range(B):
            seq_tok[b, cur[b]] = int(first[b]); cur[b] += 1
        big = gmb.Record(n, K, d)
        acc = []
        for it in range(n_steps):
            rec = gmb.Record(B, K, d)
            dtok, dl = z((B, K), torch.int32), z((B, K, V), torch.bfloat16)
            tl, th = z((B, K + 1, V), torch.bfloat16), z((B, K + 1, d), torch.bfloat16)
            a, t = z((B,), torch.int32), z((B,), torch.int32)
            gmb.gm_record_begin(ctx, st, rec)
            gmb.gm_draft(ctx, st, K, T, None, seed, 1 + it, dtok, dl)
            gmb.gm_verify(ctx, st, K, dtok, tl, th)
            gmb.gm_accept(ctx, st, B, K, T, tl, dl, dtok, None, seed, 1 + it, a, t, None, None, th, commit_state=True)
            gmb.gm_record_end(ctx, B, K, T, tl, dtok, a, rec)
            an, tn, dn = a.cpu().numpy(), t.cpu().numpy(), dtok.cpu().numpy()
            acc.append(an.copy())
            for b in range(B):
                new = [int(x) for x in dn[b, :an[b]]] + [int(tn[b])]
                seq_tok[b, cur[b]:cur[b] + len(new)] = new
                cur[b] += len(new)
            for name in ("start_hidden", "start_pos", "drafts", "top_logprob", "top_index", "accepted"):
                getattr(big, name)[it * B:(it + 1) * B].copy_(getattr(rec, name))
        gmb.gm_capture_hidden(ctx, None)
        assert gmb.gm_last_status(ctx) == 0
        return big, seq_tok, cur, capture, float(np.mean(np.concatenate(acc)))

    step, trained, other = 0, [], []
    for lap in range(4):
        big, seq_tok, cur, capture, tau = rollout(3 + lap, 5)
        _, _, _, _, tau_other = rollout(100 + lap, 77)                       # other prompts, other draws
        trained.append(tau)
        other.append(tau_other)
        st2 = gmb.State(ctx, B, pt, hpt)
        tok_d = torch.from_numpy(seq_tok).cuda()
        len_d = torch.tensor(cur, dtype=torch.int32, device="cuda")
        cycle_seq = torch.arange(n, dtype=torch.int32, device="cuda") % B
        scratch = torch.arange(hnpg, hnpg + 2 * n, dtype=torch.int32, device="cuda").reshape(n, 2)
        mean = z((1,), torch.float32)
        losses = []
        for _ in range(epochs):
            step += 1
            lr = float(np.float32(oupdate.head_lr(step - 1, peak, 4 * epochs, warmup=5)))
            gmb.gm_head_update_step(ctx, st2, n, K, T, cycle_seq, big, tok_d, scratch, capture, len_d, max(cur), step, lr, mean)
            losses.append(float(mean[0]))
        assert gmb.gm_last_status(ctx) == 0
        assert all(np.isfinite(losses)) and losses[-1] < losses[0] - 0.02, losses
        print(f"lap {lap}: accepted drafts per cycle {tau:.3f} (training prompts) {tau_other:.3f} (other prompts); "
              f"objective over the lap's updates {losses[0]:.3f} -> {losses[-1]:.3f}")
    assert trained[-1] > trained[0] + 0.2 and min(trained[1:]) > trained[0] + 0.1       # measured 0.35 -> 0.70 / 0.80 / 0.87
    assert np.mean(other[1:]) >= other[0] - 0.1          # 192 cycles: a standard error of about 0.05 per figure
    ctx.close()
