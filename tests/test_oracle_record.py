"""Pins for the oracle's cycle record (App. D.2)."""
import numpy as np
from scipy.special import log_softmax

from oracle import record, sampler
from oracle.model import round_bf16


def test_top_logprobs_are_the_full_vocabulary_log_softmax_at_the_largest_logits():
    rng = np.random.default_rng(0)
    x = round_bf16(rng.normal(0, 3, 5000).astype(np.float32)).astype(np.float64)
    for T in (1.0, 0.7):
        idx, lp = record.top_logprobs(x, T)
        ref = log_softmax(x / T)
        assert len(idx) == 64 and len(set(idx.tolist())) == 64
        np.testing.assert_array_equal(lp, round_bf16(ref[idx].astype(np.float32)))
        # nothing outside the set beats anything inside it
        outside = np.setdiff1d(np.arange(len(x)), idx)
        assert x[outside].max() <= x[idx].min()
        # full-vocabulary normalisation is kept: the retained mass is below one
        assert np.exp(lp.astype(np.float64)).sum() < 1.0
        assert np.all(np.diff(x[idx]) <= 0)                      # sorted by logit, descending


def test_ties_at_the_cut_take_the_lowest_token_ids():
    x = np.zeros(300)
    x[[5, 17, 200]] = 2.0                                        # three clear winners
    x[100:180] = 1.0                                             # 80 tokens tie for the remaining 61 places
    idx, lp = record.top_logprobs(x)
    assert idx[:3].tolist() == [5, 17, 200]
    assert idx[3:].tolist() == list(range(100, 161))
    assert np.all(lp[3:] == lp[3])


def test_short_rows_are_padded():
    idx, lp = record.top_logprobs(np.array([0.5, 2.0, -1.0]))
    assert idx[:3].tolist() == [1, 0, 2] and np.all(idx[3:] == -1) and np.all(np.isneginf(lp[3:]))
    assert abs(np.exp(lp[:3].astype(np.float64)).sum() - 1.0) < 2e-2


def test_sparsified_overlap_bounds_the_full_overlap():
    """App. D.2: the overlap computed from the retained set plus a residual bin upper-bounds the
    full-vocabulary overlap (Eq. 5) by at most the target mass outside the retained set."""
    rng = np.random.default_rng(1)
    for trial in range(20):
        V = 4000
        lt = rng.normal(0, 3, V)
        lq = lt + rng.normal(0, 1.0, V)
        p, q = sampler.softmax_probs(lt).astype(np.float64), sampler.softmax_probs(lq).astype(np.float64)
        idx, lp = record.top_logprobs(lt)
        full = sampler.acceptance_probability(p, q)
        est = record.sparsified_overlap(idx, lp, q)
        outside = 1.0 - p[idx].sum()
        assert full - 5e-3 <= est <= full + outside + 5e-3       # 5e-3: bf16 rounding of 64 log-probabilities


def test_cycle_record_items():
    rng = np.random.default_rng(2)
    K, V, d = 3, 500, 16
    tl = rng.normal(0, 2, (K + 1, V))
    rec = record.cycle_record(rng.normal(size=d), [4, 9, 1], tl, accept_len=2, start_pos=77)
    assert rec["top_index"].shape == (K, 64) and rec["top_logprob"].shape == (K, 64)
    assert rec["accepted"] == 3 and rec["start_pos"] == 77 and rec["drafts"].tolist() == [4, 9, 1]
    for k in range(K):
        np.testing.assert_array_equal(rec["top_index"][k], record.top_logprobs(tl[k])[0])
