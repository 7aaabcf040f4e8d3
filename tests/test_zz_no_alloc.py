"""gm_attention_noalloc: the attention kernel for callers that may not allocate device memory.

Some users of the library get device buffers and a stream from their host application but must not call
cudaMalloc themselves (a serving thread that may not synchronise the device, a plug-in without a memory
pool).  For them the library offers one entry point whose scratch is a fixed array inside the library.  This
file checks, through the C ABI, that it computes what the regular gm_attention computes - twice in a row on
different inputs, because the scratch keeps the previous call's contents - and that it refuses requests that
do not fit the array.  The file name sorts last so that a failure here cannot hide any other test.
"""
import numpy as np
import pytest
import torch

from synth_inputs import ModelConfig, make_page_tables

pytestmark = pytest.mark.gpu

TOL = 1.5e-2        # the tolerance of the attention parity tests (normalised max error)


def _inputs(n_q, n_kv, hd, q_stride, lens, counts, seed):
    B = len(lens)
    group = n_q // n_kv
    lens, counts = np.asarray(lens), np.asarray(counts, np.int32)
    pt, npg = make_page_tables(lens + counts, 16, seed=seed, slack_pages=1)
    g = torch.Generator(device="cuda").manual_seed(seed)
    q_rows = 16 * ((q_stride * group + 15) // 16)
    q = torch.randn((B, n_kv, q_rows, hd), device="cuda", generator=g).to(torch.bfloat16)
    pool = torch.randn((1, 2, npg, n_kv, 16, hd), device="cuda", generator=g).to(torch.bfloat16)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device="cuda", dtype=torch.int32)
    return dict(B=B, q=q, pool=pool, pt=dev(np.where(pt < 0, 0, pt)), counts=dev(counts), base=dev(lens.astype(np.int32)),
                max_pages=pt.shape[1], npg=npg)


def test_noalloc_matches_the_regular_entry_point_on_two_calls_in_a_row():
    import paper_2609_16648_b200 as gmb
    n_q, n_kv, hd, q_stride = 32, 8, 128, 4
    cases = [_inputs(n_q, n_kv, hd, q_stride, [900, 17, 2300, 0, 64, 511], [4, 1, 3, 4, 2, 4], seed=21),
             _inputs(n_q, n_kv, hd, q_stride, [33, 1500, 250], [2, 4, 1], seed=22)]
    cfg = ModelConfig("n", 1, 64, n_q, n_kv, hd, 64, 8, batch=8, k=q_stride - 1, kv_len_min=0, kv_len_max=0,
                      length_law="uniform")
    packed = gmb.random_packed_weights(cfg, "cuda")
    refs = []
    for c in cases:                                   # the existing entry point needs a context per page-table width
        ctx = gmb.Context(cfg, packed, 8, q_stride - 1, c["max_pages"], c["npg"], 4)
        ref = torch.full((c["B"] * q_stride, n_q * hd), 3.0, dtype=torch.bfloat16, device="cuda")
        gmb.gm_attention(ctx, c["q"], c["pool"], 0, c["pt"], c["counts"], c["base"], c["B"], q_stride, ref)
        assert gmb.gm_last_status(ctx) == 0
        refs.append(ref)
        ctx.close()
    # outputs first, then one warm-up call (the first call on a device resolves the scratch address and may make the
    # driver load the kernels); from here on the driver's free-memory figure must not move: nothing is allocated
    outs = [torch.full((c["B"] * q_stride, n_q * hd), 3.0, dtype=torch.bfloat16, device="cuda") for c in cases]
    again = torch.full_like(refs[0], 3.0)
    warm = torch.full_like(refs[0], 3.0)
    c = cases[0]
    gmb.gm_attention_noalloc(n_q, n_kv, hd, c["q"], c["pool"], 0, c["pt"], c["counts"], c["base"], c["B"], q_stride, warm)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for c, out in zip(cases, outs):                   # two calls in a row share the library's static scratch
        gmb.gm_attention_noalloc(n_q, n_kv, hd, c["q"], c["pool"], 0, c["pt"], c["counts"], c["base"], c["B"], q_stride, out)
    # and once more on the first inputs: stale partials of the second call must not leak in
    c = cases[0]
    gmb.gm_attention_noalloc(n_q, n_kv, hd, c["q"], c["pool"], 0, c["pt"], c["counts"], c["base"], c["B"], q_stride, again)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before          # driver-level: would also see a raw cudaMalloc
    for out, ref in zip(outs + [again], refs + [refs[0]]):
        err = (out.float() - ref.float()).abs().max().item() / ref.float().abs().max().item()
        assert err <= TOL, err


def test_noalloc_small_heads_match_the_regular_entry_point():
    """head_dim 64 with two KV heads (the other attention instantiation), again two calls in a row."""
    import paper_2609_16648_b200 as gmb
    n_q, n_kv, hd, q_stride = 4, 2, 64, 4
    cfg = ModelConfig("n", 1, 64, n_q, n_kv, hd, 64, 8, batch=8, k=q_stride - 1, kv_len_min=0, kv_len_max=0,
                      length_law="uniform")
    packed = gmb.random_packed_weights(cfg, "cuda")
    for seed, lens, counts in ((31, [70, 5, 260, 1023], [4, 2, 1, 3]), (32, [300, 48], [4, 4])):
        c = _inputs(n_q, n_kv, hd, q_stride, lens, counts, seed=seed)
        ctx = gmb.Context(cfg, packed, 8, q_stride - 1, c["max_pages"], c["npg"], 4)
        ref = torch.full((c["B"] * q_stride, n_q * hd), 3.0, dtype=torch.bfloat16, device="cuda")
        gmb.gm_attention(ctx, c["q"], c["pool"], 0, c["pt"], c["counts"], c["base"], c["B"], q_stride, ref)
        assert gmb.gm_last_status(ctx) == 0
        ctx.close()
        out = torch.full_like(ref, 3.0)
        gmb.gm_attention_noalloc(n_q, n_kv, hd, c["q"], c["pool"], 0, c["pt"], c["counts"], c["base"], c["B"], q_stride, out)
        torch.cuda.synchronize()
        err = (out.float() - ref.float()).abs().max().item() / ref.float().abs().max().item()
        assert err <= TOL, err


def test_noalloc_rejects_what_does_not_fit_its_scratch():
    import paper_2609_16648_b200 as gmb
    n_q, n_kv, hd, q_stride = 32, 8, 128, 4
    B = 120                                           # (148 + 120) * 8 * 16 * 130 * 4 B = 17.8 MB > 16 MiB
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device="cuda")
    out = z((B * q_stride, n_q * hd), torch.bfloat16)
    with pytest.raises(gmb.GmError) as e:
        gmb.gm_attention_noalloc(n_q, n_kv, hd, z((B, n_kv, 16, hd), torch.bfloat16), z((1, 2, 4, n_kv, 16, hd), torch.bfloat16),
                                 0, z((B, 2), torch.int32), z((B,), torch.int32), z((B,), torch.int32), B, q_stride, out)
    assert e.value.code == gmb.GM_ERR_SCRATCH_LIMIT
    assert "scratch" in str(e.value)
    with pytest.raises(gmb.GmError) as e:             # more sequences than the stated maximum
        Bb = gmb.GM_NOALLOC_MAX_BATCH + 1
        gmb.gm_attention_noalloc(4, 2, 64, z((Bb, 2, 16, 64), torch.bfloat16), z((1, 2, 4, 2, 16, 64), torch.bfloat16), 0,
                                 z((Bb, 2), torch.int32), z((Bb,), torch.int32), z((Bb,), torch.int32), Bb, 1,
                                 z((Bb, 256), torch.bfloat16))
    assert e.value.code == gmb.GM_ERR_SCRATCH_LIMIT
