"""tcgen05 GEMM (gm_gemm) against an fp64 matmul, and against the plain mma.sync kernel."""
import numpy as np
import pytest
import torch

from synth_inputs import ModelConfig

pytestmark = pytest.mark.gpu


def _ctx(flags=0):
    import paper_2609_16648_b200 as gmb
    cfg = ModelConfig("g", 1, 64, 1, 1, 64, 64, 8, batch=4, k=1, kv_len_min=0, kv_len_max=0, length_law="uniform")
    return gmb, gmb.Context(cfg, gmb.random_packed_weights(cfg, "cuda"), 4, 1, 4, 8, 8, flags=flags)


SHAPES = [(1, 128, 64), (16, 128, 128), (4, 136, 256), (64, 2560, 2560), (100, 1000, 704), (256, 6144, 2560),
          (300, 384, 512), (256, 2560, 9728), (20, 8, 64), (513, 264, 192)]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("out_fp32", [True, False])
def test_gemm_matches_fp64_matmul(M, N, K, out_fp32):
    gmb, ctx = _ctx()
    g = torch.Generator(device="cpu").manual_seed(M * 7 + N * 3 + K)
    x = (torch.randn((M, K), generator=g)).to(torch.bfloat16)
    w = (torch.randn((N, K), generator=g) * 0.05).to(torch.bfloat16)
    ref = x.double().numpy() @ w.double().numpy().T
    out = torch.full((M, N), float("nan"), dtype=torch.float32 if out_fp32 else torch.bfloat16, device="cuda")
    gmb.gm_gemm(ctx, x.cuda(), w.cuda(), out, M, N, K, out_fp32)
    assert gmb.gm_last_status(ctx) == 0
    got = out.float().cpu().numpy().astype(np.float64)
    tol = (3e-5 if out_fp32 else 5e-3) * np.abs(ref).max() + 1e-6
    assert np.abs(got - ref).max() <= tol, np.abs(got - ref).max() / np.abs(ref).max()
    ctx.close()


def test_gemm_argument_checks():
    gmb, ctx = _ctx()
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((24, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((4, 24), dtype=torch.bfloat16, device="cuda")
    for call, code in ((lambda: gmb.gm_gemm(ctx, x, w, out, 4, 24, 48, False), gmb.GM_ERR_UNSUPPORTED),      # K % 64
                       (lambda: gmb.gm_gemm(ctx, x, w, out, 4, 20, 64, False), gmb.GM_ERR_UNSUPPORTED),      # N % 8
                       (lambda: gmb.gm_gemm_swiglu(ctx, x, w, out, 4, 24, 64), gmb.GM_ERR_UNSUPPORTED),      # N % 16
                       (lambda: gmb.gm_gemm(ctx, x, w, out, 0, 24, 64, False), gmb.GM_ERR_INVALID_ARG),
                       (lambda: gmb.gm_gemm(ctx, x, None, out, 4, 24, 64, False), gmb.GM_ERR_INVALID_ARG)):
        with pytest.raises(gmb.GmError) as e:
            call()
        assert e.value.code == code
    gmb.gm_gemm(ctx, x, w, out, 4, 24, 64, False)
    assert gmb.gm_last_status(ctx) == 0
    ctx.close()


def test_simple_kernel_agrees():
    gmb, ctx = _ctx(flags=1)
    M, N, K = 70, 200, 192
    g = torch.Generator(device="cpu").manual_seed(5)
    x = torch.randn((M, K), generator=g).to(torch.bfloat16)
    w = torch.randn((N, K), generator=g).to(torch.bfloat16)
    out = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    gmb.gm_gemm(ctx, x.cuda(), w.cuda(), out, M, N, K, True)
    ref = x.double().numpy() @ w.double().numpy().T
    assert np.abs(out.cpu().numpy() - ref).max() <= 1e-5 * np.abs(ref).max()
    ctx.close()


@pytest.mark.parametrize("M,N,K", [(256, 151936, 2560), (64, 151936, 2560), (256, 19456, 2560), (256, 6144, 2560),
                                   (256, 2560, 4096)])
def test_full_size_projections_on_sampled_outputs(M, N, K):
    """The 4B-shaped projections in the launch configuration the benchmark times (LM head at M = 256 and
    M = 64, gate/up, QKV, O): sampled output columns against fp64 dot products."""
    gmb, ctx = _ctx()
    g = torch.Generator(device="cuda").manual_seed(N + K)
    x = torch.randn((M, K), device="cuda", generator=g).to(torch.bfloat16)
    w = (torch.randn((N, K), device="cuda", generator=g) * 0.02).to(torch.bfloat16)
    out = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    gmb.gm_gemm(ctx, x, w, out, M, N, K, False)
    assert gmb.gm_last_status(ctx) == 0
    assert not torch.isnan(out.float()).any()                      # every tile was written
    cols = torch.tensor(sorted(set([0, 1, 127, 128, 255, 256, N - 1, N - 129] +
                                   np.random.default_rng(0).integers(0, N, 300).tolist())), device="cuda")
    ref = x.double().cpu().numpy() @ w[cols].double().cpu().numpy().T
    got = out[:, cols].float().cpu().numpy()
    assert np.abs(got - ref).max() <= 5e-3 * np.abs(ref).max()
    ctx.close()


@pytest.mark.parametrize("M", [256, 64, 300, 37])
@pytest.mark.parametrize("chain", ["1", "0"], ids=["pair_wave_kernel", "full_wave_plus_tail"])
def test_gate_up_projection_with_fused_swiglu_full_matrix(M, chain, monkeypatch):
    """The 4B gate/up projection over the whole output, plain stores and the fused SwiGLU epilogue on interleaved
    gate/up rows, against fp64.  The SwiGLU form runs as one exact wave of the persistent-pair kernel (74 tiles of 256 or
    288 features; two token blocks at M = 300) or, with GM_CHAIN_MODE=0, as 152 feature tiles: a full wave plus a
    split tail launch."""
    N, K = 19456, 2560
    monkeypatch.setenv("GM_CHAIN_MODE", chain)
    gmb, ctx = _ctx()
    g = torch.Generator(device="cuda").manual_seed(M)
    x = torch.randn((M, K), device="cuda", generator=g).to(torch.bfloat16)
    w = (torch.randn((N, K), device="cuda", generator=g) * 0.02).to(torch.bfloat16)
    ref = (x.double() @ w.double().T).cpu().numpy()
    act_ref = ref[:, 0::2] / (1 + np.exp(-ref[:, 0::2])) * ref[:, 1::2]
    o32 = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    act = torch.full((M, N // 2), float("nan"), dtype=torch.bfloat16, device="cuda")
    gmb.gm_gemm(ctx, x, w, o32, M, N, K, True)
    gmb.gm_gemm_swiglu(ctx, x, w, act, M, N, K)
    assert gmb.gm_last_status(ctx) == 0
    assert np.abs(o32.cpu().numpy() - ref).max() <= 3e-5 * np.abs(ref).max()
    assert np.abs(act.float().cpu().numpy() - act_ref).max() <= 6e-3 * np.abs(act_ref).max()
    ctx.close()


@pytest.mark.parametrize("M", [256, 64, 96])
def test_cta_pair_kernel_equals_single_cta_kernel(M, monkeypatch):
    """The full wave of a wide projection runs on CTA pairs (one MMA over two SMs, each CTA staging half of the
    activation box).  Same K order and the same accumulation per output as the single-CTA kernel: bit-identical."""
    N, K = 19456, 2560
    monkeypatch.setenv("GM_CHAIN_MODE", "0")                  # both runs on the tile kernels this test compares
    g = torch.Generator(device="cuda").manual_seed(100 + M)
    x = torch.randn((M, K), device="cuda", generator=g).to(torch.bfloat16)
    w = (torch.randn((N, K), device="cuda", generator=g) * 0.02).to(torch.bfloat16)
    outs = []
    for pair in (True, False):
        if not pair:
            monkeypatch.setenv("GM_NO_PAIR_GEMM", "1")
        gmb, ctx = _ctx()
        o32 = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        act = torch.full((M, N // 2), float("nan"), dtype=torch.bfloat16, device="cuda")
        for rep in range(2):
            gmb.gm_gemm(ctx, x, w, o32, M, N, K, True)
            gmb.gm_gemm_swiglu(ctx, x, w, act, M, N, K)
        assert gmb.gm_last_status(ctx) == 0
        outs.append((o32.clone(), act.clone()))
        ctx.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    ref = (x.double() @ w.double().T).cpu().numpy()
    assert np.abs(outs[0][0].cpu().numpy() - ref).max() <= 3e-5 * np.abs(ref).max()
