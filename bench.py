#!/usr/bin/env python
"""Benchmark of one speculative-decoding rollout step (draft k tokens, verify k+1 positions, accept).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 4b] [--impl reference]

Prints ONE JSON line.  A "step" is one whole cycle (gm_spec_step: all draft applications, the target
verify forward over the paged KV cache, rejection sampling and the state commit) over one batch of
seeded synthetic sequences; consecutive steps feed on each other's committed state.  `value` is the
whole-job committed tokens per second with all inputs resident in HBM; `e2e` is the same metric
through the host-buffer entry point (uniforms copied from pinned host memory, results copied back,
every step).  With N > 1 every rank runs an independent replica (no collective on the data path).
Other workloads, each with its own line: `--workload sampler` (accept / resample alone), `--workload rollout` (prefill +
cycles with the library's page allocator), `--workload head_update` (one update of the draft head on recorded cycles).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM bytes per algorithmic byte of the attention kernel, from the ncu capture summarised in
# profiles/attention_kernel_4b-shape_small.md (traffic grows in proportion to the positions attended).
ATTENTION_TRAFFIC_RATIO = 1.022
METRIC = "committed_tokens_per_s"
UNIT = "tokens/s"
SMI_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def measured_peaks():
    """(HBM copy GB/s, bf16 TFLOP/s burst, bf16 TFLOP/s sustained, source).  The burst figure is the denominator for
    a kernel class timed launch by launch; the sustained one (under the power cap) for work timed inside a long step."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            p = json.load(open(path))
            burst = float(p["bf16_tflops"])
            return float(p["hbm_gbs"]), burst, float(p.get("bf16_tflops_sustained", burst)), "measured"
        except Exception:
            pass
    return 6650.0, 1590.0, 1400.0, "fallback"


NOMINAL_HBM_GBS = 8000.0        # the figure the benchmark spec states its 70 % bar on


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs (read-only)."""

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={SMI_QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
                for n, v in zip(names, r[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---- workload -------------------------------------------------------------------------------------------------------

def lengths_for(cfg, seed):
    from synth_inputs import kv_lengths_lognormal, kv_lengths_uniform
    if cfg.length_law == "lognormal":
        return kv_lengths_lognormal(cfg.batch, 4096, 0.7, cfg.kv_len_min, cfg.kv_len_max, seed)
    return kv_lengths_uniform(cfg.batch, cfg.kv_len_min, cfg.kv_len_max, seed)


def build_workload(name: str, rank: int, total_steps: int, k: int, device, layers: int = 0, batch: int = 0,
                   top_p: float = 1.0):
    """Random-init model of the named shape + a batch of sequences with ragged, fragmented KV caches.
    `layers` / `batch` > 0 shrink the model depth / the batch (profiling captures on a few GB)."""
    import torch
    import paper_2609_16648_b200 as gmb
    from synth_inputs import get_config, make_page_tables
    cfg = get_config(name)
    cfg = cfg.with_(k=k)
    if layers > 0:
        cfg = cfg.with_(n_layers=layers)
    if batch > 0:
        cfg = cfg.with_(batch=batch)
    lens = lengths_for(cfg, seed=3 + rank).astype(np.int64)
    free_b, _ = torch.cuda.mem_get_info()
    w_bytes = 2 * (cfg.target_params() + cfg.layer_params() + 2 * cfg.d_model ** 2 + cfg.vocab * cfg.d_model)
    logits_bytes = 2 * cfg.batch * (2 * k + 1) * cfg.vocab
    budget = free_b - w_bytes - logits_bytes - (8 << 30)
    grow = total_steps * (k + 1) + 2 * (k + 1)
    per_tok = cfg.kv_bytes_per_token() + cfg.kv_bytes_per_token(1)
    # keep the first B' sequences whose caches fit (the 7B and long-tail batches exceed one GPU as written)
    keep, used = 0, 0
    for b in range(cfg.batch):
        need = ((lens[b] + grow + 15) // 16) * 16 * per_tok
        if used + need > budget:
            break
        used += need
        keep += 1
    if keep == 0:
        raise RuntimeError("no sequence fits in device memory")
    lens = lens[:keep]
    cfg = cfg.with_(batch=keep)
    cap = lens + grow
    pt, npg = make_page_tables(cap, 16, seed=7 + rank)
    hpt, hnpg = make_page_tables(cap, 16, seed=8 + rank)
    packed = gmb.random_packed_weights(cfg, device, seed=rank)
    # GM_FLAG_GRAPH: on a stream of its own the library replays one captured CUDA graph per cycle (whenever no
    # per-launch timing is requested); on the default stream the flag has no effect
    ctx = gmb.Context(cfg, packed, keep, k, pt.shape[1], npg, hnpg, flags=gmb.GM_FLAG_GRAPH)
    if top_p < 1.0:
        gmb.gm_set_top_p(ctx, top_p)
    st = gmb.State(ctx, keep, np.where(pt < 0, 0, pt), np.where(hpt < 0, 0, hpt), device)
    gen = torch.Generator(device=device)
    gen.manual_seed(100 + rank)

    def fill(t):                                    # N(0,1) keys/values, in slabs
        flat = t.view(-1)
        step = 1 << 28
        for i in range(0, flat.numel(), step):
            n = min(step, flat.numel() - i)
            flat[i:i + n] = torch.randn(n, device=device, generator=gen, dtype=torch.float32).to(torch.bfloat16)

    fill(st.kv_pool)
    fill(st.head_kv_pool)
    st.kv_len.copy_(torch.from_numpy(lens.astype(np.int32)))
    st.pending_n.fill_(1)
    st.pending_tok.copy_(torch.randint(0, cfg.vocab, st.pending_tok.shape, device=device, generator=gen, dtype=torch.int32))
    st.pending_hidden.copy_(torch.randn(st.pending_hidden.shape, device=device, generator=gen).to(torch.bfloat16))
    torch.cuda.synchronize()
    return cfg, ctx, st, lens


def algorithmic_bytes_per_step(cfg, k, sum_len):
    """What one cycle must move at least once: weights, KV, logits (bytes)."""
    d, V = cfg.d_model, cfg.vocab
    verify_w = 2 * cfg.target_params()
    draft_w = k * 2 * (cfg.layer_params() + 2 * d * d + V * d)
    kv = sum_len * cfg.kv_bytes_per_token() + k * sum_len * cfg.kv_bytes_per_token(1)
    logits = 2 * 2 * cfg.batch * (2 * k + 1) * V
    return verify_w + draft_w + kv + logits


# ---- CPU oracle leg -----------------------------------------------------------------------------------------------------

class OracleSample:
    """Times the oracle, as it stands, on a bounded sample of the workload: ONE sequence of the named
    shape at a typical KV length through the draft head (k applications), ONE of the target's decoder
    layers, the LM head and the sampler; the layer time is multiplied by the layer count
    (extrapolated).  The weights are generated once and handed over as float64 arrays, so that the
    oracle's up-casts are no-ops and the time is spent on its arithmetic."""

    def __init__(self, name: str, k: int, kv_len: int = 4608):
        from oracle import model as omodel
        from synth_inputs import get_config, make_page_tables, make_weights
        t0 = time.time()
        self.name, self.k, self.kv_len = name, k, kv_len
        self.n_layers = get_config(name).n_layers
        self.cfg = cfg = get_config(name).with_(k=k, batch=1)
        if name == "tiny":
            self.kv_len = kv_len = 200
        w = make_weights(cfg, 0, n_layers=1)

        def up(o):
            if isinstance(o, dict):
                return {k_: up(v) for k_, v in o.items()}
            if isinstance(o, list):
                return [up(v) for v in o]
            return np.asarray(o, dtype=np.float64)
        self.w = up(w)
        rng = np.random.default_rng(0)
        pt, npg = make_page_tables(np.array([kv_len + 2 * (k + 1)]), 16, seed=1)
        self.kv = omodel.PagedKV(1, cfg.n_kv_heads, cfg.head_dim, pt, npg)
        self.hkv = omodel.PagedKV(1, cfg.n_kv_heads, cfg.head_dim, pt, npg)
        self.kv.pool[:] = rng.standard_normal(self.kv.pool.shape)
        self.hkv.pool[:] = rng.standard_normal(self.hkv.pool.shape)
        self.setup_s = time.time() - t0

    def run(self, seed: int = 0):
        from oracle import model as omodel, philox, sampler as osampler
        cfg, w, k, kv_len = self.cfg, self.w, self.k, self.kv_len
        rng = np.random.default_rng(seed)
        hidden = rng.standard_normal((1, cfg.d_model))
        tok = [int(rng.integers(cfg.vocab))]
        t1 = time.time()
        g = omodel.head_forward(w, hidden, tok, np.array([kv_len - 1]), self.hkv, 0, cfg)
        d, q = [], []
        for j in range(k):
            if j > 0:
                g = omodel.head_forward(w, g, [d[-1]], np.array([kv_len - 1 + j]), self.hkv, 0, cfg)
            qj = osampler.softmax_probs(omodel.round_bf16(omodel.head_logits(w, g, cfg)[0]))
            d.append(osampler.draw_token(qj, philox.u24(seed, 1, 0, j))[0])
            q.append(qj)
        t_draft = time.time() - t1
        t3 = time.time()
        x = w["embed"][tok + d]
        H = omodel.decoder_layer(w["layers"][0], x, np.arange(kv_len, kv_len + k + 1), self.kv, 0, 0, cfg)
        t_layer = time.time() - t3
        t4 = time.time()
        p = osampler.softmax_probs(omodel.round_bf16(omodel.target_logits(w, H, cfg)))
        a, _, _ = osampler.decide(p, np.array(q), d, philox.u24_accept(seed, 1, 1, k)[0])
        t_tail = time.time() - t4
        step_s = t_draft + self.n_layers * t_layer + t_tail
        return {"step_s": step_s, "committed": int(a + 1), "t_draft": t_draft, "t_layer": t_layer, "t_tail": t_tail,
                "cpu_s": time.time() - t1}

    def describe(self, runs, cpu_s):
        import torch
        return (f"{runs} x [1 sequence of the {self.name} shape at kv_len {self.kv_len}, k={self.k}: draft head x{self.k}, "
                f"1 of {self.n_layers} target layers (its time extrapolated x{self.n_layers}), LM head + sampler]; "
                f"{cpu_s:.1f} s of CPU work; sequences run one after another on the CPU, so tokens/s does not depend on "
                f"the batch; float64 weights prepared once ({self.setup_s:.0f} s, excluded); "
                f"BLAS threads {torch.get_num_threads()}")


def host_cores():
    return len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)


def cpu_baseline(name: str, k: int, budget_s: float = 15.0, max_runs: int = 40):
    smp = OracleSample(name, k)
    runs, t0 = [], time.time()
    while len(runs) < max_runs and (not runs or time.time() - t0 < budget_s):
        runs.append(smp.run(seed=len(runs)))
    value = sum(r["committed"] for r in runs) / sum(r["step_s"] for r in runs)
    return {"value": value, "unit": UNIT, "cores": host_cores(), "kind": "oracle",
            "sample": smp.describe(len(runs), sum(r["cpu_s"] for r in runs))}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    smp = OracleSample(args.workload, args.k)
    runs = []
    for i in range(args.warmup + args.steps):
        r = smp.run(seed=i)
        if i >= args.warmup:
            runs.append(r)
    value = sum(r["committed"] for r in runs) / sum(r["step_s"] for r in runs)
    secs = float(np.mean([r["step_s"] for r in runs]))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "k": args.k,
                       "note": "CPU oracle; every step is a bounded sample (one sequence, one layer extrapolated)"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_cores(), "kind": "oracle",
                             "sample": smp.describe(len(runs), sum(r["cpu_s"] for r in runs))},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ---- product leg ---------------------------------------------------------------------------------------------------------

def reduce_over_ranks(maxima, sums, device, world):
    """Replicas share nothing on the data path; only the report is reduced: times as the max over ranks,
    token and launch counts as sums.  Works on any backend (NCCL on GPUs, gloo in the CPU tests)."""
    import torch
    mx = torch.tensor(list(maxima), dtype=torch.float64, device=device)
    sm = torch.tensor(list(sums), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(mx, op=dist.ReduceOp.MAX)
        dist.all_reduce(sm, op=dist.ReduceOp.SUM)
    return mx.tolist(), sm.tolist()


def run_product(args):
    import torch
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_2609_16648_b200.build import build
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    import paper_2609_16648_b200 as gmb
    # a stream of this rank's own (the default stream cannot be captured into a CUDA graph); everything below -
    # the library's context, the torch ops and the timing events - runs on it
    torch.cuda.set_stream(torch.cuda.Stream(device))

    K, W, S = args.k, args.warmup, args.steps
    total_steps = W + 2 * S + 12
    cfg, ctx, st, lens = build_workload(args.workload, rank, total_steps, K, device, args.layers, args.batch, args.top_p)
    B = cfg.batch
    a_dev = torch.zeros(B, dtype=torch.int32, device=device)
    t_dev = torch.zeros(B, dtype=torch.int32, device=device)
    acc_sum = torch.zeros(1, dtype=torch.int64, device=device)
    seed = 1234 + rank
    step_id = 0

    rec = gmb.Record(B, K, cfg.d_model, device) if args.record else None
    d_dev = torch.zeros((B, K), dtype=torch.int32, device=device)

    def one_step():
        nonlocal step_id
        if rec is not None:
            gmb.gm_spec_step_rec(ctx, st, K, 1.0, seed, step_id, a_dev, t_dev, d_dev, rec)
        else:
            gmb.gm_spec_step(ctx, st, K, 1.0, seed, step_id, a_dev, t_dev)
        acc_sum.add_(a_dev.sum())
        step_id += 1

    for _ in range(W):
        one_step()
    torch.cuda.synchronize()
    if gmb.gm_last_status(ctx) != 0:
        raise RuntimeError("device status set during warm-up")
    acc_sum.zero_()
    len0 = int(st.kv_len.sum().item())

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    clocks = ClockSampler(local)
    gmb.gm_profile(ctx, (1 << gmb.GM_KC_ATTENTION) | (1 << gmb.GM_KC_RECORD))
    launches0 = gmb.gm_launch_count(ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    clocks.start()
    e0.record()
    for _ in range(S):
        one_step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    clk = clocks.stop()
    launches = gmb.gm_launch_count(ctx) - launches0
    att_ms, att_n = gmb.gm_profile_read(ctx, gmb.GM_KC_ATTENTION)
    rec_ms, rec_n = gmb.gm_profile_read(ctx, gmb.GM_KC_RECORD)
    gmb.gm_profile(ctx, 0)
    accepted = int(acc_sum.item())
    committed = accepted + S * B
    len1 = int(st.kv_len.sum().item())
    status = gmb.gm_last_status(ctx)
    if status != 0:
        raise RuntimeError(f"device status {status} ({gmb.gm_strerror(status)}) during the timed region")

    # ---- optional: device time per kernel class, from a separate pass with every launch bracketed by events ---------
    breakdown = None
    if args.breakdown:
        gmb.gm_profile(ctx, 0xF)
        nb = min(S, 5)
        for _ in range(nb):
            one_step()
        names = {gmb.GM_KC_GEMM: "gemm", gmb.GM_KC_ATTENTION: "attention", gmb.GM_KC_ELEMENTWISE: "elementwise",
                 gmb.GM_KC_SAMPLER: "sampler"}
        breakdown = {}
        for cls, nm in names.items():
            t_ms, n = gmb.gm_profile_read(ctx, cls)
            breakdown[nm] = {"ms_per_step": t_ms / nb, "launches_per_step": n / nb}
        gmb.gm_profile(ctx, 0)

    # ---- the other kernel classes the bars are stated on: a short separate pass through the three sub-calls, every
    # GEMM / sampler launch bracketed by events (so the timed region above stays clean) ---------------------------------
    np_steps = 3
    dl_buf = torch.zeros((B, K, cfg.vocab), dtype=torch.bfloat16, device=device)
    tl_buf = torch.zeros((B, K + 1, cfg.vocab), dtype=torch.bfloat16, device=device)
    th_buf = torch.zeros((B, K + 1, cfg.d_model), dtype=torch.bfloat16, device=device)
    mask = (1 << gmb.GM_KC_GEMM) | (1 << gmb.GM_KC_SAMPLER)
    phase_ms = {"draft_gemm": 0.0, "verify_gemm": 0.0, "accept_sampler": 0.0}
    phase_n = {"draft_gemm": 0, "verify_gemm": 0, "accept_sampler": 0}
    rows_read = 0
    for _ in range(np_steps):
        gmb.gm_profile(ctx, mask)
        gmb.gm_draft(ctx, st, K, 1.0, None, seed, step_id, d_dev, dl_buf)
        t_ms, n = gmb.gm_profile_read(ctx, gmb.GM_KC_GEMM)
        phase_ms["draft_gemm"] += t_ms; phase_n["draft_gemm"] += n
        gmb.gm_profile(ctx, mask)
        gmb.gm_verify(ctx, st, K, d_dev, tl_buf, th_buf)
        t_ms, n = gmb.gm_profile_read(ctx, gmb.GM_KC_GEMM)
        phase_ms["verify_gemm"] += t_ms; phase_n["verify_gemm"] += n
        gmb.gm_profile(ctx, mask)
        gmb.gm_accept(ctx, st, B, K, 1.0, tl_buf, dl_buf, d_dev, None, seed, step_id, a_dev, t_dev, None, None, th_buf,
                      commit_state=True)
        t_ms, n = gmb.gm_profile_read(ctx, gmb.GM_KC_SAMPLER)
        phase_ms["accept_sampler"] += t_ms; phase_n["accept_sampler"] += n
        av = a_dev.cpu().numpy()
        rows_read += int(np.where(av < K, 2 * (av + 1), 2 * K + 1).sum())   # the walk stops at the first rejection
        step_id += 1
    gmb.gm_profile(ctx, 0)
    del dl_buf, tl_buf, th_buf
    c3 = sampler_c3_roofline(gmb, device, K) if (rank == 0 and args.workload in ("4b", "7b")) else None

    # ---- end to end through the host-buffer entry point -------------------------------------------------------------
    ud_h = torch.randint(0, 1 << 24, (B, K), dtype=torch.int32).pin_memory()
    ua_h = torch.randint(0, 1 << 24, (B, K + 1), dtype=torch.int32).pin_memory()
    a_h = torch.zeros(B, dtype=torch.int32).pin_memory()
    t_h = torch.zeros(B, dtype=torch.int32).pin_memory()
    d_h = torch.zeros((B, K), dtype=torch.int32).pin_memory()
    gmb.gm_spec_step_host(ctx, st, K, 1.0, seed, step_id, a_h, t_h, d_h, ud_h, ua_h)      # warm the path
    barrier()
    t0 = time.perf_counter()
    committed_e2e = 0
    accept_hist = np.zeros(K + 1, np.int64)                # accepted lengths seen on the host (free: they arrive anyway)
    for i in range(S):
        gmb.gm_spec_step_host(ctx, st, K, 1.0, seed, step_id + 1 + i, a_h, t_h, d_h, ud_h, ua_h)
        committed_e2e += int(a_h.sum()) + B
        accept_hist += np.bincount(a_h.numpy(), minlength=K + 1)[:K + 1]
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    h2d = int(ud_h.numel() + ua_h.numel()) * 4
    d2h = int(a_h.numel() + t_h.numel() + d_h.numel()) * 4

    # ---- reduce over ranks (max time, summed tokens) ---------------------------------------------------------------------
    (ms_max, e2e_ms_max), (committed_all, committed_e2e_all, launches_all, batch_all) = reduce_over_ranks(
        [ms, e2e_s * 1e3], [committed, committed_e2e, launches, B], device, world)

    if rank == 0:
        hbm, tf_burst, tf_sust, which = measured_peaks()
        M_rows = B * (K + 1)
        layer_params = cfg.layer_params()
        head_params = layer_params + 2 * cfg.d_model ** 2
        lm_params = cfg.vocab * cfg.d_model
        v_flops = 2.0 * M_rows * (cfg.n_layers * layer_params + lm_params)
        v_bytes = 2.0 * (cfg.n_layers * layer_params + lm_params)
        v_ms = phase_ms["verify_gemm"] / np_steps
        d_bytes = 2.0 * K * (head_params + lm_params)
        d_ms = phase_ms["draft_gemm"] / np_steps
        s_ms = phase_ms["accept_sampler"] / max(phase_n["accept_sampler"], 1)
        s_bytes_all = B * (2 * K + 1) * cfg.vocab * 2.0
        s_bytes_read = rows_read / np_steps * cfg.vocab * 2.0
        rooflines = [
            {"kernel": "verify_gemm (target projections of all layers + LM head, M = batch x (k+1) rows)", "bound": "tensor",
             "achieved": v_flops / (v_ms * 1e-3) / 1e12, "peak": tf_burst, "unit": "TFLOP/s",
             "frac": v_flops / (v_ms * 1e-3) / 1e12 / tf_burst, "frac_of_sustained": v_flops / (v_ms * 1e-3) / 1e12 / tf_sust,
             "ms_per_step": v_ms, "launches_per_step": phase_n["verify_gemm"] / np_steps,
             "weights_GB_per_s": v_bytes / (v_ms * 1e-3) / 1e9, "weights_frac_of_hbm": v_bytes / (v_ms * 1e-3) / 1e9 / hbm,
             "note": "launches bracketed by events one by one (no overlap between them): peak = the burst figure"},
            {"kernel": "draft_gemm (k head applications: projection, one layer, shared LM head)", "bound": "hbm",
             "achieved": d_bytes / (d_ms * 1e-3) / 1e9, "peak": hbm, "unit": "GB/s",
             "frac": d_bytes / (d_ms * 1e-3) / 1e9 / hbm, "ms_per_step": d_ms,
             "launches_per_step": phase_n["draft_gemm"] / np_steps},
            {"kernel": "sampler (the cycle's accept / resample launch)", "bound": "hbm",
             "achieved": s_bytes_read / (s_ms * 1e-3) / 1e9, "peak": hbm, "unit": "GB/s",
             "frac": s_bytes_read / (s_ms * 1e-3) / 1e9 / hbm, "ms_per_launch": s_ms,
             "bytes_read_per_launch": s_bytes_read, "bytes_all_rows": s_bytes_all,
             "effective_GB_per_s_all_rows": s_bytes_all / (s_ms * 1e-3) / 1e9,
             "note": "achieved counts the rows the walk reads (it stops at the first rejection); all_rows = (2k+1) rows per sequence"},
        ]
        if c3 is not None:
            c3.update({"peak": hbm, "frac": c3["achieved"] / hbm, "frac_of_nominal_8TBs": c3["achieved"] / NOMINAL_HBM_GBS})
            rooflines.append(c3)
        sum_len_avg = 0.5 * (len0 + len1) + B * (K + 1)               # positions attended per launch (incl. new ones)
        att_bytes = sum_len_avg * cfg.kv_bytes_per_token(1)
        att_avg_ms = att_ms / max(att_n, 1)
        achieved = att_bytes / (att_avg_ms * 1e-3) / 1e9
        step_bytes = algorithmic_bytes_per_step(cfg, K, 0.5 * (len0 + len1))
        step_roof_ms = step_bytes / (hbm * 1e9) * 1e3
        line = {
            "metric": METRIC, "value": committed_all / (ms_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": S,
            "warmup": W, "ms_per_step": ms_max / S, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "n_layers": cfg.n_layers, "batch_per_gpu": B, "k": K, "temperature": 1.0,
                       "top_p": args.top_p, "kv_len_mean": float(lens.mean()), "kv_len_min": int(lens.min()), "kv_len_max": int(lens.max()),
                       "page": 16, "tau": committed / (S * B),
                       # per-position acceptance alpha_k = P(draft k accepted | drafts 1..k-1 accepted), rank 0, e2e region
                       "accept_by_position": [float(accept_hist[k:].sum() / max(accept_hist[k - 1:].sum(), 1))
                                              for k in range(1, K + 1)],
                       "parallelism": f"replicas x{world}",
                       "l2": "per-step working set (weights + KV, tens of GB) >> 126 MB L2: no flush needed",
                       "step_algorithmic_GB": step_bytes / 1e9, "step_roofline_ms": step_roof_ms,
                       "step_roofline_frac": step_roof_ms / (ms / S), "peaks": which},
            "clocks": clk,
            "e2e": {"value": committed_e2e_all / (e2e_ms_max * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms_max / S,
                    "launch": "one captured CUDA graph per cycle (the device-timed region above is host-launched: "
                              "its attention launches are bracketed by events for the roofline)"},
            "gpu_launches": int(launches_all),
            "roofline": {"kernel": "attention_kernel (paged multi-query decode attention, one layer per launch)",
                         "bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s", "frac": achieved / hbm,
                         "traffic": ATTENTION_TRAFFIC_RATIO * att_bytes, "launches": int(att_n), "avg_launch_ms": att_avg_ms,
                         "algorithmic_bytes_per_launch": att_bytes, "peak_source": which,
                         "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS},
            "rooflines": rooflines,
            "peaks": {"hbm_GB_per_s": hbm, "bf16_TFLOP_per_s_burst": tf_burst, "bf16_TFLOP_per_s_sustained": tf_sust,
                      "source": which, "nominal_hbm_GB_per_s": NOMINAL_HBM_GBS},
        }
        if breakdown is not None:
            line["config"]["breakdown"] = breakdown
        if rec is not None and rec_n:
            rb = B * K * cfg.vocab * 2
            line["config"]["record"] = {"what": "per-cycle record (top-64 target log-probs of k positions + 4 small items)",
                                        "topk_ms_per_launch": rec_ms / rec_n, "algorithmic_bytes": rb,
                                        "GB_per_s": rb / (rec_ms / rec_n * 1e-3) / 1e9}
        if not args.no_cpu_baseline and world >= 1:
            try:
                line["cpu_baseline"] = cpu_baseline(args.workload, K)
            except Exception as exc:                        # the baseline is reported, never required
                line["cpu_baseline"] = {"value": None, "unit": UNIT, "cores": 0, "kind": "oracle",
                                        "sample": f"failed: {exc}"}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_rollout(args):
    """Whole-rollout workload on the 4B shape (not the default line): prompts of 128..1024 random tokens are
    prefilled on the device, pages come from the library's allocator, and the rollout driver runs cycles (one
    captured CUDA graph per cycle) with responses collected on the device.  A step is one cycle over the batch;
    `e2e` is the whole job (prompt upload, prefill, warm-up + timed cycles, response download) by the host clock."""
    import torch
    import paper_2609_16648_b200 as gmb
    from paper_2609_16648_b200.build import build
    from synth_inputs import get_config
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the product path has no CPU fallback")
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    torch.cuda.set_stream(torch.cuda.Stream(device))
    K, W, S = args.k, args.warmup, args.steps
    cfg = get_config("4b").with_(k=K)
    if args.layers > 0:
        cfg = cfg.with_(n_layers=args.layers)
    if args.batch > 0:
        cfg = cfg.with_(batch=args.batch)
    B, V = cfg.batch, cfg.vocab
    rng = np.random.default_rng(11 + rank)
    plen = rng.integers(128, 1025, B).astype(np.int32)
    pmax = int(plen.max())
    tok = np.zeros((B, pmax), np.int32)
    for b in range(B):
        tok[b, :plen[b]] = rng.integers(0, V, plen[b])
    cycles = W + S
    max_new = cycles * (K + 1) + 1
    per_seq_pages = (pmax + max_new + K + 1 + 15) // 16 + 1
    npg = int(sum((int(l) + max_new + K + 1 + 15) // 16 + 1 for l in plen))       # what the batch can need, not B x the cap
    packed = gmb.random_packed_weights(cfg, device, seed=rank)
    ctx = gmb.Context(cfg, packed, B, K, per_seq_pages, npg, npg, flags=gmb.GM_FLAG_GRAPH)
    empty = np.full((B, per_seq_pages), -1, np.int32)
    st = gmb.State(ctx, B, empty, empty, device)
    ro = gmb.Rollout(B, max_new, -1, device)
    tok_h, len_h = torch.from_numpy(tok).pin_memory(), torch.from_numpy(plen).pin_memory()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    barrier()
    t_job = time.perf_counter()
    tok_d, len_d = tok_h.to(device, non_blocking=True), len_h.to(device, non_blocking=True)
    gmb.gm_pages_reset(ctx, st)
    gmb.gm_pages_reserve(ctx, st, len_d, K + 1)
    e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    e[0].record()
    gmb.gm_prefill(ctx, st, tok_d, len_d, pmax, 1.0, None, 77 + rank)
    e[1].record()
    gmb.gm_rollout_begin(ctx, st, ro)
    gmb.gm_rollout_run(ctx, st, ro, K, 1.0, 77 + rank, 1, W, W)
    n0 = int(ro.out_len.sum().item())
    len0 = int(st.kv_len.sum().item())
    clocks = ClockSampler(local)
    launches0 = gmb.gm_launch_count(ctx)
    barrier()
    clocks.start()
    e[2].record()
    steps, running = gmb.gm_rollout_run(ctx, st, ro, K, 1.0, 77 + rank, 1 + W, S, S)
    e[3].record()
    barrier()
    clk = clocks.stop()
    ms = e[2].elapsed_time(e[3])
    prefill_ms = e[0].elapsed_time(e[1])
    launches = gmb.gm_launch_count(ctx) - launches0
    out_len = ro.out_len.cpu()
    resp = ro.out_tok.cpu()                                   # the responses leave the device
    torch.cuda.synchronize()
    job_s = time.perf_counter() - t_job
    committed = int(out_len.sum().item()) - n0
    len1 = int(st.kv_len.sum().item())
    status = gmb.gm_last_status(ctx)
    if status != 0 or steps != S or running != B:
        raise RuntimeError(f"rollout workload: status {status}, {steps} cycles, {running} rows running")
    free_t, free_h = gmb.gm_pages_free_count(ctx)
    (ms_max, job_ms_max, prefill_ms_max), (committed_all, launches_all, tokens_job, prompt_tokens) = reduce_over_ranks(
        [ms, job_s * 1e3, prefill_ms], [committed, launches, int(out_len.sum().item()), int(plen.sum())], device, world)
    if rank == 0:
        hbm, _, _, which = measured_peaks()
        step_bytes = algorithmic_bytes_per_step(cfg, K, 0.5 * (len0 + len1))
        achieved = step_bytes / (ms_max / S * 1e-3) / 1e9
        line = {"metric": METRIC, "value": committed_all / (ms_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": S,
                "warmup": W, "ms_per_step": ms_max / S, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic",
                "config": {"workload": "rollout", "n_layers": cfg.n_layers, "batch_per_gpu": B, "k": K, "temperature": 1.0,
                           "prompt_len": "uniform 128..1024", "prompt_tokens": int(prompt_tokens),
                           "prefill_ms": prefill_ms_max, "prefill_tokens_per_s": prompt_tokens / (prefill_ms_max * 1e-3),
                           "kv_len_mean": 0.5 * (len0 + len1) / B, "tau": committed / (S * B),
                           "pages": {"pool": npg, "free_after": free_t}, "launch": "one captured CUDA graph per cycle",
                           "parallelism": f"replicas x{world}",
                           "l2": "per-cycle working set (weights + KV) >> 126 MB L2: no flush needed", "peaks": which},
                "clocks": clk,
                "e2e": {"value": tokens_job / (job_ms_max * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0, "h2d_bytes_per_job": int(tok.nbytes + plen.nbytes),
                        "d2h_bytes_per_job": int(resp.numel() * 4 + out_len.numel() * 4), "job_ms": job_ms_max,
                        "note": "whole job by the host clock: prompt upload, page reservation, prefill, warm-up and timed "
                                "cycles, response download; response tokens / job time"},
                "gpu_launches": int(launches_all),
                "roofline": {"kernel": "whole cycle (per-kernel events are not recorded inside a replayed graph)",
                             "bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s", "frac": achieved / hbm,
                             "traffic": None, "algorithmic_bytes_per_launch": step_bytes, "peak_source": which},
                "cpu_baseline": None}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def sampler_c3_roofline(gmb, device, K, batch=256, launches=20):
    """The sampler-only configuration (256 sequences x (k+1) positions, vocabulary 151936) timed launch by launch:
    the configuration the sampler's bar is stated on, reported beside the cycle's numbers."""
    import torch
    from synth_inputs import get_config, sampler_only_logits
    from synth_inputs.workload import random_u24
    cfg = get_config("sampler")
    V = cfg.vocab
    mcfg = cfg.with_(n_layers=1, d_model=64, n_q_heads=1, n_kv_heads=1, head_dim=64, d_ffn=64, batch=batch)
    ctx = gmb.Context(mcfg, gmb.random_packed_weights(mcfg, device), batch, K, 4, 8, 8)
    tgt, drf = sampler_only_logits(batch, K, V, sigma=0.908, seed=4)
    t_dev = torch.from_numpy(tgt).to(torch.bfloat16).to(device)
    d_dev = torch.from_numpy(drf).to(torch.bfloat16).to(device)
    ud = torch.from_numpy(random_u24((batch, K), seed=5).astype(np.int32)).to(device)
    ua = torch.from_numpy(random_u24((batch, K + 1), seed=6).astype(np.int32)).to(device)
    dtok = torch.zeros((batch, K), dtype=torch.int32, device=device)
    col = torch.zeros(batch, dtype=torch.int32, device=device)
    for k in range(K):
        gmb.gm_draw(ctx, d_dev[:, k].contiguous(), batch, 1.0, ud[:, k].contiguous(), col)
        dtok[:, k] = col
    a = torch.zeros(batch, dtype=torch.int32, device=device)
    t = torch.zeros(batch, dtype=torch.int32, device=device)
    for _ in range(3):
        gmb.gm_accept(ctx, None, batch, K, 1.0, t_dev, d_dev, dtok, ua, 0, 0, a, t)
    gmb.gm_profile(ctx, 1 << gmb.GM_KC_SAMPLER)
    for _ in range(launches):
        gmb.gm_accept(ctx, None, batch, K, 1.0, t_dev, d_dev, dtok, ua, 0, 0, a, t)
    ms, n = gmb.gm_profile_read(ctx, gmb.GM_KC_SAMPLER)
    gmb.gm_profile(ctx, 0)
    av = a.cpu().numpy()
    rows = int(np.where(av < K, 2 * (av + 1), 2 * K + 1).sum())
    ctx.close()
    avg = ms / max(n, 1)
    return {"kernel": "sampler, sampler-only configuration (256 x (k+1) positions, V = 151936, acceptance 0.65)", "bound": "hbm",
            "achieved": rows * V * 2.0 / (avg * 1e-3) / 1e9, "unit": "GB/s", "ms_per_launch": avg,
            "bytes_read_per_launch": rows * V * 2.0, "bytes_all_rows": batch * (2 * K + 1) * V * 2.0,
            "effective_GB_per_s_all_rows": batch * (2 * K + 1) * V * 2.0 / (avg * 1e-3) / 1e9,
            "note": "achieved counts the rows the walk reads (it stops at the first rejection)"}


def run_sampler_only(args):
    """Sampler-only workload: 256 sequences x (k+1) positions over the 151936-token vocabulary.  A step is one
    gm_accept over the whole batch (the draft tokens were drawn once, on the device, by gm_draw)."""
    import torch
    import paper_2609_16648_b200 as gmb
    from paper_2609_16648_b200.build import build
    from synth_inputs import get_config, sampler_only_logits
    from synth_inputs.workload import random_u24
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the product path has no CPU fallback")
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    build()
    cfg = get_config("sampler")
    B, K, V, S, W = (args.batch or cfg.batch), args.k, cfg.vocab, args.steps, args.warmup
    mcfg = cfg.with_(n_layers=1, d_model=64, n_q_heads=1, n_kv_heads=1, head_dim=64, d_ffn=64, batch=B)
    ctx = gmb.Context(mcfg, gmb.random_packed_weights(mcfg, device), B, K, 4, 8, 8)
    if args.top_p < 1.0:
        gmb.gm_set_top_p(ctx, args.top_p)
    tgt, drf = sampler_only_logits(B, K, V, sigma=0.908, seed=4 + rank)
    t_h = torch.from_numpy(tgt).to(torch.bfloat16).pin_memory()
    d_h = torch.from_numpy(drf).to(torch.bfloat16).pin_memory()
    t_dev, d_dev = t_h.to(device), d_h.to(device)
    ud = torch.from_numpy(random_u24((B, K), seed=5).astype(np.int32)).to(device)
    ua_h = torch.from_numpy(random_u24((B, K + 1), seed=6).astype(np.int32)).pin_memory()
    ua = ua_h.to(device)
    dtok = torch.zeros((B, K), dtype=torch.int32, device=device)
    col = torch.zeros(B, dtype=torch.int32, device=device)
    for k in range(K):
        gmb.gm_draw(ctx, d_dev[:, k].contiguous(), B, 1.0, ud[:, k].contiguous(), col)
        dtok[:, k] = col
    a = torch.zeros(B, dtype=torch.int32, device=device)
    t = torch.zeros(B, dtype=torch.int32, device=device)
    step = lambda: gmb.gm_accept(ctx, None, B, K, 1.0, t_dev, d_dev, dtok, ua, 0, 0, a, t)
    for _ in range(W):
        step()
    torch.cuda.synchronize()
    clocks = ClockSampler(local)
    gmb.gm_profile(ctx, 1 << gmb.GM_KC_SAMPLER)
    l0 = gmb.gm_launch_count(ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    clocks.start()
    e0.record()
    for _ in range(S):
        step()
    e1.record()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    clk = clocks.stop()
    k_ms, k_n = gmb.gm_profile_read(ctx, gmb.GM_KC_SAMPLER)
    gmb.gm_profile(ctx, 0)
    launches = gmb.gm_launch_count(ctx) - l0
    committed = (int(a.sum().item()) + B) * S
    # end to end: logits, tokens and uniforms from pinned host memory every step, results back to the host
    a_h, n_h = torch.zeros(B, dtype=torch.int32).pin_memory(), torch.zeros(B, dtype=torch.int32).pin_memory()
    dtok_h = dtok.cpu().pin_memory()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(S):
        t_dev.copy_(t_h, non_blocking=True)
        d_dev.copy_(d_h, non_blocking=True)
        dtok.copy_(dtok_h, non_blocking=True)
        ua.copy_(ua_h, non_blocking=True)
        step()
        a_h.copy_(a, non_blocking=True)
        n_h.copy_(t, non_blocking=True)
        torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    h2d = (t_h.numel() + d_h.numel()) * 2 + (dtok_h.numel() + ua_h.numel()) * 4
    (ms_max, e2e_max), (committed_all, launches_all) = reduce_over_ranks([ms, e2e_ms], [committed, launches], device, world)
    if rank == 0:
        hbm, _, _, which = measured_peaks()
        av = a.cpu().numpy()
        rows = int(np.where(av < K, 2 * (av + 1), 2 * K + 1).sum())     # the walk stops at the first rejection
        bytes_all = B * (2 * K + 1) * V * 2
        bytes_launch = rows * V * 2
        avg_ms = k_ms / max(k_n, 1)
        achieved = bytes_launch / (avg_ms * 1e-3) / 1e9
        line = {"metric": METRIC, "value": committed_all / (ms_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": S,
                "warmup": W, "ms_per_step": ms_max / S, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic",
                "config": {"workload": "sampler", "batch_per_gpu": B, "k": K, "vocab": V, "temperature": 1.0, "top_p": args.top_p,
                           "tau": committed / (S * B), "l2": "544 MB of logits per step > 126 MB L2: no flush needed",
                           "peaks": which},
                "clocks": clk,
                "e2e": {"value": committed_all / (e2e_max * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": 2 * B * 4, "ms_per_step": e2e_max / S},
                "gpu_launches": int(launches_all),
                "roofline": {"kernel": "sampler_kernel (softmax + rejection + residual resampling)", "bound": "hbm",
                             "achieved": achieved, "peak": hbm, "unit": "GB/s", "frac": achieved / hbm, "traffic": None,
                             "launches": int(k_n), "avg_launch_ms": avg_ms, "algorithmic_bytes_per_launch": bytes_launch,
                             "bytes_all_rows": bytes_all, "effective_GB_per_s_all_rows": bytes_all / (avg_ms * 1e-3) / 1e9,
                             "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "peak_source": which,
                             "note": "achieved counts the rows the walk reads (it stops at the first rejection); "
                                     "all_rows = (2k+1) rows per sequence, the scope table's figure"}}
        if not args.no_cpu_baseline:
            from oracle import sampler as osampler
            n = 8
            t1 = time.time()
            ea, _, _ = osampler.accept_batch(tgt[:n], drf[:n], dtok_h.numpy()[:n], ua_h.numpy()[:n].astype(np.uint32), 1.0)
            dt = time.time() - t1
            line["cpu_baseline"] = {"value": float((ea.sum() + n) / dt), "unit": UNIT, "cores": host_cores(), "kind": "oracle",
                                    "sample": f"oracle softmax + decision function on the first {n} of {B} rows ({dt:.1f} s)"}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def spawn_ranks(args):
    """`python bench.py --gpus N` outside a launcher: start one rank per GPU on this node ourselves (the same
    torch.distributed.run invocation the scaling driver uses) and hand over to it."""
    import subprocess
    cmd = [sys.executable, "-m", "torch.distributed.run", "--standalone", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--local-addr", "127.0.0.1", os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    sys.exit(subprocess.run(cmd, env=env).returncode)


def run_dry(args):
    """Launcher check without kernels (`--dry-run`): every rank joins the process group (NCCL on GPUs, gloo without),
    the replicas' token counts are summed and their times maximised as in a real run, and rank 0 prints the line."""
    import torch
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    cuda = torch.cuda.is_available()
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0"))) if cuda else torch.device("cpu")
    if world > 1:
        dist.init_process_group("nccl" if cuda else "gloo")
    from synth_inputs import get_config
    lens = lengths_for(get_config("4b"), seed=3 + rank)            # every replica draws its own batch
    (ms_max,), (tokens, ranks) = reduce_over_ranks([1.0 + rank], [len(lens), 1], device, world)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT, "n_gpus": int(ranks), "dry_run": True,
                          "sequences_all_ranks": int(tokens), "ms_max_over_ranks": ms_max, "scaling": "weak",
                          "config": {"workload": "launcher check", "parallelism": f"replicas x{world}"}}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_head_update(args):
    """Head-update workload (not the default line): one update of the draft head (Alg. 1, "update phi") per step on synthetic
    recorded cycles at the 4B head's dimensions - 256 cycles spread over 64 recorded sequences of 512 positions, chains
    replayed in chunks of --update-chunk (the context's max_batch; 128 measured best: 42.0 / 33.5 / 34.3 ms at 64 / 128 / 256).  A step is one gm_head_update_step: cache rebuild, reconstruction, objective, backward pass
    over every head parameter, AdamW.  `e2e` adds the upload of the step's records from pinned host memory and the
    download of the objective."""
    import torch
    import paper_2609_16648_b200 as gmb
    from paper_2609_16648_b200.build import build
    from synth_inputs import get_config, make_page_tables
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the product path has no CPU fallback")
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    K, W, S = args.k, args.warmup, args.steps
    n_seq, L, n = (args.batch if args.batch > 0 else 64), 512, 256
    cfg = get_config("4b").with_(n_layers=1, batch=n_seq, k=K, qk_norm=True)
    d, V, F = cfg.d_model, cfg.vocab, cfg.d_ffn
    hpt, hnpg = make_page_tables(np.full(n_seq, L + 8), 16, seed=8 + rank)
    MB = args.update_chunk
    ctx = gmb.Context(cfg, gmb.random_packed_weights(cfg, device, seed=rank), MB, K, hpt.shape[1], 8, hnpg + 2 * n)
    gst = gmb.State(ctx, n_seq, hpt, hpt, device)
    g = torch.Generator(device=device).manual_seed(1 + rank)
    tok = torch.randint(0, V, (n_seq, L), device=device, generator=g, dtype=torch.int32)
    hid = torch.randn((n_seq, L, d), device=device, generator=g).to(torch.bfloat16)
    slen = torch.full((n_seq,), L, dtype=torch.int32, device=device)
    rng = np.random.default_rng(3 + rank)
    seq = rng.integers(0, n_seq, n).astype(np.int32)
    start = rng.integers(L // 2, L - K - 1, n).astype(np.int32)
    rec = gmb.Record(n, K, d, device)
    rec.start_pos.copy_(torch.from_numpy(start))
    rec.start_hidden.copy_(hid[torch.from_numpy(seq).long().to(device), torch.from_numpy(start - 2).long().to(device)])
    rec.drafts.copy_(torch.randint(0, V, (n, K), device=device, generator=g, dtype=torch.int32))
    rec.top_index.copy_(torch.rand((n * K, V), device=device, generator=g).topk(64, dim=-1).indices.reshape(n, K, 64).to(torch.int32))
    lp = torch.log_softmax(torch.randn((n, K, 64), device=device, generator=g) * 2, -1) - 0.3
    rec.top_logprob.copy_(lp.sort(dim=-1, descending=True).values.to(torch.bfloat16))
    rec.accepted.copy_(torch.randint(1, K + 2, (n,), device=device, generator=g, dtype=torch.int32))
    cyc = torch.from_numpy(seq).to(device)
    scratch = torch.arange(hnpg, hnpg + 2 * n, dtype=torch.int32, device=device).reshape(n, 2)
    mean = torch.zeros(1, device=device)
    step_no = [0]

    def step():
        step_no[0] += 1
        gmb.gm_head_update_step(ctx, gst, n, K, 1.0, cyc, rec, tok, scratch, hid, slen, L, step_no[0], 1e-4, mean)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(W):
        step()
    clocks = ClockSampler(local)
    launches0 = gmb.gm_launch_count(ctx)
    barrier()
    clocks.start()
    e = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    e[0].record()
    for _ in range(S):
        step()
    e[1].record()
    barrier()
    clk = clocks.stop()
    ms = e[0].elapsed_time(e[1])
    launches = gmb.gm_launch_count(ctx) - launches0
    # end to end: the step's records come from pinned host memory, the objective goes back
    fields = ("start_hidden", "start_pos", "drafts", "top_logprob", "top_index", "accepted")
    host = {f: getattr(rec, f).cpu().pin_memory() for f in fields}
    mean_h = torch.zeros(1).pin_memory()
    barrier()
    t0 = time.perf_counter()
    for _ in range(S):
        for f in fields:
            getattr(rec, f).copy_(host[f], non_blocking=True)
        step()
        mean_h.copy_(mean, non_blocking=True)
        torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    h2d = sum(host[f].numel() * host[f].element_size() for f in fields)
    # device time of the projections, every launch bracketed by events, in a pass of its own
    gmb.gm_profile(ctx, 1 << 0)
    step()
    gemm_ms, gemm_n = gmb.gm_profile_read(ctx, 0)
    gmb.gm_profile(ctx, 0)
    status = gmb.gm_last_status(ctx)
    if status != 0 or not np.isfinite(float(mean[0])):
        raise RuntimeError(f"head_update workload: status {status}, objective {float(mean[0])}")
    (ms_max, e2e_max), (launches_all,) = reduce_over_ranks([ms, e2e_ms], [launches], device, world)
    if rank == 0:
        _, burst, sustained, which = measured_peaks()
        nqkv, q = cfg.q_dim + 2 * cfg.kv_dim, cfg.q_dim
        P, C = n_seq * (L - 1), n * K                     # prefix rows, chain rows (one per application)
        zf, qf, of, ff, lf = 2.0 * 2 * d * d, 2.0 * nqkv * d, 2.0 * q * d, 2.0 * F * d, 2.0 * V * d
        # prefix rows: z and QKV in the rebuild and again in the backward pass, then dh, dW_qkv, d zin, dW_p
        flops = P * (2 * (zf + qf) + 2 * qf + 2 * zf)
        # chain rows: one replay (z, layer, LM head; the call-by-call sequence makes two), LM-head gradient, feed-forward backward (recomputed gate/up + four
        # products), attention half (z, QKV, W_o forward; d out, dh, two weight gradients), input (d zin, dW_p)
        flops += C * ((zf + qf + of + 3 * ff + lf) + lf + (2 * ff + ff + 2 * ff + ff + 2 * ff) + (zf + qf + of + of + qf + of + qf) + 2 * zf)
        tf = flops / (gemm_ms * 1e-3) / 1e12
        line = {"metric": "head_update_cycles_per_s", "value": n * S * world / (ms_max * 1e-3), "unit": "recorded cycles/s",
                "n_gpus": world, "steps": S, "warmup": W, "ms_per_step": ms_max / S, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": "head_update", "cycles_per_step": n, "sequences": n_seq, "positions": L, "k": K,
                           "head": "4B dimensions (d 2560, 32/8 heads of 128 with head norms, FFN 9728, vocabulary 151936)",
                           "chains_per_chunk": MB, "l2": "the head's matrices and fp32 gradients (0.7 GB) exceed the 126 MB L2: no flush needed",
                           "peaks": which},
                "clocks": clk,
                "e2e": {"value": n * S * world / (e2e_max * 1e-3), "unit": "recorded cycles/s", "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": 4, "ms_per_step": e2e_max / S},
                "gpu_launches": int(launches_all),
                "roofline": {"kernel": "gemm_tc_kernel (every product of the update: forward recomputation, input gradients, weight gradients)",
                             "bound": "tensor", "achieved": tf, "peak": burst, "unit": "TFLOP/s", "frac": tf / burst,
                             "frac_of_sustained": tf / sustained, "traffic": None, "launches": int(gemm_n), "ms_per_step": gemm_ms,
                             "flops_per_step": flops, "peak_source": which,
                             "note": "launches bracketed by events one by one in a separate pass; most products have --update-chunk or 2048 rows"}}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="4b", choices=["tiny", "4b", "7b", "longtail", "sampler", "rollout", "head_update"])
    ap.add_argument("--k", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (small profiling cases)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (small profiling cases)")
    ap.add_argument("--record", action="store_true", help="also write the per-cycle verification record every step")
    ap.add_argument("--top-p", type=float, default=1.0,
                    help="nucleus of the target distributions (1 = none, the paper's rollout setting; its evaluation uses 0.7)")
    ap.add_argument("--update-chunk", type=int, default=128, help="head_update workload: chains replayed per pass (the context's max_batch)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--breakdown", action="store_true", help="add device time per kernel class (extra pass)")
    ap.add_argument("--dry-run", action="store_true", help="launcher check: ranks rendezvous and reduce, no kernels run")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "ours" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args)                               # does not return
    if args.impl == "ours" and args.gpus != int(os.environ.get("WORLD_SIZE", "1")):
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {os.environ.get('WORLD_SIZE', '1')} rank(s)")
    if args.dry_run:
        run_dry(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.workload == "sampler":
        run_sampler_only(args)
    elif args.workload == "rollout":
        run_rollout(args)
    elif args.workload == "head_update":
        run_head_update(args)
    else:
        run_product(args)


if __name__ == "__main__":
    main()
