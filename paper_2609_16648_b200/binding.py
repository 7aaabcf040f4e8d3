"""ctypes binding of libgm.so: the same entry points as include/gm.h, taking torch CUDA tensors.

Argument marshalling only - every step of the path runs in the library's kernels.  PyTorch is used
for device memory and streams.  Importing this module never falls back to a CPU path: if the
shared library is missing or fails to load, `lib()` raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libgm.so")

GM_OK = 0
GM_ERR_INVALID_ARG, GM_ERR_UNSUPPORTED, GM_ERR_KV_CAPACITY, GM_ERR_CUDA = -1, -2, -3, -4
GM_ERR_DEVICE_TIMEOUT, GM_ERR_BAD_PAGE, GM_ERR_NO_EXTENSION, GM_ERR_SCRATCH_LIMIT, GM_ERR_OVERRUN = -5, -6, -7, -8, -9
GM_NOALLOC_SCRATCH_BYTES, GM_NOALLOC_MAX_BATCH = 16 << 20, 256
GM_MAX_K, GM_PAGE = 7, 16
GM_FLAG_SIMPLE_GEMM, GM_FLAG_SAMPLER_CLUSTER, GM_FLAG_SAMPLER_STREAM, GM_FLAG_GRAPH, GM_FLAG_SAMPLER_FLOW = 1, 2, 4, 8, 16
GM_KC_GEMM, GM_KC_ATTENTION, GM_KC_ELEMENTWISE, GM_KC_SAMPLER, GM_KC_RECORD = 0, 1, 2, 3, 4

EXPORTS = ["gm_init", "gm_destroy", "gm_draft", "gm_verify", "gm_accept", "gm_spec_step", "gm_draw", "gm_set_top_p", "gm_nucleus", "gm_prefill",
           "gm_rollout_begin", "gm_rollout_step", "gm_rollout_run", "gm_pages_reset", "gm_pages_reserve",
           "gm_pages_release", "gm_pages_free_count", "gm_capture_hidden", "gm_head_prefill", "gm_reconstruct", "gm_reconstruct_states", "gm_head_state_grad", "gm_head_ffn_backward", "gm_attention_backward", "gm_head_attn_backward", "gm_head_update_backward", "gm_head_update_step", "gm_head_input_backward", "gm_adamw_step", "gm_overlap", "gm_dca_loss", "gm_dca_grad",
           "gm_spec_step_host", "gm_gemm", "gm_gemm_swiglu", "gm_attention", "gm_attention_noalloc", "gm_record_begin", "gm_record_end",
           "gm_spec_step_rec", "gm_profile", "gm_profile_read", "gm_chain_trace", "gm_chain_trace_read", "gm_selftest_wait_expiry", "gm_launch_count",
           "gm_last_status", "gm_strerror"]


class gm_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn",
                                          "vocab", "page_size", "max_batch", "max_k", "max_pages_per_seq",
                                          "num_pages", "head_num_pages")] + \
               [("rope_base", C.c_float), ("rms_eps", C.c_float), ("flags", C.c_int32)]


class gm_layer_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("ln1", "wqkv", "wo", "ln2", "w_gate_up", "w_down", "b_qkv", "q_norm", "k_norm")]


class gm_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("layers", C.POINTER(gm_layer_weights)),
                ("head_enorm", C.c_void_p), ("head_hnorm", C.c_void_p), ("head_proj", C.c_void_p),
                ("head_final_norm", C.c_void_p), ("head_layer", gm_layer_weights)]


class gm_state(C.Structure):
    _fields_ = [("batch", C.c_int32), ("kv_len", C.c_void_p), ("page_table", C.c_void_p), ("kv_pool", C.c_void_p),
                ("head_page_table", C.c_void_p), ("head_kv_pool", C.c_void_p), ("pending_n", C.c_void_p),
                ("pending_tok", C.c_void_p), ("pending_hidden", C.c_void_p)]


class gm_rollout(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("out_tok", "out_len", "finished", "n_running")] + \
               [(n, C.c_int32) for n in ("out_stride", "eos_token", "max_new")]


class gm_record(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("start_hidden", "start_pos", "drafts", "top_logprob", "top_index", "accepted")]


HEAD_GRAD_FIELDS = ("proj", "enorm", "hnorm", "final_norm", "ln1", "ln2", "wqkv", "wo", "w_gate_up", "w_down", "b_qkv", "qk_norm")


class gm_head_grads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in HEAD_GRAD_FIELDS]


_lib = None


def lib() -> C.CDLL:
    """Load libgm.so (built in-tree by paper_2609_16648_b200.build); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2609_16648_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i32, u64, f32 = C.c_void_p, C.c_int, C.c_uint64, C.c_float
    L.gm_init.argtypes = [C.POINTER(vp), C.POINTER(gm_config), C.POINTER(gm_weights), vp]
    L.gm_destroy.argtypes = [vp]
    L.gm_destroy.restype = None
    L.gm_draft.argtypes = [vp, C.POINTER(gm_state), i32, f32, vp, u64, u64, vp, vp, vp]
    L.gm_verify.argtypes = [vp, C.POINTER(gm_state), i32, vp, vp, vp]
    L.gm_accept.argtypes = [vp, C.POINTER(gm_state), i32, i32, f32, vp, vp, vp, vp, u64, u64, vp, vp, vp, vp, vp, i32]
    L.gm_spec_step.argtypes = [vp, C.POINTER(gm_state), i32, f32, u64, u64, vp, vp, vp]
    L.gm_spec_step_host.argtypes = [vp, C.POINTER(gm_state), i32, f32, u64, u64, vp, vp, vp, vp, vp]
    L.gm_draw.argtypes = [vp, vp, i32, f32, vp, vp, vp]
    L.gm_set_top_p.argtypes = [vp, f32]
    L.gm_rollout_begin.argtypes = [vp, C.POINTER(gm_state), C.POINTER(gm_rollout)]
    L.gm_rollout_step.argtypes = [vp, C.POINTER(gm_state), C.POINTER(gm_rollout), i32, f32, u64, u64]
    L.gm_rollout_run.argtypes = [vp, C.POINTER(gm_state), C.POINTER(gm_rollout), i32, f32, u64, u64, i32, i32,
                                 C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    L.gm_pages_reset.argtypes = [vp, C.POINTER(gm_state)]
    L.gm_capture_hidden.argtypes = [vp, vp, i32]
    L.gm_head_prefill.argtypes = [vp, C.POINTER(gm_state), vp, i32, vp, i32, vp, i32]
    L.gm_reconstruct.argtypes = [vp, C.POINTER(gm_state), i32, i32, vp, C.POINTER(gm_record), vp, i32, vp, vp]
    L.gm_reconstruct_states.argtypes = [vp, C.POINTER(gm_state), i32, i32, vp, C.POINTER(gm_record), vp, i32, vp, vp, vp]
    L.gm_head_state_grad.argtypes = [vp, i32, vp, vp, vp, vp, i32]
    L.gm_head_ffn_backward.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, i32]
    L.gm_attention_backward.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, i32, i32, vp, vp, vp]
    L.gm_head_attn_backward.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, i32]
    L.gm_head_update_backward.argtypes = [vp, C.POINTER(gm_state), i32, i32, vp, C.POINTER(gm_record), vp, i32, vp, vp, vp, i32, vp, i32, vp,
                                          vp, C.POINTER(gm_head_grads)]
    L.gm_head_update_step.argtypes = [vp, C.POINTER(gm_state), i32, i32, f32, vp, C.POINTER(gm_record), vp, i32, vp, vp, i32, vp, i32, i32,
                                      f32, f32, f32, f32, f32, vp]
    L.gm_head_input_backward.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, i32]
    L.gm_adamw_step.argtypes = [vp, C.c_int64, vp, vp, vp, vp, vp, i32, f32, f32, f32, f32, f32, f32]
    L.gm_overlap.argtypes = [vp, i32, i32, f32, vp, C.POINTER(gm_record), vp, vp]
    L.gm_dca_loss.argtypes = [vp, i32, i32, vp, vp, vp, vp]
    L.gm_dca_grad.argtypes = [vp, i32, i32, f32, vp, C.POINTER(gm_record), vp, vp, vp, vp]
    L.gm_pages_reserve.argtypes = [vp, C.POINTER(gm_state), vp, i32, vp]
    L.gm_pages_release.argtypes = [vp, C.POINTER(gm_state), vp]
    L.gm_pages_free_count.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    L.gm_prefill.argtypes = [vp, C.POINTER(gm_state), vp, vp, i32, i32, f32, vp, u64, vp, vp]
    L.gm_nucleus.argtypes = [vp, vp, i32, f32, f32, vp, vp]
    L.gm_gemm.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32]
    L.gm_gemm_swiglu.argtypes = [vp, vp, vp, vp, i32, i32, i32]
    L.gm_attention.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp, i32, i32, vp]
    L.gm_attention_noalloc.argtypes = [i32, i32, i32, i32, vp, vp, i32, i32, i32, vp, vp, vp, i32, i32, vp, vp]
    L.gm_record_begin.argtypes = [vp, C.POINTER(gm_state), C.POINTER(gm_record)]
    L.gm_record_end.argtypes = [vp, i32, i32, f32, vp, vp, vp, C.POINTER(gm_record)]
    L.gm_spec_step_rec.argtypes = [vp, C.POINTER(gm_state), i32, f32, u64, u64, vp, vp, vp, C.POINTER(gm_record)]
    L.gm_profile.argtypes = [vp, i32]
    L.gm_profile_read.argtypes = [vp, i32, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    L.gm_chain_trace.argtypes = [vp, i32]
    L.gm_chain_trace_read.argtypes = [vp, vp, i32]
    L.gm_selftest_wait_expiry.argtypes = [vp]
    L.gm_launch_count.argtypes = [vp]
    L.gm_launch_count.restype = C.c_int64
    L.gm_last_status.argtypes = [vp]
    L.gm_strerror.argtypes = [i32]
    L.gm_strerror.restype = C.c_char_p
    _lib = L
    return L


class GmError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {gm_strerror(code)} ({code})")


def gm_strerror(code: int) -> str:
    return lib().gm_strerror(code).decode()


def _check(code: int, where: str):
    if code != GM_OK:
        raise GmError(code, where)


def _p(t):
    """Device pointer of a tensor (None -> NULL)."""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    return C.c_void_p(t.data_ptr())


# ---- weights ---------------------------------------------------------------------------------------------------

def pack_layer(lw: dict, device) -> dict:
    """Canonical per-projection matrices -> the library's fused layout (bf16 on `device`):
    wqkv = [wq; wk; wv] stacked by rows, w_gate_up rows interleaved (2i = gate_i, 2i+1 = up_i).
    Family extras when present: b_qkv = [bq; bk; bv], q_norm, k_norm."""
    bf = lambda a: torch.as_tensor(a).to(device=device, dtype=torch.bfloat16).contiguous()
    wg, wu = torch.as_tensor(lw["wg"]), torch.as_tensor(lw["wu"])
    extra = {}
    if "bq" in lw:
        extra["b_qkv"] = bf(torch.cat([torch.as_tensor(lw[n]) for n in ("bq", "bk", "bv")], 0))
    if "qnorm" in lw:
        extra["q_norm"], extra["k_norm"] = bf(lw["qnorm"]), bf(lw["knorm"])
    return {
        **extra,
        "ln1": bf(lw["ln1"]), "ln2": bf(lw["ln2"]),
        "wqkv": bf(torch.cat([torch.as_tensor(lw["wq"]), torch.as_tensor(lw["wk"]), torch.as_tensor(lw["wv"])], 0)),
        "wo": bf(lw["wo"]),
        "w_gate_up": bf(torch.stack([wg, wu], 1).reshape(2 * wg.shape[0], wg.shape[1])),
        "w_down": bf(lw["wd"]),
    }


def pack_weights(w: dict, device="cuda") -> dict:
    """Canonical weights -> the library's layout.  A head whose "concat" entry is "hidden_first" was
    trained on [hidden ; embedding]: the two column halves of its projection are swapped here, so the
    library's fixed order [embedding ; hidden] computes the same function (App. B.1)."""
    bf = lambda a: torch.as_tensor(a).to(device=device, dtype=torch.bfloat16).contiguous()
    proj = torch.as_tensor(w["head"]["proj"])
    if w["head"].get("concat", "embedding_first") == "hidden_first":
        d = proj.shape[0]
        proj = torch.cat([proj[:, d:], proj[:, :d]], 1)
    w = dict(w, head=dict(w["head"], proj=proj))
    return {
        "embed": bf(w["embed"]), "lm_head": bf(w["lm_head"]), "final_norm": bf(w["final_norm"]),
        "layers": [pack_layer(lw, device) for lw in w["layers"]],
        "head": {"enorm": bf(w["head"]["enorm"]), "hnorm": bf(w["head"]["hnorm"]), "proj": bf(w["head"]["proj"]),
                 "final_norm": bf(w["head"]["final_norm"]), "layer": pack_layer(w["head"]["layer"], device)},
    }


def random_packed_weights(cfg, device="cuda", seed=0, std=0.02) -> dict:
    """Random weights generated directly on the device in the packed layout (large shapes)."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)

    def rnd(*shape):
        out = torch.empty(shape, device=device, dtype=torch.bfloat16)
        rows = max(1, (1 << 26) // max(1, shape[-1]))
        for r0 in range(0, shape[0], rows):          # in slabs, to bound the fp32 temporary
            r1 = min(shape[0], r0 + rows)
            out[r0:r1] = (torch.randn((r1 - r0,) + tuple(shape[1:]), device=device, generator=gen) * std).to(torch.bfloat16)
        return out

    ones = lambda n: torch.ones(n, device=device, dtype=torch.bfloat16)
    d, f = cfg.d_model, cfg.d_ffn

    def layer():
        lw = {"ln1": ones(d), "ln2": ones(d), "wqkv": rnd(cfg.q_dim + 2 * cfg.kv_dim, d), "wo": rnd(d, cfg.q_dim),
              "w_gate_up": rnd(2 * f, d), "w_down": rnd(d, f)}
        if getattr(cfg, "qkv_bias", False):
            lw["b_qkv"] = rnd(cfg.q_dim + 2 * cfg.kv_dim, 1).reshape(-1)
        if getattr(cfg, "qk_norm", False):
            lw["q_norm"], lw["k_norm"] = ones(cfg.head_dim), ones(cfg.head_dim)
        return lw

    return {"embed": rnd(cfg.vocab, d), "lm_head": rnd(cfg.vocab, d), "final_norm": ones(d),
            "layers": [layer() for _ in range(cfg.n_layers)],
            "head": {"enorm": ones(d), "hnorm": ones(d), "proj": rnd(d, 2 * d), "final_norm": ones(d),
                     "layer": layer()}}


def _layer_struct(lw: dict) -> gm_layer_weights:
    opt = [lw[n].data_ptr() if n in lw else None for n in ("b_qkv", "q_norm", "k_norm")]
    return gm_layer_weights(*[lw[n].data_ptr() for n in ("ln1", "wqkv", "wo", "ln2", "w_gate_up", "w_down")], *opt)


class Context:
    """Owns a gm_ctx and keeps the weight tensors alive."""

    def __init__(self, cfg, packed: dict, max_batch: int, max_k: int, max_pages_per_seq: int, num_pages: int,
                 head_num_pages: int, flags: int = 0, stream=None):
        self.cfg, self.packed = cfg, packed
        self.max_batch, self.max_k, self.max_pages_per_seq = max_batch, max_k, max_pages_per_seq
        self.num_pages, self.head_num_pages = num_pages, head_num_pages
        self._layers = (gm_layer_weights * len(packed["layers"]))(*[_layer_struct(l) for l in packed["layers"]])
        h = packed["head"]
        self._w = gm_weights(packed["embed"].data_ptr(), packed["lm_head"].data_ptr(), packed["final_norm"].data_ptr(),
                             self._layers, h["enorm"].data_ptr(), h["hnorm"].data_ptr(), h["proj"].data_ptr(),
                             h["final_norm"].data_ptr(), _layer_struct(h["layer"]))
        self._c = gm_config(len(packed["layers"]), cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn,
                            cfg.vocab, cfg.page_size, max_batch, max_k, max_pages_per_seq, num_pages, head_num_pages,
                            cfg.rope_base, cfg.rms_eps, flags)
        self.stream = torch.cuda.current_stream() if stream is None else stream
        self.handle = C.c_void_p()
        _check(lib().gm_init(C.byref(self.handle), C.byref(self._c), C.byref(self._w),
                             C.c_void_p(self.stream.cuda_stream)), "gm_init")

    def close(self):
        if self.handle:
            lib().gm_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class State:
    """Device tensors of struct gm_state."""

    def __init__(self, ctx: Context, batch: int, page_table, head_page_table, device="cuda"):
        cfg = ctx.cfg
        i32 = dict(device=device, dtype=torch.int32)
        self.batch = batch
        self.kv_len = torch.zeros(batch, **i32)
        self.page_table = torch.as_tensor(page_table).to(**i32).contiguous()
        self.head_page_table = torch.as_tensor(head_page_table).to(**i32).contiguous()
        assert self.page_table.shape == (batch, ctx.max_pages_per_seq) == self.head_page_table.shape
        L = len(ctx.packed["layers"])
        self.kv_pool = torch.zeros((L, 2, ctx.num_pages, cfg.n_kv_heads, 16, cfg.head_dim), device=device,
                                   dtype=torch.bfloat16)
        self.head_kv_pool = torch.zeros((1, 2, ctx.head_num_pages, cfg.n_kv_heads, 16, cfg.head_dim), device=device,
                                        dtype=torch.bfloat16)
        self.pending_n = torch.ones(batch, **i32)
        self.pending_tok = torch.zeros((batch, ctx.max_k + 1), **i32)
        self.pending_hidden = torch.zeros((batch, ctx.max_k + 1, cfg.d_model), device=device, dtype=torch.bfloat16)

    def struct(self) -> gm_state:
        return gm_state(self.batch, self.kv_len.data_ptr(), self.page_table.data_ptr(), self.kv_pool.data_ptr(),
                        self.head_page_table.data_ptr(), self.head_kv_pool.data_ptr(), self.pending_n.data_ptr(),
                        self.pending_tok.data_ptr(), self.pending_hidden.data_ptr())


# ---- entry points (same names as the C ABI) ------------------------------------------------------------------------

def gm_draft(ctx: Context, st: State, k: int, temperature: float, u24_draft, seed: int, step: int, draft_tok,
             draft_logits, dbg_q=None):
    s = st.struct()
    _check(lib().gm_draft(ctx.handle, C.byref(s), k, temperature, _p(u24_draft), seed, step, _p(draft_tok),
                          _p(draft_logits), _p(dbg_q)), "gm_draft")


def gm_verify(ctx: Context, st: State, k: int, draft_tok, target_logits, target_hidden):
    s = st.struct()
    _check(lib().gm_verify(ctx.handle, C.byref(s), k, _p(draft_tok), _p(target_logits), _p(target_hidden)), "gm_verify")


def gm_accept(ctx: Context, st, batch: int, k: int, temperature: float, target_logits, draft_logits, draft_tok,
              u24_accept, seed: int, step: int, accept_len, next_token, dbg_p=None, dbg_q=None, target_hidden=None,
              commit_state: bool = False):
    s = st.struct() if st is not None else None
    _check(lib().gm_accept(ctx.handle, C.byref(s) if s is not None else None, batch, k, temperature,
                           _p(target_logits), _p(draft_logits), _p(draft_tok), _p(u24_accept), seed, step,
                           _p(accept_len), _p(next_token), _p(dbg_p), _p(dbg_q), _p(target_hidden),
                           1 if commit_state else 0), "gm_accept")


def gm_spec_step(ctx: Context, st: State, k: int, temperature: float, seed: int, step: int, accept_len, next_token,
                 draft_tok=None):
    s = st.struct()
    _check(lib().gm_spec_step(ctx.handle, C.byref(s), k, temperature, seed, step, _p(accept_len), _p(next_token),
                              _p(draft_tok)), "gm_spec_step")


def gm_spec_step_host(ctx: Context, st: State, k: int, temperature: float, seed: int, step: int, accept_len_host,
                      next_token_host, draft_tok_host=None, u24_draft_host=None, u24_accept_host=None):
    """All tensor arguments are CPU tensors (pinned for asynchronous copies); int32 / uint32-valued."""
    s = st.struct()
    hp = lambda t: None if t is None else C.c_void_p(t.data_ptr())
    for t in (accept_len_host, next_token_host, draft_tok_host, u24_draft_host, u24_accept_host):
        assert t is None or (not t.is_cuda and t.is_contiguous())
    _check(lib().gm_spec_step_host(ctx.handle, C.byref(s), k, temperature, seed, step, hp(u24_draft_host),
                                   hp(u24_accept_host), hp(accept_len_host), hp(next_token_host), hp(draft_tok_host)),
           "gm_spec_step_host")


def gm_draw(ctx: Context, logits, rows: int, temperature: float, u24, out_tok, dbg_prob=None):
    _check(lib().gm_draw(ctx.handle, _p(logits), rows, temperature, _p(u24), _p(out_tok), _p(dbg_prob)), "gm_draw")


def gm_prefill(ctx: Context, st, prompt_tok, prompt_len, max_prompt_len: int, temperature: float, u24_first, seed: int,
               first_token=None, dbg_p=None):
    """prompt_tok int32 [B, stride] and prompt_len int32 [B] on the device; max_prompt_len a host integer."""
    _check(lib().gm_prefill(ctx.handle, C.byref(st.struct()), _p(prompt_tok), _p(prompt_len), prompt_tok.shape[1],
                            max_prompt_len, temperature, _p(u24_first), seed, _p(first_token), _p(dbg_p)), "gm_prefill")


class Rollout:
    """Device tensors of struct gm_rollout."""

    def __init__(self, batch: int, max_new: int, eos_token: int = -1, device="cuda"):
        i32 = dict(device=device, dtype=torch.int32)
        self.max_new, self.eos_token = max_new, eos_token
        self.out_tok = torch.zeros((batch, max_new), **i32)
        self.out_len = torch.zeros(batch, **i32)
        self.finished = torch.zeros(batch, **i32)
        self.n_running = torch.zeros(1, **i32)

    def struct(self) -> gm_rollout:
        return gm_rollout(self.out_tok.data_ptr(), self.out_len.data_ptr(), self.finished.data_ptr(),
                          self.n_running.data_ptr(), self.out_tok.shape[1], self.eos_token, self.max_new)

    def responses(self):
        tok, n = self.out_tok.cpu().numpy(), self.out_len.cpu().numpy()
        return [tok[b, :n[b]].tolist() for b in range(len(n))]


def gm_rollout_begin(ctx: Context, st: State, ro: Rollout):
    _check(lib().gm_rollout_begin(ctx.handle, C.byref(st.struct()), C.byref(ro.struct())), "gm_rollout_begin")


def gm_rollout_step(ctx: Context, st: State, ro: Rollout, k: int, temperature: float, seed: int, step: int):
    _check(lib().gm_rollout_step(ctx.handle, C.byref(st.struct()), C.byref(ro.struct()), k, temperature, seed, step),
           "gm_rollout_step")


def gm_rollout_run(ctx: Context, st: State, ro: Rollout, k: int, temperature: float, seed: int, first_step: int,
                   max_steps: int, check_every: int = 8):
    """Returns (cycles run, rows still running)."""
    steps, running = C.c_int32(0), C.c_int32(0)
    _check(lib().gm_rollout_run(ctx.handle, C.byref(st.struct()), C.byref(ro.struct()), k, temperature, seed, first_step,
                                max_steps, check_every, C.byref(steps), C.byref(running)), "gm_rollout_run")
    return steps.value, running.value


def gm_capture_hidden(ctx: Context, seq_hidden):
    """seq_hidden: bf16 [max_batch, stride, d] on the device, or None to stop capturing."""
    ctx._capture = seq_hidden                                # keeps the buffer alive
    _check(lib().gm_capture_hidden(ctx.handle, _p(seq_hidden), 0 if seq_hidden is None else seq_hidden.shape[1]),
           "gm_capture_hidden")


def gm_head_prefill(ctx: Context, st: State, seq_hidden, seq_tok, seq_len, max_len: int):
    """seq_hidden bf16 [B, S, d], seq_tok int32 [B, S'], seq_len int32 [B] on the device; max_len a host integer."""
    _check(lib().gm_head_prefill(ctx.handle, C.byref(st.struct()), _p(seq_hidden), seq_hidden.shape[1], _p(seq_tok),
                                 seq_tok.shape[1], _p(seq_len), max_len), "gm_head_prefill")


def gm_reconstruct(ctx: Context, st: State, n_cycles: int, k: int, cycle_seq, rec, seq_tok, scratch_pages, draft_logits,
                   head_states=None):
    """head_states (fp32 [n_cycles, k, d]) given: gm_reconstruct_states, which also returns g_j of every chain."""
    if head_states is None:
        _check(lib().gm_reconstruct(ctx.handle, C.byref(st.struct()), n_cycles, k, _p(cycle_seq), C.byref(rec.struct()),
                                    _p(seq_tok), seq_tok.shape[1], _p(scratch_pages), _p(draft_logits)), "gm_reconstruct")
    else:
        _check(lib().gm_reconstruct_states(ctx.handle, C.byref(st.struct()), n_cycles, k, _p(cycle_seq), C.byref(rec.struct()),
                                           _p(seq_tok), seq_tok.shape[1], _p(scratch_pages), _p(draft_logits),
                                           _p(head_states)), "gm_reconstruct_states")


def gm_head_state_grad(ctx: Context, rows: int, grad_logits, grad_normed, head_states=None, grad_states=None,
                       refresh_weights: bool = False):
    _check(lib().gm_head_state_grad(ctx.handle, rows, _p(grad_logits), _p(head_states), _p(grad_normed), _p(grad_states),
                                    int(refresh_weights)), "gm_head_state_grad")


def gm_head_ffn_backward(ctx: Context, rows: int, x, dg, dx, dw_gate_up, dw_down, dln2, refresh_weights: bool = False):
    _check(lib().gm_head_ffn_backward(ctx.handle, rows, _p(x), _p(dg), _p(dx), _p(dw_gate_up), _p(dw_down), _p(dln2),
                                      int(refresh_weights)), "gm_head_ffn_backward")


def gm_attention_backward(ctx: Context, q, dout, kv_pool, layer: int, page_table, q_count, q_base, batch: int, q_stride: int,
                          dq, dk_pool, dv_pool):
    pool_layers, num_pages = kv_pool.shape[0], kv_pool.shape[2]
    _check(lib().gm_attention_backward(ctx.handle, _p(q), _p(dout), _p(kv_pool), pool_layers, num_pages, layer, _p(page_table),
                                       _p(q_count), _p(q_base), batch, q_stride, _p(dq), _p(dk_pool), _p(dv_pool)),
           "gm_attention_backward")


def gm_head_attn_backward(ctx: Context, x, dxmid, kv_pool, page_table, q_count, q_base, batch: int, q_stride: int, dk_pool, dv_pool,
                          dx, dw_qkv, dw_o, dln1, db_qkv=None, dqk_norm=None, refresh_weights: bool = False):
    _check(lib().gm_head_attn_backward(ctx.handle, _p(x), _p(dxmid), _p(kv_pool), kv_pool.shape[2], _p(page_table), _p(q_count),
                                       _p(q_base), batch, q_stride, _p(dk_pool), _p(dv_pool), _p(dx), _p(dw_qkv), _p(dw_o),
                                       _p(dln1), _p(db_qkv), _p(dqk_norm), int(refresh_weights)), "gm_head_attn_backward")


def head_grad_buffers(cfg, device="cuda") -> dict:
    """fp32 device buffers for every parameter of the head, in the shapes gm_head_update_backward fills."""
    d, f, nqkv = cfg.d_model, cfg.d_ffn, cfg.q_dim + 2 * cfg.kv_dim
    z = lambda *shape: torch.zeros(shape, dtype=torch.float32, device=device)
    g = {"proj": z(d, 2 * d), "enorm": z(d), "hnorm": z(d), "final_norm": z(d), "ln1": z(d), "ln2": z(d), "wqkv": z(nqkv, d),
         "wo": z(d, cfg.q_dim), "w_gate_up": z(2 * f, d), "w_down": z(d, f)}
    if getattr(cfg, "qkv_bias", False):
        g["b_qkv"] = z(nqkv)
    if getattr(cfg, "qk_norm", False):
        g["qk_norm"] = z(2 * cfg.head_dim)
    return g


def gm_head_update_backward(ctx: Context, st: State, n_cycles: int, k: int, cycle_seq, rec, seq_tok, scratch_pages, grad_logits,
                            seq_hidden, seq_len, max_len: int, dk_pool, dv_pool, grads: dict):
    """grads: head_grad_buffers(cfg); overwritten with the gradient of the mean objective."""
    gs = gm_head_grads(*[_p(grads.get(n)) for n in HEAD_GRAD_FIELDS])
    _check(lib().gm_head_update_backward(ctx.handle, C.byref(st.struct()), n_cycles, k, _p(cycle_seq), C.byref(rec.struct()),
                                         _p(seq_tok), seq_tok.shape[1], _p(scratch_pages), _p(grad_logits), _p(seq_hidden),
                                         seq_hidden.shape[1], _p(seq_len), max_len, _p(dk_pool), _p(dv_pool), C.byref(gs)),
           "gm_head_update_backward")


def gm_head_update_step(ctx: Context, st: State, n_cycles: int, k: int, temperature: float, cycle_seq, rec, seq_tok, scratch_pages,
                        seq_hidden, seq_len, max_len: int, step: int, lr: float, mean_loss, beta1: float = 0.9, beta2: float = 0.999,
                        eps: float = 1e-8, weight_decay: float = 0.01):
    _check(lib().gm_head_update_step(ctx.handle, C.byref(st.struct()), n_cycles, k, temperature, _p(cycle_seq), C.byref(rec.struct()),
                                     _p(seq_tok), seq_tok.shape[1], _p(scratch_pages), _p(seq_hidden), seq_hidden.shape[1],
                                     _p(seq_len), max_len, step, lr, beta1, beta2, eps, weight_decay, _p(mean_loss)),
           "gm_head_update_step")


def gm_head_input_backward(ctx: Context, rows: int, tokens, hidden, dz, dhidden, dproj, denorm, dhnorm, refresh_weights: bool = False):
    _check(lib().gm_head_input_backward(ctx.handle, rows, _p(tokens), _p(hidden), _p(dz), _p(dhidden), _p(dproj), _p(denorm),
                                        _p(dhnorm), int(refresh_weights)), "gm_head_input_backward")


def gm_adamw_step(ctx: Context, master, grad, m, v, step: int, lr: float, param_bf16=None, beta1: float = 0.9,
                  beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.01, grad_scale: float = 1.0):
    _check(lib().gm_adamw_step(ctx.handle, master.numel(), _p(master), _p(param_bf16), _p(grad), _p(m), _p(v), step, lr, beta1,
                               beta2, eps, weight_decay, grad_scale), "gm_adamw_step")


def gm_overlap(ctx: Context, n_cycles: int, k: int, temperature: float, draft_logits, rec, alpha, lse=None):
    _check(lib().gm_overlap(ctx.handle, n_cycles, k, temperature, _p(draft_logits), C.byref(rec.struct()), _p(alpha),
                            _p(lse)), "gm_overlap")


def gm_dca_loss(ctx: Context, n_cycles: int, k: int, alpha, accepted, loss, mean):
    _check(lib().gm_dca_loss(ctx.handle, n_cycles, k, _p(alpha), _p(accepted), _p(loss), _p(mean)), "gm_dca_loss")


def gm_dca_grad(ctx: Context, n_cycles: int, k: int, temperature: float, draft_logits, rec, alpha, accepted, grad_logits,
                lse=None):
    _check(lib().gm_dca_grad(ctx.handle, n_cycles, k, temperature, _p(draft_logits), C.byref(rec.struct()), _p(alpha),
                             _p(lse), _p(accepted), _p(grad_logits)), "gm_dca_grad")


def gm_pages_reset(ctx: Context, st: State):
    _check(lib().gm_pages_reset(ctx.handle, C.byref(st.struct())), "gm_pages_reset")


def gm_pages_reserve(ctx: Context, st: State, length, extra: int, finished=None):
    _check(lib().gm_pages_reserve(ctx.handle, C.byref(st.struct()), _p(length), extra, _p(finished)), "gm_pages_reserve")


def gm_pages_release(ctx: Context, st: State, finished):
    _check(lib().gm_pages_release(ctx.handle, C.byref(st.struct()), _p(finished)), "gm_pages_release")


def gm_pages_free_count(ctx: Context):
    a, b = C.c_int32(0), C.c_int32(0)
    _check(lib().gm_pages_free_count(ctx.handle, C.byref(a), C.byref(b)), "gm_pages_free_count")
    return a.value, b.value


def gm_set_top_p(ctx: Context, top_p: float):
    _check(lib().gm_set_top_p(ctx.handle, top_p), "gm_set_top_p")


def gm_nucleus(ctx: Context, logits, rows: int, temperature: float, top_p: float, out, dbg_weight=None):
    _check(lib().gm_nucleus(ctx.handle, _p(logits), rows, temperature, top_p, _p(out), _p(dbg_weight)), "gm_nucleus")


def gm_gemm_swiglu(ctx: Context, x, w, out, M: int, N: int, K: int):
    _check(lib().gm_gemm_swiglu(ctx.handle, _p(x), _p(w), _p(out), M, N, K), "gm_gemm_swiglu")


def gm_gemm(ctx: Context, x, w, out, M: int, N: int, K: int, out_fp32: bool):
    _check(lib().gm_gemm(ctx.handle, _p(x), _p(w), _p(out), M, N, K, 1 if out_fp32 else 0), "gm_gemm")


def gm_attention(ctx: Context, q, kv_pool, layer: int, page_table, q_count, q_base, batch: int, q_stride: int, out):
    """kv_pool: bf16 [pool_layers, 2, num_pages, n_kv, 16, head_dim]."""
    _check(lib().gm_attention(ctx.handle, _p(q), _p(kv_pool), kv_pool.shape[0], kv_pool.shape[2], layer,
                              _p(page_table), _p(q_count), _p(q_base), batch, q_stride, _p(out)), "gm_attention")


def gm_attention_noalloc(n_q_heads: int, n_kv_heads: int, head_dim: int, q, kv_pool, layer: int, page_table, q_count,
                         q_base, batch: int, q_stride: int, out, stream=None):
    """gm_attention without a context and without any allocation inside the library: for callers that are
    handed device buffers and a stream but may not allocate (the scratch is a fixed 16 MiB array inside the
    library).  Raises GmError(GM_ERR_SCRATCH_LIMIT) when the request does not fit that array."""
    stream = torch.cuda.current_stream() if stream is None else stream
    _check(lib().gm_attention_noalloc(n_q_heads, n_kv_heads, head_dim, page_table.shape[1], _p(q), _p(kv_pool),
                                      kv_pool.shape[0], kv_pool.shape[2], layer, _p(page_table), _p(q_count), _p(q_base),
                                      batch, q_stride, _p(out), C.c_void_p(stream.cuda_stream)), "gm_attention_noalloc")


class Record:
    """Device tensors of struct gm_record."""

    def __init__(self, batch: int, k: int, d_model: int, device="cuda"):
        z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=device)
        self.start_hidden = z((batch, d_model), torch.bfloat16)
        self.start_pos = z((batch,), torch.int32)
        self.drafts = z((batch, k), torch.int32)
        self.top_logprob = z((batch, k, 64), torch.bfloat16)
        self.top_index = z((batch, k, 64), torch.int32)
        self.accepted = z((batch,), torch.int32)

    def struct(self) -> gm_record:
        return gm_record(*[getattr(self, n).data_ptr() for n in ("start_hidden", "start_pos", "drafts", "top_logprob",
                                                                  "top_index", "accepted")])


def gm_record_begin(ctx: Context, st: State, rec: Record):
    s, r = st.struct(), rec.struct()
    _check(lib().gm_record_begin(ctx.handle, C.byref(s), C.byref(r)), "gm_record_begin")


def gm_record_end(ctx: Context, batch: int, k: int, temperature: float, target_logits, draft_tok, accept_len, rec: Record):
    r = rec.struct()
    _check(lib().gm_record_end(ctx.handle, batch, k, temperature, _p(target_logits), _p(draft_tok), _p(accept_len),
                               C.byref(r)), "gm_record_end")


def gm_spec_step_rec(ctx: Context, st: State, k: int, temperature: float, seed: int, step: int, accept_len, next_token,
                     draft_tok, rec: Record):
    s, r = st.struct(), rec.struct()
    _check(lib().gm_spec_step_rec(ctx.handle, C.byref(s), k, temperature, seed, step, _p(accept_len), _p(next_token),
                                  _p(draft_tok), C.byref(r)), "gm_spec_step_rec")


def gm_profile(ctx: Context, class_mask: int):
    _check(lib().gm_profile(ctx.handle, class_mask), "gm_profile")


def gm_profile_read(ctx: Context, kernel_class: int):
    ms, n = C.c_double(), C.c_int64()
    _check(lib().gm_profile_read(ctx.handle, kernel_class, C.byref(ms), C.byref(n)), "gm_profile_read")
    return ms.value, n.value


def gm_chain_trace(ctx: Context, enable: bool):
    _check(lib().gm_chain_trace(ctx.handle, 1 if enable else 0), "gm_chain_trace")


def gm_chain_trace_read(ctx: Context):
    """Stamps of the last traced chain launch as an int64 array [CTAs, 64] (nanoseconds; 0 = slot not reached)."""
    import numpy as np
    buf = np.zeros(1024 * 64, dtype=np.uint64)
    n = lib().gm_chain_trace_read(ctx.handle, buf.ctypes.data_as(C.c_void_p), buf.size)
    if n < 0:
        raise GmError(n, "gm_chain_trace_read")
    return buf[:n].astype(np.int64).reshape(-1, 64)


def gm_selftest_wait_expiry(ctx: Context):
    _check(lib().gm_selftest_wait_expiry(ctx.handle), "gm_selftest_wait_expiry")


def gm_launch_count(ctx: Context) -> int:
    return lib().gm_launch_count(ctx.handle)


def gm_last_status(ctx: Context) -> int:
    return lib().gm_last_status(ctx.handle)
