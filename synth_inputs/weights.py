"""Random model weights in a canonical, implementation-neutral form.

Every linear layer, the embedding and the LM head are drawn from a normal
distribution with standard deviation ``cfg.init_std`` (0.02) and rounded to
bf16; every RMSNorm weight is one.  The arrays are returned as float32 numpy
arrays whose values are exactly representable in bf16, so a consumer may
convert them to bf16 or to float64 without loss.  Matrices are stored
``[out_features, in_features]`` (row-major), one array per projection; any
packing (fused QKV, interleaved gate/up) is the consumer's business.
"""
from __future__ import annotations

import numpy as np
import torch

from .configs import ModelConfig


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round a float array to the nearest bf16 value (ties to even); returns float32."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


def _normal(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    return bf16_round(rng.standard_normal(shape, dtype=np.float32) * np.float32(std))


def _layer(rng: np.random.Generator, cfg: ModelConfig) -> dict:
    d, f = cfg.d_model, cfg.d_ffn
    s = cfg.init_std
    lw = {
        "ln1": np.ones(d, np.float32),
        "wq": _normal(rng, (cfg.q_dim, d), s),
        "wk": _normal(rng, (cfg.kv_dim, d), s),
        "wv": _normal(rng, (cfg.kv_dim, d), s),
        "wo": _normal(rng, (d, cfg.q_dim), s),
        "ln2": np.ones(d, np.float32),
        "wg": _normal(rng, (f, d), s),
        "wu": _normal(rng, (f, d), s),
        "wd": _normal(rng, (d, f), s),
    }
    # family extras; the biases are drawn four times wider than the weights so that a consumer
    # that drops them is far outside any parity tolerance
    if cfg.qkv_bias:
        lw["bq"] = _normal(rng, (cfg.q_dim,), 4 * s)
        lw["bk"] = _normal(rng, (cfg.kv_dim,), 4 * s)
        lw["bv"] = _normal(rng, (cfg.kv_dim,), 4 * s)
    if cfg.qk_norm:
        lw["qnorm"] = np.ones(cfg.head_dim, np.float32)
        lw["knorm"] = np.ones(cfg.head_dim, np.float32)
    return lw


def make_weights(cfg: ModelConfig, seed: int = 0, n_layers: int | None = None) -> dict:
    """Target decoder + draft head weights from ``seed``.

    ``n_layers`` overrides ``cfg.n_layers`` (used to materialise a few layers of a
    large shape on the host).
    """
    rng = np.random.Generator(np.random.Philox(seed))
    d = cfg.d_model
    nl = cfg.n_layers if n_layers is None else n_layers
    w = {
        "embed": _normal(rng, (cfg.vocab, d), cfg.init_std),
        "lm_head": _normal(rng, (cfg.vocab, d), cfg.init_std),
        "final_norm": np.ones(d, np.float32),
        "layers": [_layer(rng, cfg) for _ in range(nl)],
    }
    w["head"] = {
        "enorm": np.ones(d, np.float32),
        "hnorm": np.ones(d, np.float32),
        "proj": _normal(rng, (d, 2 * d), cfg.init_std),
        "layer": _layer(rng, cfg),
        "final_norm": np.ones(d, np.float32),
    }
    return w


def perturb_norm_weights(w: dict, seed: int = 123, spread: float = 0.25) -> dict:
    """Replace the all-ones RMSNorm weights by 1 + U(-spread, spread) (bf16 values).

    With all norm weights equal to one a kernel that forgets to apply them would go
    unnoticed; parity tests use this variant.
    """
    rng = np.random.Generator(np.random.Philox(seed))

    def pert(a):
        return bf16_round(1.0 + rng.uniform(-spread, spread, a.shape).astype(np.float32))

    w["final_norm"] = pert(w["final_norm"])
    for lw in w["layers"] + [w["head"]["layer"]]:
        lw["ln1"] = pert(lw["ln1"])
        lw["ln2"] = pert(lw["ln2"])
        for name in ("qnorm", "knorm"):
            if name in lw:
                lw[name] = pert(lw[name])
    for name in ("enorm", "hnorm", "final_norm"):
        w["head"][name] = pert(w["head"][name])
    return w
