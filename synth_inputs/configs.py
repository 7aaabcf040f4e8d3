"""Model and workload shapes of the five benchmark configurations.

Shapes only.  The names follow the usual dense-decoder notation: ``n_layers``
decoder layers of width ``d_model`` with grouped-query attention
(``n_q_heads`` query heads sharing ``n_kv_heads`` key/value heads of size
``head_dim``), a SwiGLU feed-forward of width ``d_ffn`` and a vocabulary of
``vocab`` tokens.  The draft head is one more layer of the same shape.
"""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class ModelConfig:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    # workload
    batch: int
    k: int                      # drafting depth K
    kv_len_min: int
    kv_len_max: int
    length_law: str             # "uniform" | "lognormal" | "prompt"
    page_size: int = 16
    rope_base: float = 1.0e4
    rms_eps: float = 1.0e-6
    temperature: float = 1.0
    init_std: float = 0.02      # standard deviation of every linear / embedding weight
    prompt_len: int = 0         # Tiny only: prompts are prefetched by a real prefill
    qkv_bias: bool = False      # decoder-layer family with a bias on the q/k/v projections
    qk_norm: bool = False       # decoder-layer family with an RMSNorm on every query and key head

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def layer_params(self) -> int:
        d, f = self.d_model, self.d_ffn
        return d * (self.q_dim + 2 * self.kv_dim) + self.q_dim * d + 3 * d * f

    def target_params(self) -> int:
        """Parameters streamed by one verify forward (layers + LM head)."""
        return self.n_layers * self.layer_params() + self.vocab * self.d_model

    def kv_bytes_per_token(self, n_layers: int | None = None) -> int:
        n = self.n_layers if n_layers is None else n_layers
        return n * 2 * self.kv_dim * 2

    def with_(self, **kw) -> "ModelConfig":
        return replace(self, **kw)


CONFIGS = {
    # 2-layer toy model; the only one on which a full step of the oracle runs in seconds.
    "tiny": ModelConfig("tiny", 2, 256, 4, 2, 64, 1024, 4096, batch=4, k=3,
                        kv_len_min=64, kv_len_max=256, length_law="prompt", prompt_len=64),
    # 4B-shaped dense decoder, batch 64, KV lengths uniform 1k..8k.
    "4b": ModelConfig("4b", 36, 2560, 32, 8, 128, 9728, 151936, batch=64, k=3,
                      kv_len_min=1024, kv_len_max=8192, length_law="uniform"),
    # sampler-only: 256 rows x (k+1) positions over the 4B vocabulary (model fields unused).
    "sampler": ModelConfig("sampler", 0, 2560, 32, 8, 128, 9728, 151936, batch=256, k=3,
                           kv_len_min=0, kv_len_max=0, length_law="uniform"),
    # 7B-shaped dense decoder, batch 128, KV lengths uniform 2k..16k.
    "7b": ModelConfig("7b", 36, 4096, 32, 8, 128, 11008, 151680, batch=128, k=3,
                      kv_len_min=2048, kv_len_max=16384, length_law="uniform"),
    # long-tail RL rollout batch on the 4B shape, lognormal lengths (median 4k, max 32k).
    "longtail": ModelConfig("longtail", 36, 2560, 32, 8, 128, 9728, 151936, batch=256, k=3,
                            kv_len_min=256, kv_len_max=32768, length_law="lognormal"),
}


def get_config(name: str) -> ModelConfig:
    return CONFIGS[name]
