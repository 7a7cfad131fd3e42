"""Decoder shapes used by the tests and the benchmark.

The paper only says that the target is a Llama / Vicuna class decoder and the
draft a TinyLlama class one (Section V-A); the concrete shapes below are the
synthetic stand-ins for those models.
"""
from dataclasses import dataclass


@dataclass(frozen=True)
class ModelConfig:
    name: str
    n_layers: int
    d_model: int
    n_heads: int       # query heads (Hq)
    n_kv_heads: int    # key/value heads (Hkv); Hq % Hkv == 0
    head_dim: int      # dh
    ffn: int           # SwiGLU inner width (F)
    vocab: int
    eps: float = 1e-6
    rope_base: float = 1e4

    @property
    def q_dim(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def group(self) -> int:
        return self.n_heads // self.n_kv_heads

    def n_params(self) -> int:
        per_layer = (self.d_model * (self.q_dim + 2 * self.kv_dim) + self.q_dim * self.d_model
                     + 3 * self.d_model * self.ffn)
        return self.n_layers * per_layer + 2 * self.vocab * self.d_model


CONFIGS = {
    # 2-layer MHA decoder the oracle finishes in well under a second.
    "tiny": ModelConfig("tiny", 2, 256, 4, 4, 64, 688, 4096),
    # smallest shape with grouped-query attention and ragged tile edges.
    "micro": ModelConfig("micro", 2, 128, 4, 2, 32, 200, 520),
    # GQA with the 7B head geometry (dh 128, group 4) at a size the oracle runs in seconds.
    "small": ModelConfig("small", 2, 512, 8, 2, 128, 1408, 8192),
    "1b": ModelConfig("1b", 16, 2048, 32, 8, 64, 8192, 32000),
    "7b": ModelConfig("7b", 32, 4096, 32, 8, 128, 14336, 32000),
    "0.5b": ModelConfig("0.5b", 24, 896, 14, 2, 64, 4864, 32000),
    # 13B-class target (the largest target of Section V-A): multi-head attention, 40 layers.
    "13b": ModelConfig("13b", 40, 5120, 40, 40, 128, 13824, 32000),
}


def get_config(name: str, **overrides) -> ModelConfig:
    cfg = CONFIGS[name]
    if overrides:
        fields = {**cfg.__dict__, **overrides}
        cfg = ModelConfig(**fields)
    return cfg
