"""The workload configurations (model shape + context recipe + draft length)."""
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
    tied_lm_head: bool = False
    qkv_bias: bool = False
    rope_theta: float = 1.0e6
    rms_eps: float = 1.0e-6
    # workload
    n_ctx: int = 512            # context tokens prefetched into the KV cache
    chunk: int = 256            # prefill chunk length
    k: int = 8                  # draft length per verify step
    gen: int = 128              # tokens to generate
    ngram_n: int = 3            # longest suffix the drafter tries to match
    ngram_min: int = 1          # shortest suffix match that still yields a draft
    span: int = 16              # planted-repeat span length
    repeat_spans: int = -1      # exact number of copied spans (>=0) ...
    repeat_frac: float = 0.25   # ... or a fraction of all spans (when repeat_spans < 0)
    zipf_s: float = 1.1
    resid_scale: float = 0.5    # Wo / Wd scale relative to an embedding row (see make_weights)
    qk_var: float = 1.0         # variance of the attention scores the random Wq, Wk produce
    seed: int = 0

    @property
    def max_seq(self) -> int:
        # committed context + generated tokens + one verify window of slack
        return self.n_ctx + self.gen + 32

    @property
    def n_qkv(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    def with_(self, **kw) -> "ModelConfig":
        return replace(self, **kw)

    def linear_params(self) -> int:
        d, f = self.d_model, self.d_ffn
        per_layer = self.n_qkv * d + d * self.n_q_heads * self.head_dim + 3 * d * f
        return self.n_layers * per_layer + self.vocab * d

    def kv_bytes_per_token(self) -> int:
        return self.n_layers * 2 * self.n_kv_heads * self.head_dim * 2


CONFIGS = {
    "tiny": ModelConfig("tiny", 2, 256, 4, 4, 64, 1024, 4096, rope_theta=1.0e4,
                        n_ctx=512, chunk=256, k=4, gen=32, ngram_n=3, repeat_spans=8),
    "qwen0.5b": ModelConfig("qwen0.5b", 24, 896, 14, 2, 64, 4864, 151936, tied_lm_head=True,
                            n_ctx=1024, chunk=256, k=8, gen=128),
    "qwen1.5b": ModelConfig("qwen1.5b", 28, 1536, 12, 2, 128, 8960, 151936,
                            n_ctx=2048, chunk=256, k=8, gen=256),
    "llama3b": ModelConfig("llama3b", 28, 3072, 24, 8, 128, 8192, 128256, rope_theta=5.0e5,
                           rms_eps=1.0e-5, n_ctx=4096, chunk=256, k=16, gen=256, repeat_frac=0.30),
    "qwen7b": ModelConfig("qwen7b", 28, 3584, 28, 4, 128, 18944, 152064,
                          n_ctx=8192, chunk=256, k=16, gen=64),
}
# small shapes used by tests only (several tiles, ragged tails, GQA, bias, tied head)
CONFIGS["mini_gqa"] = ModelConfig("mini_gqa", 3, 320, 10, 2, 64, 704, 2000 + 16, tied_lm_head=True,
                                  qkv_bias=True, rope_theta=1.0e6, n_ctx=300, chunk=64, k=8, gen=24,
                                  repeat_frac=0.3)
CONFIGS["mini_hd128"] = ModelConfig("mini_hd128", 2, 384, 6, 2, 128, 640, 3024, rope_theta=5.0e5,
                                    rms_eps=1.0e-5, n_ctx=200, chunk=48, k=16, gen=20, repeat_frac=0.3)


def get_config(name: str) -> ModelConfig:
    return CONFIGS[name]
