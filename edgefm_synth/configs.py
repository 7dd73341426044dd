"""Shape table of the five decoder workloads (tiny + four Qwen2.5-shaped models)."""
from __future__ import annotations

from dataclasses import dataclass, replace

GLOBAL_SEED = 20260427


@dataclass(frozen=True)
class DecoderConfig:
    name: str
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    qkv_bias: bool
    tied: bool
    cache_len: int          # positions already in the KV cache when decoding starts (T0)
    steps: int              # greedy decode steps of the canonical run
    first_position: int     # RoPE position of the first decoded token (differs from the slot for C2)
    rms_eps: float = 1e-6
    rope_theta: float = 1e6
    w_std: float = 0.02
    kv_std: float = 1.0

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def qkv_rows(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    @property
    def max_context(self) -> int:
        return self.cache_len + self.steps

    def weight_elems(self) -> int:
        """bf16 elements a step reads as weights (one embedding row, not the table)."""
        L, H, F, V = self.n_layers, self.hidden, self.ffn, self.vocab
        R, qd = self.qkv_rows, self.n_q_heads * self.head_dim
        per_layer = R * H + (R if self.qkv_bias else 0) + H * qd + 3 * F * H + 2 * H
        return L * per_layer + H + V * H + H

    def step_bytes(self, cur_len: int) -> int:
        """Algorithmic HBM bytes of one decode step at cache length cur_len:
        weights once, K and V of all attended positions read, one K and one V row written."""
        kv_row = 2 * self.n_layers * self.n_kv_heads * self.head_dim * 2   # K+V, bf16
        return 2 * self.weight_elems() + kv_row * (cur_len + 1) + kv_row

    def mean_step_bytes(self) -> float:
        s = [self.step_bytes(self.cache_len + i) for i in range(self.steps)]
        return sum(s) / len(s)

    def with_(self, **kw) -> "DecoderConfig":
        return replace(self, **kw)


def _c(**kw) -> DecoderConfig:
    return DecoderConfig(**kw)


CONFIGS = {
    # Tiny decoder: one step at slot = position = 128.
    "tiny": _c(name="tiny", n_layers=2, hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=688,
               vocab=4096, qkv_bias=False, tied=False, cache_len=128, steps=1, first_position=128),
    # Qwen2.5-0.5B-shaped; first 256 cache slots stand for a 16x16 vision grid, which advances the
    # multimodal RoPE counter by 16 instead of 256, so the first decode position is 1024 - 240.
    "qwen2.5-0.5b": _c(name="qwen2.5-0.5b", n_layers=24, hidden=896, n_q_heads=14, n_kv_heads=2,
                       head_dim=64, ffn=4864, vocab=151936, qkv_bias=True, tied=True, cache_len=1024,
                       steps=128, first_position=784),
    "qwen2.5-1.5b": _c(name="qwen2.5-1.5b", n_layers=28, hidden=1536, n_q_heads=12, n_kv_heads=2,
                       head_dim=128, ffn=8960, vocab=151936, qkv_bias=True, tied=False, cache_len=2048,
                       steps=128, first_position=2048),
    "qwen2.5-3b": _c(name="qwen2.5-3b", n_layers=36, hidden=2048, n_q_heads=16, n_kv_heads=2,
                     head_dim=128, ffn=11008, vocab=151936, qkv_bias=True, tied=False, cache_len=4096,
                     steps=128, first_position=4096),
    "qwen2.5-7b-32k": _c(name="qwen2.5-7b-32k", n_layers=28, hidden=3584, n_q_heads=28, n_kv_heads=4,
                         head_dim=128, ffn=18944, vocab=152064, qkv_bias=True, tied=False,
                         cache_len=32768, steps=64, first_position=32768),
}
