"""Table of verify-step workloads.

Shapes follow the target models the paper evaluates (Qwen2.5-VL-7B and
Gemma3-12B, Sec. 4 "Models"), gamma = 5 and T in {0, 1} follow its inference
settings (Sec. 4 "Inference Settings").  The paper's evaluation sets are not
available; context lengths and the image-token share of the prefix are
synthetic stand-ins for a VLM prompt (m projected image features followed by
text tokens, Sec. 2.2).
"""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    batch: int
    gamma: int                 # speculation length; gamma+1 query rows per sequence
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    hidden: int
    vocab: int
    temperature: float         # 0 => greedy verification
    ctx_lo: int                # committed context length L_b drawn uniformly in [ctx_lo, ctx_hi]
    ctx_hi: int
    image_tokens: float        # >=1: absolute count of leading image tokens; <1: fraction of L_b
    draft_noise_std: float     # std of the Gaussian noise added to target logits to form the drafter
    seed: int
    hidden_std: float = 1.0    # std of the hidden states (4.0 gives peaked distributions)
    window: int = 0            # sliding-window attention length (0 = full attention)
    page_size: int = 16

    @property
    def rows(self) -> int:
        return self.gamma + 1

    @property
    def m(self) -> int:
        return self.batch * (self.gamma + 1)


_QWEN = dict(n_q_heads=28, n_kv_heads=4, head_dim=128, hidden=3584, vocab=152064)
_GEMMA = dict(n_q_heads=16, n_kv_heads=8, head_dim=256, hidden=3840, vocab=262144)
_TINY = dict(n_q_heads=4, n_kv_heads=1, head_dim=64, hidden=256, vocab=1024)

CONFIGS: dict[str, VerifyConfig] = {}


def _add(cfg: VerifyConfig) -> None:
    CONFIGS[cfg.name] = cfg


# config 1: tiny, both temperatures, seed 0
_add(VerifyConfig("tiny_t0", 1, 5, **_TINY, temperature=0.0, ctx_lo=256, ctx_hi=256,
                  image_tokens=64, draft_noise_std=1.0, seed=0))
_add(VerifyConfig("tiny_t1", 1, 5, **_TINY, temperature=1.0, ctx_lo=256, ctx_hi=256,
                  image_tokens=64, draft_noise_std=1.0, seed=0))
# config 2: Qwen2.5-VL-7B shape, batch 1, greedy
_add(VerifyConfig("qwen7b_b1_t0", 1, 5, **_QWEN, temperature=0.0, ctx_lo=1280, ctx_hi=1280,
                  image_tokens=1024, draft_noise_std=1.5, seed=2))
# config 3: Qwen2.5-VL-7B shape, batch 16, T = 1
_add(VerifyConfig("qwen7b_b16_t1", 16, 5, **_QWEN, temperature=1.0, ctx_lo=1024, ctx_hi=4096,
                  image_tokens=0.25, draft_noise_std=1.0, seed=3))
# config 4: Gemma3-12B shape, batch 32, T = 1
_add(VerifyConfig("gemma12b_b32_t1", 32, 5, **_GEMMA, temperature=1.0, ctx_lo=2048, ctx_hi=8192,
                  image_tokens=256, draft_noise_std=1.0, seed=4))
# config 5: long-context sweep, Qwen shape, batch 64
for _g in (3, 5, 7):
    for _t in (0, 1):
        _add(VerifyConfig(f"qwen7b_long_g{_g}_t{_t}", 64, _g, **_QWEN, temperature=float(_t),
                          ctx_lo=8192, ctx_hi=32768, image_tokens=4096,
                          draft_noise_std=1.5 if _t == 0 else 1.0, seed=5))

# Supplementary parity inputs (not timed).
# Greedy drafter whose noise is small enough that about half the drafts match
# the target's argmax (the std-1.5 recipe of config 2 accepts only a few percent).
_add(replace(CONFIGS["qwen7b_b1_t0"], name="qwen7b_b1_t0_calibrated", draft_noise_std=0.2, seed=12))
# Peaked distributions: top-token probability ~0.1-0.5, so sampled tokens have
# wide CDF intervals and the decision-margin exemption rarely applies.
_add(VerifyConfig("tiny_peaked_t1", 4, 5, **_TINY, temperature=1.0, ctx_lo=1, ctx_hi=300,
                  image_tokens=0.25, draft_noise_std=1.0, seed=21, hidden_std=8.0))
_add(VerifyConfig("tiny_ragged_t1", 7, 3, **_TINY, temperature=0.7, ctx_lo=0, ctx_hi=97,
                  image_tokens=0.25, draft_noise_std=1.0, seed=22))
_add(VerifyConfig("tiny_ragged_t0", 5, 7, **_TINY, temperature=0.0, ctx_lo=0, ctx_hi=200,
                  image_tokens=0.25, draft_noise_std=0.3, seed=23))
_add(replace(CONFIGS["qwen7b_b16_t1"], name="qwen7b_b16_t1_peaked", hidden_std=5.0, seed=13))


# A local-attention layer of the Gemma3-shaped target (sliding window of 1024 positions).
_add(replace(CONFIGS["gemma12b_b32_t1"], name="gemma12b_b32_t1_local", window=1024))
# Reduced-batch copies of the long-context points, small enough for multi-pass profiler captures.
for _g in (5, 7):
    _add(replace(CONFIGS[f"qwen7b_long_g{_g}_t0"], name=f"qwen7b_long_b16_g{_g}_t0", batch=16))


# The LM-head shapes of the long-context sweep (M = 256 / 384 / 512 rows) with short contexts: the
# acceptance call is the same, the attention part is small enough for multi-pass profiler captures.
for _g in (3, 5, 7):
    _add(replace(CONFIGS[f"qwen7b_long_g{_g}_t0"], name=f"qwen7b_lmhead_g{_g}_t0", ctx_lo=64, ctx_hi=256, image_tokens=0.25))
_add(replace(CONFIGS["qwen7b_long_g5_t1"], name="qwen7b_lmhead_g5_t1", ctx_lo=64, ctx_hi=256, image_tokens=0.25))


def get_config(name: str) -> VerifyConfig:
    if name not in CONFIGS:
        raise KeyError(f"unknown workload {name!r}; known: {sorted(CONFIGS)}")
    return CONFIGS[name]
