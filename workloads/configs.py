"""Shapes of the five benchmark workloads and of the small parity cases.

The shapes stand in for a Llama-2-7B layer (hidden 4096, 32 heads x 128) decoding
conversations of 0.5k-4k tokens, which is what the paper evaluates on (Section 3.1,
Appendix A dataset statistics, Appendix B controller sizes). Where the paper gives a
default it is used: cache about twice the top-K (Section 3.1: K=96, m=192), eight
rebuilt tokens per step, controller hidden size 128.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Iterator, Tuple

BASE_SEED = 20240702


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    dtype: str            # "f32" | "bf16": element type of q, k, v, x, out and the cache
    n_layers: int
    batch: int
    n_heads: int
    head_dim: int
    hidden: int           # d: controller input width and projection K-dim
    capacity: int         # C slots per sequence
    topk: int             # K of the in-attention top-K mask
    rebuild_max: int      # R_max; retained budget m = C - R_max
    prompt: int           # tokens loaded in bulk before decoding
    steps: int            # decode steps
    rope_theta: float     # 0 => no rotary embedding
    rebuild_mode: str     # "policy" (top-R by score) | "explicit" (caller flags tokens)
    rebuild_p: float      # per-token, per-step flag probability in explicit mode
    seed: int
    ctrl_hidden: int = 128
    pos_scale: float = 4096.0
    identity_projection: bool = False   # W_k = W_v = I (needs hidden == n_heads*head_dim)
    per_layer_inputs: bool = False      # every layer has its own RMS-normalised input rows
    ctrl_no_recurrence: bool = False    # controller ablation without the GRU's memory: every token sees a zero state
    score_from_attention: bool = False  # tokens ranked by cumulative attention weight instead of the controller's score
    ctrl_weight_std: float = 0.02         # standard deviation of the random-init controller parameters
    ctrl_relative_position: bool = False  # controller re-scores every token at every step by its distance to the current one
    q_scale: float = 1.0                # factor on the queries: > 1 gives the peaked, long-tailed softmax of real attention

    @property
    def retained_max(self) -> int:
        return self.capacity - self.rebuild_max

    @property
    def max_tokens(self) -> int:
        return self.prompt + self.steps

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def scaled(self, **kw) -> "WorkloadConfig":
        return replace(self, **kw)


def _llama_layer(name: str, k: int, **kw) -> WorkloadConfig:
    base = dict(dtype="bf16", n_layers=1, n_heads=32, head_dim=128, hidden=4096,
                rope_theta=1.0e4, seed=BASE_SEED + k)
    base.update(kw)
    return WorkloadConfig(name=name, **base)


CONFIGS: Dict[int, WorkloadConfig] = {
    # fp32 correctness case: q, k, v i.i.d. N(0,1) (identity projection), no prompt.
    1: WorkloadConfig(name="cfg1_f32_b1_h8_dh64_c64", dtype="f32", n_layers=1, batch=1, n_heads=8,
                      head_dim=64, hidden=512, capacity=64, topk=64, rebuild_max=8, prompt=0,
                      steps=256, rope_theta=0.0, rebuild_mode="explicit", rebuild_p=0.1,
                      seed=BASE_SEED + 1, identity_projection=True),
    2: _llama_layer("cfg2_llama7b_b16_c256", 2, batch=16, capacity=256, topk=128, rebuild_max=8,
                    prompt=512, steps=512, rebuild_mode="policy", rebuild_p=0.0),
    3: _llama_layer("cfg3_llama7b_b64_c512_rebuild20pct", 3, batch=64, capacity=512, topk=256,
                    rebuild_max=256, prompt=1024, steps=1024, rebuild_mode="explicit",
                    rebuild_p=0.2),
    4: _llama_layer("cfg4_llama7b_L32_b32_c1024", 4, n_layers=32, batch=32, capacity=1024,
                    topk=512, rebuild_max=8, prompt=2048, steps=512, rebuild_mode="policy",
                    rebuild_p=0.0, per_layer_inputs=True),
}


def sweep_points() -> Iterator[Tuple[int, int, WorkloadConfig]]:
    """Capacity x batch sweep: context 4096 = prompt 3840 + 256 steps, K=C/2, R_max=C/4."""
    for cap in (128, 256, 512, 1024, 2048):
        for b in (1, 8, 32, 128, 256):
            yield cap, b, _llama_layer(f"cfg5_sweep_c{cap}_b{b}", 5, batch=b, capacity=cap,
                                       topk=cap // 2, rebuild_max=cap // 4, prompt=3840,
                                       steps=256, rebuild_mode="explicit", rebuild_p=0.1)


def get_config(k: int) -> WorkloadConfig:
    return CONFIGS[k]
