"""Seeded synthetic inputs shared by the tests, the benchmark and the oracle checks.

This module holds model shapes, prompts and forcing schedules only -- none of
the method's arithmetic.  Prompts and schedules stand in for the reasoning
benchmarks the paper evaluates on (their items are not reproduced): what is
kept is the structure -- a prompt of a few hundred tokens, outputs of thousands
of tokens, a paragraph delimiter every few dozen tokens, and a reflective
keyword after a fraction of the delimiters.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import numpy as np


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rope_theta: float
    rms_eps: float = 1e-6
    tie_embeddings: int = 1
    qkv_bias: int = 1

    def as_dict(self):
        d = asdict(self)
        d.pop("name")
        return d

    @property
    def n_params_streamed(self) -> int:
        """Weight elements one decode step must read (all layer matrices, biases, gains, LM head)."""
        h, qd, kd, f = self.hidden, self.n_q_heads * self.head_dim, self.n_kv_heads * self.head_dim, self.ffn
        per_layer = (qd + 2 * kd) * h + (qd + 2 * kd) * self.qkv_bias + h * qd + 2 * f * h + h * f + 2 * h
        return self.n_layers * per_layer + h + self.vocab * h

    @property
    def kv_bytes_per_token(self) -> int:
        return 2 * 2 * self.n_layers * self.n_kv_heads * self.head_dim


TINY_S = ModelShape("tiny-S", 2, 256, 4, 2, 64, 688, 1024, 1e4)
TINY_L = ModelShape("tiny-L", 4, 512, 8, 2, 64, 1376, 1024, 1e4)
QWEN_1P5B = ModelShape("1.5B", 28, 1536, 12, 2, 128, 8960, 151936, 1e6, tie_embeddings=1)
QWEN_7B = ModelShape("7B", 28, 3584, 28, 4, 128, 18944, 152064, 1e6, tie_embeddings=0)
QWEN_32B = ModelShape("32B", 64, 5120, 40, 8, 128, 27648, 152064, 1e6, tie_embeddings=0)

DELIMITER_ID = 10
KEYWORD_IDS = (11, 12, 13)
N1 = 20  # tokens per Affirmation/Reflection takeover (paper appendix "Hyperparameters of Speculative Thinking")


def prompt_ids(seed: int, length: int, vocab: int) -> np.ndarray:
    """Uniform token ids in [0, vocab)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(0, vocab, size=length, dtype=np.int64).astype(np.int32)


def forcing_schedule(seed: int, n_steps: int, *, mean_interval: float = 40.0, keyword_rate: float = 0.3,
                     delimiter_id: int = DELIMITER_ID, keyword_ids=KEYWORD_IDS) -> np.ndarray:
    """force[t] per emission step: the delimiter at steps separated by Geometric(1/mean_interval) gaps
    (support >= 1); with probability keyword_rate the step after a delimiter carries a keyword drawn
    uniformly from keyword_ids; -1 elsewhere (the sampled token stands)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    force = np.full(n_steps, -1, dtype=np.int32)
    t = -1
    while True:
        t += int(rng.geometric(1.0 / mean_interval))
        if t >= n_steps:
            break
        force[t] = delimiter_id
        if rng.random() < keyword_rate and t + 1 < n_steps:
            force[t + 1] = int(keyword_ids[int(rng.integers(0, len(keyword_ids)))])
            t += 1
    return force


def full_forcing(seed: int, n_steps: int, vocab: int, **kw) -> np.ndarray:
    """A schedule with every step forced: the delimiter/keyword schedule above, uniform ids elsewhere.
    Routing under such a schedule does not depend on any logit."""
    force = forcing_schedule(seed, n_steps, **kw)
    rng = np.random.Generator(np.random.PCG64(seed + 7919))
    fill = rng.integers(14, vocab, size=n_steps, dtype=np.int64).astype(np.int32)
    return np.where(force >= 0, force, fill).astype(np.int32)


@dataclass(frozen=True)
class Workload:
    name: str
    small: ModelShape
    large: ModelShape | None
    prompt_len: int
    max_new_tokens: int
    mean_interval: float = 40.0
    keyword_rate: float = 0.3
    forced: bool = True
    weight_seed: int = 0
    input_seed: int = 100


CONFIGS = {
    "tiny_pair": Workload("tiny_pair", TINY_S, TINY_L, 32, 128, 8.0, 0.5),
    "qwen1p5b_alone": Workload("qwen1p5b_alone", QWEN_1P5B, None, 256, 2048, forced=False),
    "qwen1p5b_32b": Workload("qwen1p5b_32b", QWEN_1P5B, QWEN_32B, 256, 6000, 40.0, 0.3),
    "qwen7b_32b_long": Workload("qwen7b_32b_long", QWEN_7B, QWEN_32B, 4096, 8192, 40.0, 0.5),
}


def batch_inputs(seed: int, n_seqs: int, vocab: int, *, prompt_range=(64, 512), budget_range=(1024, 8192),
                 mean_interval: float = 40.0, keyword_rate: float = 0.3):
    """The batched workload: n_seqs independent sequences with prompt lengths uniform in prompt_range, token
    budgets uniform in budget_range ("up to 8192" generated tokens; drawn so that the live KV fits beside the
    weights) and one seeded forcing schedule each.  Returns (prompts, budgets, forces) as lists."""
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = rng.integers(prompt_range[0], prompt_range[1] + 1, size=n_seqs)
    budgets = rng.integers(budget_range[0], budget_range[1] + 1, size=n_seqs)
    prompts = [prompt_ids(seed + 1 + i, int(lens[i]), vocab) for i in range(n_seqs)]
    forces = [forcing_schedule(seed + 10_000 + i, 2 * int(budgets[i]), mean_interval=mean_interval,
                               keyword_rate=keyword_rate) for i in range(n_seqs)]
    return prompts, [int(b) for b in budgets], forces


def workload_inputs(w: Workload):
    vshared = w.small.vocab if w.large is None else min(w.small.vocab, w.large.vocab)
    prompt = prompt_ids(w.input_seed, w.prompt_len, vshared)
    force = forcing_schedule(w.input_seed + 1, 2 * w.max_new_tokens, mean_interval=w.mean_interval,
                             keyword_rate=w.keyword_rate) if w.forced else None
    return prompt, force
