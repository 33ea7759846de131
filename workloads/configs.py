"""The five synthetic workloads (shapes only; see generators.py for the value recipes).

Shapes follow the Dream-7B and LLaDA-8B attention stacks and the generation settings of the
paper's configuration table (block cache size 256, LLaDA block length 64, speculation block
size 32).  Weights and datasets are not involved: every tensor is random.
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    batch: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    prompt_len: int          # cached rows before generation starts
    gen_len: int             # rows generated after the prompt
    block_len: int           # active block (rows recomputed every step)
    steps_per_block: int     # denoising steps spent on one block (top-k policy)
    vocab: int
    top_k: int               # positions unmasked per step (0: guided accept decides)
    logit_sigma: tuple       # per-position logit scale ~ U(lo, hi); lo == hi: constant
    policy: str              # "topk" or "guided"
    p_agree: float = 0.0     # guided: per-token agreement probability of the AR argmax

    @property
    def capacity(self) -> int:
        return self.prompt_len + self.gen_len

    @property
    def n_blocks(self) -> int:
        return self.gen_len // self.block_len

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


CONFIGS = {
    # 0: tiny single step, full oracle in seconds
    "tiny": WorkloadConfig("tiny", 1, 1, 4, 2, 64, 256, 32, 32, 1, 1024, 4, (3.0, 3.0), "topk"),
    # 1: Dream-7B-shaped stack, batch 1, prompt 1024, 8 blocks of 32, 8 steps per block
    "dream7b": WorkloadConfig("dream7b", 1, 28, 28, 4, 128, 1024, 256, 32, 8, 152064, 4,
                              (1.0, 8.0), "topk"),
    # 2: LLaDA-8B-shaped MHA stack, batch 4, prompt 2048, 8 blocks of 64, 16 steps per block
    "llada8b": WorkloadConfig("llada8b", 4, 32, 32, 32, 128, 2048, 512, 64, 16, 126464, 4,
                              (1.0, 8.0), "topk"),
    # 3: long context, Dream shape, 16384 cached rows, one block of 32
    "longctx": WorkloadConfig("longctx", 1, 28, 28, 4, 128, 16384, 32, 32, 8, 152064, 4,
                              (1.0, 8.0), "topk"),
    # 4: guided diffusion loop, Dream shape, batch 8
    "guided": WorkloadConfig("guided", 8, 28, 28, 4, 128, 1024, 256, 32, 0, 152064, 0,
                             (1.0, 8.0), "guided", 0.8),
}

_ORDER = ["tiny", "dream7b", "llada8b", "longctx", "guided"]


def get_config(key) -> WorkloadConfig:
    """Look a workload up by name or by its position in the list above."""
    if isinstance(key, int):
        return CONFIGS[_ORDER[key]]
    return CONFIGS[key]
