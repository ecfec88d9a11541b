"""Model and workload shapes used by the tests and the benchmark.

The shapes are the Vicuna/Llama dimensions the paper evaluates on (Section 4.1:
Vicuna 7B / 13B / 33B, K = 4 drafting heads; Appendix A.1: a depth-4 tree of 64
nodes including the root) plus a tiny model that a CPU finishes in seconds.
Only shapes live here; no arithmetic of the method.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Tuple


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    dtype: str            # "fp32" or "bf16": storage type of weights and KV cache
    K: int = 4            # drafting heads (Section 3.2)
    n_sal: int = 2        # staged adaptation layers (Section 3.1)
    aeb_layers: int = 1   # self-attention layers in the Auto-embedding Block
    lm_rank: int = 0      # 0: full drafting vocabulary heads; r > 0: each head is B[V, r] . A[r, d] (Appendix A.2.4)
    use_sampled_token: bool = True   # False: the "w/o Sampled-Token" ablation of Section 4.5 (fc: d -> d on the hidden state alone)
    topk: Tuple[int, ...] = (10, 10, 10, 10)   # candidates kept per head
    n_nodes: int = 64     # tree nodes including the root
    prompt_len: int = 512
    steps: int = 128
    rms_eps: float = 1e-6
    rope_theta: float = 10000.0
    max_ctx: int = 0      # 0 = prompt_len + steps*(K+1) + n_nodes, rounded up

    @property
    def ctx_capacity(self) -> int:
        if self.max_ctx:
            return self.max_ctx
        need = self.prompt_len + self.steps * (self.K + 1) + self.n_nodes
        return (need + 127) // 128 * 128

    def with_(self, **kw) -> "ModelShape":
        return replace(self, **kw)


SHAPES = {
    # 2 layers, d=256, 4 heads of 64, SwiGLU 688, vocab 1000; 16-node tree with
    # per-head widths 4,2,2,1; prompt 32; 8 steps; fp32 everywhere.
    "tiny": ModelShape("tiny", 2, 256, 4, 64, 688, 1000, "fp32", topk=(4, 2, 2, 1),
                       n_nodes=16, prompt_len=32, steps=8),
    # same arithmetic path as the large shapes (bf16 storage) but small enough
    # for a CPU to run every step; spans several 128-row weight tiles.
    "small_bf16": ModelShape("small_bf16", 3, 512, 4, 128, 1408, 2048, "bf16",
                             topk=(6, 5, 4, 3), n_nodes=32, prompt_len=48, steps=8),
    "7b": ModelShape("7b", 32, 4096, 32, 128, 11008, 32000, "bf16",
                     n_nodes=64, prompt_len=512, steps=128),
    # 7B widths with two target layers and a 2048-token prompt: a few GB on the device, used for
    # multi-pass profiler captures of single kernels at realistic sizes.
    "7b_l2": ModelShape("7b_l2", 2, 4096, 32, 128, 11008, 32000, "bf16",
                        n_nodes=64, prompt_len=2048, steps=8),
    # 7B shape with the drafting heads factored at rank 256 (Appendix A.2.4)
    "7b_lr256": ModelShape("7b_lr256", 32, 4096, 32, 128, 11008, 32000, "bf16", lm_rank=256,
                           n_nodes=64, prompt_len=512, steps=128),
    "13b": ModelShape("13b", 40, 5120, 40, 128, 13824, 32000, "bf16",
                      n_nodes=64, prompt_len=1024, steps=128),
    "33b": ModelShape("33b", 60, 6656, 52, 128, 17920, 32000, "bf16",
                      n_nodes=64, prompt_len=1024, steps=64),
}


def get_shape(name: str) -> ModelShape:
    return SHAPES[name]
