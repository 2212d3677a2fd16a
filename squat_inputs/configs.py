"""The five synthetic workloads, as concrete shapes and generator parameters.

They stand in for the paper's workloads (prompts of Llama-2-7B / Llama-3.1-8B shaped
attention layers, Appendix "Experimental Setup"): same head counts, head dimension,
sequence lengths, the low-rank structure of prompt queries (Section 3.2) and the
per-channel outliers of keys (Related Work, "KV cache compression").  Hyper-parameters
follow the paper's defaults where the workload is silent: lambda = 1e-3, element-wise
updates (g = 1).
"""
from dataclasses import dataclass, field, replace
from typing import Tuple


@dataclass(frozen=True)
class WorkloadConfig:
    index: int
    name: str
    dtype: str            # "f32" or "bf16": storage type of q, k, v
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_tokens: int         # prompt length (tokens whose queries build the subspace)
    q_rank: int           # rank of the low-rank part of the queries
    q_noise: float        # standard deviation of the additive query noise
    q_shared_basis: bool  # True: the query heads of one KV head share the basis B
    n_outliers: int       # number of outlier key channels
    outlier_scale: float  # their multiplier
    rank_r: int
    bits: int
    group_size: int
    lam: float = 1e-3
    block_g: int = 1
    residual: int = 0         # R: newest tokens kept in full precision by the caller
    decode_windows: int = 0   # config 3: number of R-token windows appended after the prompt
    decode_window_len: int = 0
    seed: int = 0
    sweep: Tuple[Tuple[int, int, int], ...] = field(default_factory=tuple)  # (bits, r, G) points

    @property
    def q_per_kv(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def key_vectors(self) -> int:
        """Key vectors quantized by one pass over the workload."""
        if self.decode_windows:
            return self.batch * self.n_kv_heads * self.decode_windows * self.decode_window_len
        return self.batch * self.n_kv_heads * self.n_tokens

    def with_(self, **kw) -> "WorkloadConfig":
        return replace(self, **kw)


_SWEEP = tuple((b, r, G) for b in (2, 4) for r in (8, 32, 64) for G in (32, 128))

CONFIGS = (
    WorkloadConfig(0, "tiny-f32", "f32", 1, 8, 8, 128, 256, 16, 0.1, False, 4, 10.0,
                   rank_r=8, bits=2, group_size=32, seed=0),
    WorkloadConfig(1, "llama2-7b-layer", "bf16", 1, 32, 32, 128, 4096, 16, 0.1, False, 4, 10.0,
                   rank_r=32, bits=2, group_size=32, residual=128, seed=1),
    WorkloadConfig(2, "llama3-8b-gqa-layer", "bf16", 16, 32, 8, 128, 8192, 24, 0.1, True, 8, 8.0,
                   rank_r=32, bits=2, group_size=32, seed=2),
    WorkloadConfig(3, "decode-append", "bf16", 64, 32, 32, 128, 2048, 16, 0.1, False, 4, 10.0,
                   rank_r=32, bits=2, group_size=32, residual=128,
                   decode_windows=32, decode_window_len=128, seed=3),
    WorkloadConfig(4, "long-context-sweep", "bf16", 4, 32, 32, 128, 32768, 16, 0.1, False, 4, 10.0,
                   rank_r=32, bits=2, group_size=32, seed=4, sweep=_SWEEP),
)


def get_config(index: int) -> WorkloadConfig:
    return CONFIGS[index]
