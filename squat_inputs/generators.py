"""Counter-based generators for queries, keys and values of a workload.

Every (tensor, batch, head, segment) unit owns one Philox stream keyed by the workload's
seed, so any single unit can be regenerated on its own (the CPU oracle checks sampled
units of workloads far too large for it to process whole).

Storage types: "f32" arrays are numpy float32; "bf16" arrays are numpy uint16 holding
the bfloat16 bit patterns (round-to-nearest-even from float32).  `bf16_bits_to_f32`
widens them back exactly.
"""
import numpy as np

from .configs import WorkloadConfig

_T_QA, _T_QB, _T_QN, _T_K, _T_V, _T_OUT, _T_START = 1, 2, 3, 4, 5, 6, 7


def _rng(seed: int, tensor: int, a: int = 0, b: int = 0, c: int = 0) -> np.random.Generator:
    k1 = (tensor & 0xFF) | ((a & 0xFFFF) << 8) | ((b & 0xFFFFF) << 24) | ((c & 0xFFFFF) << 44)
    return np.random.Generator(np.random.Philox(key=np.array([seed, k1], dtype=np.uint64)))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even. Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float32, exact."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    """Store float32 data in the workload's storage type."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "f32":
        return x
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    raise ValueError(dtype)


def to_f32(x: np.ndarray, dtype: str) -> np.ndarray:
    return x if dtype == "f32" else bf16_bits_to_f32(x)


def outlier_channels(cfg: WorkloadConfig, head: int) -> np.ndarray:
    """Indices of the outlier key channels of a KV head (fixed over tokens and batch)."""
    g = _rng(cfg.seed, _T_OUT, head)
    return np.sort(g.choice(cfg.head_dim, size=cfg.n_outliers, replace=False))


def gen_keys_unit(cfg: WorkloadConfig, b: int, h: int, n_tokens: int = None, segment: int = 0) -> np.ndarray:
    """Keys of one (batch, KV head): N(0,1), outlier channels scaled. Shape [n_tokens, d]."""
    n = cfg.n_tokens if n_tokens is None else n_tokens
    g = _rng(cfg.seed, _T_K, b, h, segment)
    k = g.standard_normal((n, cfg.head_dim), dtype=np.float32)
    k[:, outlier_channels(cfg, h)] *= np.float32(cfg.outlier_scale)
    return round_to_dtype(k, cfg.dtype)


def gen_values_unit(cfg: WorkloadConfig, b: int, h: int, n_tokens: int = None, segment: int = 0) -> np.ndarray:
    """Values of one (batch, KV head): N(0,1). Shape [n_tokens, d]."""
    n = cfg.n_tokens if n_tokens is None else n_tokens
    g = _rng(cfg.seed, _T_V, b, h, segment)
    return round_to_dtype(g.standard_normal((n, cfg.head_dim), dtype=np.float32), cfg.dtype)


def gen_queries_head(cfg: WorkloadConfig, hq: int, n_tokens: int = None) -> np.ndarray:
    """Prompt queries of query head `hq` of sample 0: A @ B + noise. Shape [n_tokens, d].

    A is [n, q_rank], B is [q_rank, d], all entries N(0,1).  With `q_shared_basis` the
    query heads that feed one KV head share B (so their stack keeps rank q_rank).
    """
    n = cfg.n_tokens if n_tokens is None else n_tokens
    hb = hq // cfg.q_per_kv if cfg.q_shared_basis else hq
    A = _rng(cfg.seed, _T_QA, hq).standard_normal((n, cfg.q_rank), dtype=np.float32)
    B = _rng(cfg.seed, _T_QB, hb).standard_normal((cfg.q_rank, cfg.head_dim), dtype=np.float32)
    noise = _rng(cfg.seed, _T_QN, hq).standard_normal((n, cfg.head_dim), dtype=np.float32)
    q = (A.astype(np.float64) @ B.astype(np.float64) + cfg.q_noise * noise.astype(np.float64))
    return round_to_dtype(q.astype(np.float32), cfg.dtype)


def _alloc(cfg: WorkloadConfig, shape) -> np.ndarray:
    return np.empty(shape, dtype=np.float32 if cfg.dtype == "f32" else np.uint16)


def gen_queries(cfg: WorkloadConfig, n_tokens: int = None) -> np.ndarray:
    """[n_q_heads, n_tokens, d] prompt queries of sample 0."""
    n = cfg.n_tokens if n_tokens is None else n_tokens
    out = _alloc(cfg, (cfg.n_q_heads, n, cfg.head_dim))
    for hq in range(cfg.n_q_heads):
        out[hq] = gen_queries_head(cfg, hq, n)
    return out


def gen_keys(cfg: WorkloadConfig, n_tokens: int = None, segment: int = 0, batch: int = None) -> np.ndarray:
    """[batch, n_kv_heads, n_tokens, d] keys."""
    n = cfg.n_tokens if n_tokens is None else n_tokens
    bt = cfg.batch if batch is None else batch
    out = _alloc(cfg, (bt, cfg.n_kv_heads, n, cfg.head_dim))
    for b in range(bt):
        for h in range(cfg.n_kv_heads):
            out[b, h] = gen_keys_unit(cfg, b, h, n, segment)
    return out


def gen_values(cfg: WorkloadConfig, n_tokens: int = None, segment: int = 0, batch: int = None) -> np.ndarray:
    """[batch, n_kv_heads, n_tokens, d] values."""
    n = cfg.n_tokens if n_tokens is None else n_tokens
    bt = cfg.batch if batch is None else batch
    out = _alloc(cfg, (bt, cfg.n_kv_heads, n, cfg.head_dim))
    for b in range(bt):
        for h in range(cfg.n_kv_heads):
            out[b, h] = gen_values_unit(cfg, b, h, n, segment)
    return out


def gen_start_block(seed: int, d: int, r: int, head: int = 0) -> np.ndarray:
    """Start block [d, r] (float64, standard normal) of a block power iteration: the random numbers that
    method draws, made here so that every implementation is handed the same ones."""
    return _rng(seed, _T_START, head).standard_normal((d, r))
