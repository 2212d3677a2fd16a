"""CPU tests of the host logic of the token-sharded subspace build (a prompt whose tokens are spread over ranks):
the shard boundaries, and -- with two gloo ranks -- that the ranks' Gram matrices, summed by one all-reduce, are the
Gram matrix of the whole prompt (Section 3.2: M = Qc^T Qc is a sum over tokens).  The Gram matrices here come from
the oracle; the GPU side of the same flow is tested in test_gpu_subspace.py."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402
import squat_inputs as si  # noqa: E402
from paper_2503_24358_b200.binding import token_shard  # noqa: E402  (pure Python: needs no GPU)


def test_token_shard_partitions_the_prompt_at_group_boundaries():
    for n, world, mult in ((4096, 2, 32), (4096, 8, 32), (8192, 3, 128), (96, 4, 32), (64, 4, 32)):
        cuts = [token_shard(n, r, world, mult) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == n
        for (a, b), (c, d) in zip(cuts, cuts[1:]):
            assert b == c                                     # contiguous, no gap, no overlap
        sizes = [b - a for a, b in cuts]
        assert all(s % mult == 0 and s >= 0 for s in sizes)
        assert max(sizes) - min(sizes) <= mult                # as even as the group size allows
    with pytest.raises(ValueError):
        token_shard(100, 0, 2, 32)
    with pytest.raises(ValueError):
        token_shard(128, 2, 2, 32)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = si.get_config(0)                                # 8 query heads = 8 KV heads, 256 tokens
        lo, hi = token_shard(cfg.n_tokens, rank, world, cfg.group_size)
        grams = []
        for h in range(2):                                    # two heads are enough for the host logic
            Q = si.to_f32(si.gen_queries_head(cfg, h, cfg.n_tokens), cfg.dtype).astype(np.float64)
            grams.append(oracle.gram(Q[lo:hi]) if hi > lo else np.zeros((cfg.head_dim, cfg.head_dim)))
        g = torch.from_numpy(np.stack(grams))
        dist.all_reduce(g, op=dist.ReduceOp.SUM)              # the path's one exchange step
        out[rank] = g.numpy().copy()
        # step 1 by the block power method on the summed matrices: every rank draws the same start block from the
        # workload's seed, so every rank ends with the same update matrix
        X0 = si.gen_start_block(cfg.seed, cfg.head_dim, cfg.rank_r)
        Qhat, _, _ = oracle.power_subspace(g[0].numpy(), X0, 2)
        out[("W", rank)] = oracle.update_matrices(Qhat, cfg.head_dim, cfg.lam)["W"]
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_gram_matrices_of_token_shards_add_up_gloo_world_size_2():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29621, out), nprocs=2, join=True)
    cfg = si.get_config(0)
    assert np.array_equal(out[0], out[1])                     # every rank ends with the same sum
    for h in range(2):
        Q = si.to_f32(si.gen_queries_head(cfg, h, cfg.n_tokens), cfg.dtype).astype(np.float64)
        full = oracle.gram(Q)
        assert np.abs(out[0][h] - full).max() <= 1e-12 * np.abs(full).max()
    # the power build on the all-reduced matrices: identical on both ranks, and equal to the single-process build
    assert np.array_equal(out[("W", 0)], out[("W", 1)])
    Q = si.to_f32(si.gen_queries_head(cfg, 0, cfg.n_tokens), cfg.dtype).astype(np.float64)
    ref = oracle.build_W_power(Q, si.gen_start_block(cfg.seed, cfg.head_dim, cfg.rank_r), 2, cfg.lam)
    assert np.abs(out[("W", 0)] - ref["W"]).max() <= 1e-9
