"""GPU parity of step 1 with the block power method (the accelerator named for line 5 of Algorithm 1) against the
oracle's power_subspace, through the C ABI: same Gram matrix, same start block, same number of multiplications;
compared on the update matrix W (which depends on the iterated subspace only, not on a basis of it)."""
import numpy as np
import pytest
import torch

import oracle
import squat_inputs as si
import paper_2503_24358_b200 as sq
from parity import stacked_queries, to_torch, alloc_key_outputs, compare_key_unit

pytestmark = pytest.mark.gpu

D = 128
W_TOL = 1e-7          # max-abs on the update matrix where |W| <= 1, the bar of the SVD build


def _w_err(W_gpu, W_ref):
    """max |W_gpu - W_ref| in units of the bar: the float32 rounding of W alone is 2^-24 |W| (6e-8 |W|), so the
    bar scales with |W| above 1."""
    return (np.abs(W_gpu.astype(np.float64) - W_ref) / np.maximum(1.0, np.abs(W_ref))).max()


def _build_power(cfg, X0, iters, n_tokens=None, rank_r=None, g=None, lam=None):
    q = to_torch(si.gen_queries(cfg, n_tokens), cfg.dtype)
    s = sq.Subspace(cfg.n_kv_heads, D)
    r = cfg.rank_r if rank_r is None else rank_r
    sq.squat_build_subspace_power(s, q, r, cfg.lam if lam is None else lam, torch.from_numpy(X0).cuda(), iters,
                                  cfg.block_g if g is None else g)
    W = sq.squat_subspace_export(s, ("W",))["W"]
    return s, W


def _oracle_W(cfg, h, X0, iters, n_tokens=None, rank_r=None, g=None, lam=None):
    Qc = stacked_queries(cfg, h, n_tokens)
    return oracle.build_W_power(Qc, X0, iters, cfg.lam if lam is None else lam, cfg.block_g if g is None else g)


@pytest.mark.parametrize("iters", [0, 1, 2, 4])
def test_power_build_config0_all_heads(iters):
    cfg = si.get_config(0)
    X0 = si.gen_start_block(cfg.seed, D, cfg.rank_r)
    s, W = _build_power(cfg, X0, iters)
    errs = []
    for h in range(cfg.n_kv_heads):
        m = _oracle_W(cfg, h, X0, iters)
        errs.append(_w_err(W[h], m["W"]))
    print("config0 power iters", iters, "max |W_gpu - W_oracle| =", max(errs))
    assert max(errs) <= W_TOL
    assert list(sq.squat_subspace_eig_sweeps(s)) == [cfg.rank_r] * cfg.n_kv_heads      # no direction dropped
    s.close()


def test_power_build_config1_all_heads_with_per_head_start_blocks():
    cfg = si.get_config(1)
    X0 = np.stack([si.gen_start_block(cfg.seed, D, cfg.rank_r, h) for h in range(cfg.n_kv_heads)])
    s, W = _build_power(cfg, X0, 2)
    errs = []
    for h in range(cfg.n_kv_heads):
        m = _oracle_W(cfg, h, X0[h], 2)
        errs.append(_w_err(W[h], m["W"]))
    print("config1 power max |W_gpu - W_oracle| =", max(errs))
    assert max(errs) <= W_TOL
    s.close()


def test_power_build_gqa_stacking_config2_shape():
    cfg = si.get_config(2)
    X0 = si.gen_start_block(cfg.seed, D, cfg.rank_r)
    s, W = _build_power(cfg, X0, 2, n_tokens=1024)
    for h in (0, 3, 7):
        m = _oracle_W(cfg, h, X0, 2, n_tokens=1024)
        assert _w_err(W[h], m["W"]) <= W_TOL
    s.close()


@pytest.mark.parametrize("r,g,lam,iters", [(8, 32, 1e-3, 2), (40, 64, 1e-3, 2), (5, 64, 5e-4, 3), (64, 1, 1e-3, 1),
                                          (33, 1, 1e-3, 2), (1, 1, 1e-3, 2), (60, 32, 5e-4, 2)])
def test_power_build_rank_block_lambda_variants(r, g, lam, iters):
    cfg = si.get_config(1).with_(n_kv_heads=2, n_q_heads=2, n_tokens=512)
    X0 = si.gen_start_block(7, D, r)
    s, W = _build_power(cfg, X0, iters, rank_r=r, g=g, lam=lam)
    for h in range(2):
        m = _oracle_W(cfg, h, X0, iters, rank_r=r, g=g, lam=lam)
        err = _w_err(W[h], m["W"])
        assert err <= W_TOL, (h, err)
    s.close()


def test_power_build_no_update_cases_give_zero_W():
    cfg = si.get_config(1).with_(n_kv_heads=2, n_q_heads=2, n_tokens=256)
    for r, lam in ((0, 1e-3), (16, 0.0)):
        X0 = si.gen_start_block(3, D, max(r, 1))[:, :r].copy()
        s, W = _build_power(cfg, X0, 2, rank_r=r, lam=lam)
        assert np.abs(W).max() == 0.0
        s.close()


def test_power_build_rank_deficient_gram_matches_the_svd_build():
    # 12 prompt tokens: rank(M) = 12 < r = 16; one multiplication already spans the whole row space, the dependent
    # directions are dropped, and P equals the SVD build's exactly (so W agrees with the full method's oracle)
    cfg = si.get_config(1).with_(n_kv_heads=2, n_q_heads=2, n_tokens=12)
    r = 12
    X0 = si.gen_start_block(9, D, 16)
    q = to_torch(si.gen_queries(cfg, 12), cfg.dtype)
    s = sq.Subspace(2, D)
    # rank_r is checked against the token count, so ask for 12 directions from a 12-column block first ...
    sq.squat_build_subspace_power(s, q, r, cfg.lam, torch.from_numpy(X0[:, :r].copy()).cuda(), 1, 1)
    W = sq.squat_subspace_export(s, ("W",))["W"]
    for h in range(2):
        Qc = stacked_queries(cfg, h, 12)
        exact = oracle.build_W(Qc, r, cfg.lam, 1)
        assert _w_err(W[h], exact["W"]) <= W_TOL
    s.close()
    # ... then a Gram matrix of rank 6 inside a 12-column block: the dependent directions are dropped
    cfg6 = cfg.with_(n_tokens=12)
    q6 = q.clone()
    q6[:, 6:, :] = q6[:, :6, :]                     # tokens 6..11 repeat tokens 0..5: rank 6
    s = sq.Subspace(2, D)
    sq.squat_build_subspace_power(s, q6, r, cfg.lam, torch.from_numpy(X0[:, :r].copy()).cuda(), 1, 1)
    W = sq.squat_subspace_export(s, ("W",))["W"]
    kept = list(sq.squat_subspace_eig_sweeps(s))
    # a dependent column's pivot is rounding noise around zero; one that lands above the threshold is kept as a
    # direction outside the row space of M, which changes nothing in P -- the comparison of W below is the check
    assert all(6 <= k <= 12 for k in kept) and min(kept) < 12, kept
    for h in range(2):
        Qc = stacked_queries(cfg6, h, 12)
        Qc[6:] = Qc[:6]
        exact = oracle.build_W(Qc, 6, cfg.lam, 1)
        assert _w_err(W[h], exact["W"]) <= W_TOL
    s.close()


def test_power_build_feeds_the_key_kernel():
    # the write path end to end with the power build: codes against the oracle run with the oracle's power W
    cfg = si.get_config(0)
    X0 = si.gen_start_block(cfg.seed, D, cfg.rank_r)
    s, W = _build_power(cfg, X0, 2)
    k_np = si.gen_keys(cfg)
    k = to_torch(k_np, cfg.dtype)
    B, H, T = k.shape[0], k.shape[1], k.shape[2]
    kc, ks, kz = alloc_key_outputs(B, H, T, D, cfg.bits, cfg.group_size)
    sq.squat_quantize_keys(s, k, cfg.bits, cfg.group_size, kc, ks, kz)
    torch.cuda.synchronize()
    for (b, h) in ((0, 0), (0, cfg.n_kv_heads - 1)):
        m = _oracle_W(cfg, h, X0, 2)
        K64 = si.to_f32(k_np[b, h], cfg.dtype).astype(np.float64)
        un = oracle.unpack(kc[b, h].cpu().numpy(), D, cfg.bits)
        compare_key_unit(K64, m["W"], cfg.group_size, cfg.bits, un, ks[b, h].cpu().numpy(), kz[b, h].cpu().numpy(),
                         None, m["Qhat"])
    assert sq.squat_get_device_status(clear=True) == 0
    s.close()


def test_power_build_from_summed_gram_matrices_of_token_shards_equals_the_power_build_on_all_tokens():
    # the multi-GPU layout of step 1 with the power method: Gram matrices of three token ranges summed (one all-reduce
    # between real ranks), then squat_build_subspace_power_from_gram with the start block every rank holds
    cfg = si.get_config(0)
    H, T = cfg.n_kv_heads, cfg.n_tokens
    q = to_torch(si.gen_queries(cfg), cfg.dtype)
    X0 = torch.from_numpy(si.gen_start_block(cfg.seed, D, cfg.rank_r)).cuda()
    full = sq.Subspace(H, D)
    sq.squat_build_subspace_power(full, q, cfg.rank_r, cfg.lam, X0, 2, cfg.block_g)
    W_full = sq.squat_subspace_export(full, ("W",))["W"]
    total = torch.zeros((H, D, D), dtype=torch.float64, device="cuda")
    part = torch.empty_like(total)
    for r in range(3):
        lo, hi = sq.token_shard(T, r, 3, cfg.group_size)
        if hi > lo:
            sq.squat_gram_static(q[:, lo:hi, :], H, part)
            total += part
    sharded = sq.Subspace(H, D)
    sq.squat_build_subspace_power_from_gram(sharded, total, cfg.rank_r, cfg.lam, X0, 2, cfg.block_g)
    W_sh = sq.squat_subspace_export(sharded, ("W",))["W"]
    assert np.abs(W_sh - W_full).max() <= 1e-7
    helper = sq.Subspace(H, D)
    sq.squat_build_subspace_sharded(helper, q, cfg.rank_r, cfg.lam, cfg.block_g, start_block=X0, power_iters=2)
    W_h = sq.squat_subspace_export(helper, ("W",))["W"]
    assert np.abs(W_h - W_full).max() <= 1e-7
    for h in (0, H - 1):
        m = _oracle_W(cfg, h, X0.cpu().numpy(), 2)
        assert _w_err(W_sh[h], m["W"]) <= W_TOL
    for s in (full, sharded, helper):
        s.close()


@pytest.mark.parametrize("shift", [-40, 40])
def test_power_build_is_invariant_under_a_power_of_two_scaling_of_the_queries(shift):
    # q -> 2^k q makes M -> 4^k M; with lambda -> 4^-k lambda P is unchanged, and since powers of two commute with
    # every rounding the whole computation is: W must come out bit for bit the same (exercises the exponent handling
    # of the reciprocal square roots and the relative drop threshold far from 1)
    cfg = si.get_config(0)
    q = to_torch(si.gen_queries(cfg), cfg.dtype).to(torch.float32)
    X0 = torch.from_numpy(si.gen_start_block(cfg.seed, D, cfg.rank_r)).cuda()
    a = sq.Subspace(cfg.n_kv_heads, D)
    sq.squat_build_subspace_power(a, q, cfg.rank_r, cfg.lam, X0, 2, 1)
    W_a = sq.squat_subspace_export(a, ("W",))["W"]
    b = sq.Subspace(cfg.n_kv_heads, D)
    sq.squat_build_subspace_power(b, q * (2.0 ** shift), cfg.rank_r, cfg.lam * 4.0 ** (-shift), X0, 2, 1)
    W_b = sq.squat_subspace_export(b, ("W",))["W"]
    assert np.array_equal(W_a, W_b)
    assert list(sq.squat_subspace_eig_sweeps(b)) == [cfg.rank_r] * cfg.n_kv_heads
    a.close()
    b.close()
