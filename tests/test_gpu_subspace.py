"""GPU parity: step 1 (Gram matrix, eigen-decomposition, update matrices) against the oracle, and the
whole write path end to end, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import squat_inputs as si
import paper_2503_24358_b200 as sq
from parity import (alloc_key_outputs, alloc_value_outputs, compare_key_unit, oracle_mats, stacked_queries, to_torch)

pytestmark = pytest.mark.gpu

D = 128
W_TOL = 1e-7          # max-abs on the update matrix (its float32 rounding alone is 6e-8 * |W|)


def _build(cfg, n_tokens=None, rank_r=None, g=None, lam=None, want=("W", "gram", "eigval", "eigvec")):
    q = to_torch(si.gen_queries(cfg, n_tokens), cfg.dtype)
    s = sq.Subspace(cfg.n_kv_heads, D)
    sq.squat_build_subspace(s, q, cfg.rank_r if rank_r is None else rank_r, cfg.lam if lam is None else lam,
                            cfg.block_g if g is None else g)
    out = sq.squat_subspace_export(s, want)
    return s, out


def _check_head(cfg, h, out, n_tokens=None, rank_r=None, g=None, lam=None):
    r = cfg.rank_r if rank_r is None else rank_r
    Qc = stacked_queries(cfg, h, n_tokens)
    M = oracle.gram(Qc)
    assert np.abs(out["gram"][h] - M).max() <= 1e-12 * np.abs(M).max()
    m = oracle_mats(cfg, h, n_tokens, rank_r=r, g=g, lam=lam)
    mu, V = m["mu"], m["V"]
    assert np.abs(out["eigval"][h] - mu).max() <= 1e-10 * mu[0]
    # the rank-r part of the Gram matrix (what P is made of) -- not single eigenvectors, whose sign and,
    # for close eigenvalues, direction are not unique
    Mr_gpu = (out["eigvec"][h][:r].T * out["eigval"][h][:r]) @ out["eigvec"][h][:r]
    Mr_ref = (V[:r].T * mu[:r]) @ V[:r]
    assert np.abs(Mr_gpu - Mr_ref).max() <= 1e-7 * mu[0]
    # eigenvectors of non-negligible eigenvalues are orthonormal (a null space has no preferred basis)
    nz = int((out["eigval"][h] > 1e-9 * mu[0]).sum())
    Vg = out["eigvec"][h][:nz]
    assert np.abs(Vg @ Vg.T - np.eye(nz)).max() < 1e-10
    err = np.abs(out["W"][h].astype(np.float64) - m["W"]).max()
    assert err <= W_TOL, err
    return err, m


def test_subspace_config0():
    cfg = si.get_config(0)
    s, out = _build(cfg)
    errs = [_check_head(cfg, h, out)[0] for h in range(cfg.n_kv_heads)]
    print("config0 max |W_gpu - W_oracle| =", max(errs))
    assert sq.squat_get_device_status(clear=True) & sq.FLAG_NO_CONVERGE == 0
    s.close()


def test_subspace_config1_all_heads():
    cfg = si.get_config(1)
    s, out = _build(cfg)
    errs = [_check_head(cfg, h, out)[0] for h in range(cfg.n_kv_heads)]
    print("config1 max |W_gpu - W_oracle| =", max(errs))
    s.close()


def test_subspace_gqa_stacking_config2_shape():
    # 32 query heads on 8 KV heads, shared basis per KV head; 1024 prompt tokens keep the oracle quick
    cfg = si.get_config(2)
    s, out = _build(cfg, n_tokens=1024)
    for h in (0, 3, 7):
        _check_head(cfg, h, out, n_tokens=1024)
    s.close()


@pytest.mark.parametrize("r,g,lam", [(0, 1, 1e-3), (8, 32, 1e-3), (40, 64, 1e-3), (5, 64, 5e-4), (128, 1, 1e-3), (32, 1, 0.0), (60, 32, 5e-4)])
def test_subspace_rank_block_lambda_variants(r, g, lam):
    cfg = si.get_config(1).with_(n_kv_heads=2, n_q_heads=2, n_tokens=512)
    s, out = _build(cfg, rank_r=r, g=g, lam=lam)
    for h in range(2):
        _check_head(cfg, h, out, rank_r=r, g=g, lam=lam)
        W = out["W"][h]
        for t in range(D // g):                          # block strictly lower triangular
            assert not W[: (t + 1) * g, t * g:(t + 1) * g].any()
    if r == 0 or lam == 0.0:
        assert not out["W"].any()
    s.close()


def test_subspace_fewer_tokens_than_channels():
    # 48 prompt tokens: the Gram matrix has rank 48 < d; directions beyond carry no weight
    cfg = si.get_config(1).with_(n_kv_heads=2, n_q_heads=2, n_tokens=48)
    s, out = _build(cfg, rank_r=32)
    for h in range(2):
        _check_head(cfg, h, out, rank_r=32)
    assert np.abs(out["eigval"][:, 48:]).max() < 1e-9 * out["eigval"][:, 0].max()
    s.close()


def _build_from_queries(q64, n_kv_heads, rank_r, lam, g=1, dtype=torch.float32):
    """q64 [Hq, T, d] float64 -> (handle, exported matrices); the GPU gets the values rounded to dtype."""
    q = torch.from_numpy(np.ascontiguousarray(q64)).to(dtype).cuda()
    s = sq.Subspace(n_kv_heads, D)
    sq.squat_build_subspace(s, q, rank_r, lam, g)
    return s, sq.squat_subspace_export(s, ("W", "gram", "eigval", "eigvec")), q.double().cpu().numpy()


def test_subspace_zero_queries_give_zero_update():
    # M = 0: every eigenvalue is 0, P = I, nothing is fed back; no NaN may come out of the factorisations
    s, out, _ = _build_from_queries(np.zeros((2, 64, D)), 2, 16, 1e-3)
    assert np.all(out["gram"] == 0.0) and np.abs(out["eigval"]).max() <= 1e-290
    assert np.all(np.isfinite(out["eigvec"])) and np.all(out["W"] == 0.0)
    assert sq.squat_get_device_status(clear=True) & sq.FLAG_NO_CONVERGE == 0
    s.close()


def test_subspace_rank_one_queries_single_head():
    # all query rows are multiples of one direction u: one eigenvalue |a|^2 |u|^2, the rest 0.  With
    # s = lambda mu_0, P_inv = I - s/(1+s) u u^T / |u|^2, whose LDL^T factor the oracle also gives.
    rng = np.random.default_rng(5)
    u = rng.standard_normal(D)
    a = rng.standard_normal(200)
    q64 = np.outer(a, u)[None]                                    # one query head, one KV head
    s, out, q_used = _build_from_queries(q64, 1, 8, 0.05)
    Qc = q_used[0]
    M = oracle.gram(Qc)
    assert np.abs(out["gram"][0] - M).max() <= 1e-12 * np.abs(M).max()
    mu0 = np.trace(M)
    assert abs(out["eigval"][0][0] - mu0) <= 1e-10 * mu0 and np.abs(out["eigval"][0][1:]).max() <= 1e-9 * mu0
    v0 = out["eigvec"][0][0]
    assert abs(abs(v0 @ M @ v0) - mu0) <= 1e-9 * mu0              # first eigenvector spans the direction (float32-rounded u)
    m = oracle.build_W(Qc, 8, 0.05, 1)
    assert np.abs(out["W"][0].astype(np.float64) - m["W"]).max() <= W_TOL
    # closed form of the same thing: P_inv = I - s/(1+s) v v^T, unit lower LDL^T factor L, W = L - I
    sv = 0.05 * mu0
    P_inv = np.eye(D) - sv / (1 + sv) * np.outer(v0, v0)
    Lc = np.linalg.cholesky(P_inv)
    L_unit = Lc / np.diag(Lc)
    assert np.abs(out["W"][0].astype(np.float64) - (L_unit - np.eye(D))).max() <= 2e-7
    s.close()


def test_subspace_many_heads_more_than_one_wave():
    # 40 KV heads = 160 CTAs of the eigensolver on 148 SMs: clusters run in two waves; heads must not mix
    cfg = si.get_config(0).with_(n_kv_heads=40, n_q_heads=40, n_tokens=96)
    s, out = _build(cfg, rank_r=8)
    for h in (0, 17, 36, 37, 39):
        _check_head(cfg, h, out, rank_r=8)
    assert sq.squat_get_device_status(clear=True) & sq.FLAG_NO_CONVERGE == 0
    s.close()


def test_subspace_strided_queries_and_argument_errors():
    cfg = si.get_config(1).with_(n_kv_heads=2, n_q_heads=4, n_tokens=256)
    q_np = si.gen_queries(cfg)
    q_thd = to_torch(np.ascontiguousarray(q_np.transpose(1, 0, 2)), cfg.dtype)     # [T, Hq, d] storage
    q = q_thd.permute(1, 0, 2)
    s = sq.Subspace(2, D)
    sq.squat_build_subspace(s, q, 16, 1e-3)
    a = sq.squat_subspace_export(s, ("W",))["W"]
    sq.squat_build_subspace(s, to_torch(q_np, cfg.dtype), 16, 1e-3)
    b = sq.squat_subspace_export(s, ("W",))["W"]
    assert np.array_equal(a, b)
    for bad in (dict(rank_r=129), dict(lam=-1.0), dict(lam=float("nan")), dict(block_g=3)):
        kw = dict(rank_r=16, lam=1e-3, block_g=1)
        kw.update(bad)
        with pytest.raises(sq.SquatError):
            sq.squat_build_subspace(s, q, kw["rank_r"], kw["lam"], kw["block_g"])
    with pytest.raises(sq.SquatError):
        sq.squat_build_subspace(s, to_torch(q_np[:3], cfg.dtype), 16, 1e-3)       # 3 query heads on 2 KV heads
    s.close()


# ---------------------------------------------------------------------------------- end to end
def _end_to_end(cfg, units, n_tokens=None, bits=None, G=None, rank_r=None, g=None, min_raw=0.999):
    """Build on the GPU from the generated queries, quantize keys and values of the whole batch, then
    compare the given (batch, head) units with the oracle run end to end in fp64."""
    bits = cfg.bits if bits is None else bits
    G = cfg.group_size if G is None else G
    T = cfg.n_tokens if n_tokens is None else n_tokens
    B, H = cfg.batch, cfg.n_kv_heads
    q = to_torch(si.gen_queries(cfg, n_tokens), cfg.dtype)
    s = sq.Subspace(H, D)
    sq.squat_build_subspace(s, q, cfg.rank_r if rank_r is None else rank_r, cfg.lam, cfg.block_g if g is None else g)
    k_np, v_np = si.gen_keys(cfg, n_tokens), si.gen_values(cfg, n_tokens)
    k, v = to_torch(k_np, cfg.dtype), to_torch(v_np, cfg.dtype)
    kc, ks, kz = alloc_key_outputs(B, H, T, D, bits, G)
    vc, vs, vz = alloc_value_outputs(B, H, T, D, bits, G)
    sq.squat_quantize_keys(s, k, bits, G, kc, ks, kz)
    sq.squat_quantize_values(v, bits, G, vc, vs, vz)
    deq = torch.empty((B, H, T, D), dtype=torch.float32, device="cuda")
    sq.squat_dequantize(sq.SQUAT_KEYS, kc, ks, kz, B, H, T, D, bits, G, deq)
    torch.cuda.synchronize()
    tot = {"elements": 0, "raw_equal": 0, "ties": 0}
    for b, h in units:
        m = oracle_mats(cfg, h, n_tokens, rank_r=rank_r, g=g)
        K64 = si.to_f32(k_np[b, h], cfg.dtype).astype(np.float64)
        un = oracle.unpack(kc[b, h].cpu().numpy(), D, bits)
        st = compare_key_unit(K64, m["W"], G, bits, un, ks[b, h].cpu().numpy(), kz[b, h].cpu().numpy(),
                              deq[b, h].cpu().numpy(), m["Qhat"])
        for key in tot:
            tot[key] += st[key]
        ref = oracle.quant_values_f32(si.to_f32(v_np[b, h], cfg.dtype), G, bits)
        assert np.array_equal(vc[b, h].cpu().numpy(), oracle.pack(ref["codes"], bits))
        assert np.array_equal(vs[b, h].cpu().numpy(), ref["scale"]) and np.array_equal(vz[b, h].cpu().numpy(), ref["zero"])
    assert tot["raw_equal"] >= min_raw * tot["elements"], tot
    s.close()
    return tot


def test_end_to_end_config0():
    cfg = si.get_config(0)
    tot = _end_to_end(cfg, [(0, h) for h in range(cfg.n_kv_heads)])
    print("config0 end-to-end:", tot)


def test_end_to_end_config1_full():
    cfg = si.get_config(1)
    tot = _end_to_end(cfg, [(0, h) for h in range(cfg.n_kv_heads)])
    print("config1 end-to-end:", tot)


def test_end_to_end_block_variant():
    cfg = si.get_config(1).with_(batch=2, n_kv_heads=2, n_q_heads=2, n_tokens=512)
    _end_to_end(cfg, [(0, 0), (1, 1)], rank_r=40, g=64, bits=4, G=64, min_raw=0.99)


def test_build_from_summed_gram_matrices_of_token_shards_equals_the_build_on_all_tokens():
    # a prompt spread over ranks: every rank's Gram matrices (squat_gram_static on its tokens), summed, then
    # squat_build_subspace_from_gram -- here the "ranks" are three token ranges on one GPU, one of them empty-handed
    cfg = si.get_config(0)
    H, T, d = cfg.n_kv_heads, cfg.n_tokens, cfg.head_dim
    q = to_torch(si.gen_queries(cfg), cfg.dtype)                       # [Hq, T, d]
    full = sq.Subspace(H, d)
    sq.squat_build_subspace(full, q, cfg.rank_r, cfg.lam, cfg.block_g)
    ex = sq.squat_subspace_export(full, ("W", "gram"))
    W_full, G_full = ex["W"], ex["gram"]
    total = torch.zeros((H, d, d), dtype=torch.float64, device="cuda")
    part = torch.empty_like(total)
    for r in range(3):
        lo, hi = sq.token_shard(T, r, 3, cfg.group_size)
        if hi > lo:
            sq.squat_gram_static(q[:, lo:hi, :], H, part)
            total += part
    assert np.abs(total.cpu().numpy() - G_full).max() <= 1e-12 * np.abs(G_full).max()
    sharded = sq.Subspace(H, d)
    sq.squat_build_subspace_from_gram(sharded, total, cfg.rank_r, cfg.lam, cfg.block_g)
    W_sh = sq.squat_subspace_export(sharded, ("W",))["W"]
    assert np.abs(W_sh - W_full).max() <= 1e-7
    # the helper does the same through torch.distributed when a group is up; without one it is the plain build
    helper = sq.Subspace(H, d)
    sq.squat_build_subspace_sharded(helper, q, cfg.rank_r, cfg.lam, cfg.block_g)
    W_h = sq.squat_subspace_export(helper, ("W",))["W"]
    assert np.abs(W_h - W_full).max() <= 1e-7
    for s in (full, sharded, helper):
        s.close()
