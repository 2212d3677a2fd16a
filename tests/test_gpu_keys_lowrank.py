"""GPU parity of the rank-r form of the key quantizer (small ranks, element-wise updates): the subspace is built on
the GPU, squat_quantize_keys then runs the rank-r kernel, and the result is compared with the oracle -- which runs
Algorithm 1's Quant on its own dense update matrix -- under the protocol of parity.py, and with the dense kernel on
the same handle."""
import numpy as np
import pytest
import torch

import oracle
import squat_inputs as si
import paper_2503_24358_b200 as sq
from parity import alloc_key_outputs, compare_key_unit, oracle_mats, to_torch

pytestmark = pytest.mark.gpu

D = 128


def _run(cfg, r, bits, G, m16=False, prefer_dense=False, k_np=None, handle=None):
    B, H, T = cfg.batch, cfg.n_kv_heads, cfg.n_tokens
    s = handle or sq.Subspace(H, D)
    if handle is None:
        sq.squat_build_subspace(s, to_torch(si.gen_queries(cfg), cfg.dtype), r, cfg.lam, 1)
    prepared = sq.squat_subspace_select_key_kernel(s, prefer_dense)
    assert prepared == (r if 1 <= r <= 8 else 0)
    k = to_torch(k_np, cfg.dtype)
    kc, ks, kz = alloc_key_outputs(B, H, T, D, bits, G)
    if m16:
        ks, kz = ks.to(torch.float16), kz.to(torch.float16)
    sq.squat_quantize_keys(s, k, bits, G, kc, ks, kz)
    deq = torch.empty((B, H, T, D), dtype=torch.float32, device="cuda")
    sq.squat_dequantize(sq.SQUAT_KEYS, kc, ks, kz, B, H, T, D, bits, G, deq)
    torch.cuda.synchronize()
    return s, kc, ks, kz, deq


def _compare(cfg, r, bits, G, k_np, kc, ks, kz, deq, m16=False):
    B, H, T = cfg.batch, cfg.n_kv_heads, cfg.n_tokens
    tot = {"elements": 0, "raw_equal": 0, "ties": 0}
    un = oracle.unpack(kc.cpu().numpy().reshape(B * H * T, -1), D, bits).reshape(B, H, T, D)
    for h in range(H):
        m = oracle_mats(cfg, h, rank_r=r)
        for b in range(B):
            st = compare_key_unit(si.to_f32(k_np[b, h], cfg.dtype).astype(np.float64), m["W"], G, bits, un[b, h],
                                  ks[b, h].float().cpu().numpy(), kz[b, h].float().cpu().numpy(), deq[b, h].cpu().numpy(),
                                  m["Qhat"], meta16=m16)
            for key in tot:
                tot[key] += st[key]
    return tot


@pytest.mark.parametrize("r,bits,G,dtype,m16", [
    (8, 2, 32, "bf16", False), (8, 4, 32, "bf16", False), (8, 2, 128, "bf16", False), (8, 4, 128, "bf16", False),
    (5, 2, 64, "bf16", False), (1, 4, 64, "f32", False), (8, 2, 32, "f32", False), (8, 2, 32, "bf16", True),
    (3, 4, 128, "bf16", True),
])
def test_lowrank_keys_match_the_oracle(r, bits, G, dtype, m16):
    # 3 heads x batch 3 x 2048 tokens = 2.36 M elements per case: the 99.9 % bar on the raw identical fraction applies
    base = si.get_config(1 if dtype == "bf16" else 0)
    cfg = base.with_(batch=3, n_kv_heads=3, n_q_heads=3, n_tokens=2048)
    k_np = si.gen_keys(cfg)
    sq.squat_get_device_status(clear=True)
    s, kc, ks, kz, deq = _run(cfg, r, bits, G, m16, k_np=k_np)
    tot = _compare(cfg, r, bits, G, k_np, kc, ks, kz, deq, m16)
    print(f"rank-r kernel r={r} bits={bits} G={G} {dtype} m16={m16}:", tot)
    assert tot["raw_equal"] >= 0.999 * tot["elements"], tot
    # the dense kernel on the same handle computes the same function: equal up to rounding ties and their cascades
    _, kc_d, ks_d, kz_d, _ = _run(cfg, r, bits, G, m16, prefer_dense=True, k_np=k_np, handle=s)
    same = (kc_d == kc).float().mean().item()
    assert same >= 0.998, same
    sq.squat_subspace_select_key_kernel(s, False)
    assert sq.squat_get_device_status(clear=True) & ~sq.FLAG_ZERO_RANGE == 0
    s.close()


def test_lowrank_ragged_spans_and_window_calls():
    # G = 32 with an odd number of groups per head (the warp's second span idles along), several batch entries, and the
    # split of a prompt into window calls written into a larger cache: identical bytes
    cfg = si.get_config(1).with_(batch=3, n_kv_heads=2, n_q_heads=2, n_tokens=160)      # 15 groups per head
    k_np = si.gen_keys(cfg)
    s, kc, ks, kz, deq = _run(cfg, 8, 2, 32, k_np=k_np)
    tot = _compare(cfg, 8, 2, 32, k_np, kc, ks, kz, deq)
    assert tot["ties"] <= 2, tot
    k = to_torch(k_np, cfg.dtype)
    B, H, T, G = 3, 2, 160, 32
    parts = [torch.zeros_like(t) for t in (kc, ks, kz)]
    for lo, hi in ((0, 32), (32, 128), (128, 160)):
        sq.squat_quantize_keys(s, k[:, :, lo:hi], 2, G, parts[0][:, :, lo:], parts[1][:, :, lo // G:], parts[2][:, :, lo // G:],
                               out_stride_b=H * T, out_stride_h=T)
    torch.cuda.synchronize()
    for a, b in zip((kc, ks, kz), parts):
        assert torch.equal(a, b)
    s.close()


def test_lowrank_is_not_used_where_it_does_not_apply():
    cfg = si.get_config(0)
    q = to_torch(si.gen_queries(cfg), cfg.dtype)
    s = sq.Subspace(cfg.n_kv_heads, D)
    for r, g, lam, want in ((8, 1, 1e-3, 8), (9, 1, 1e-3, 0), (8, 32, 1e-3, 0), (8, 1, 0.0, 0), (0, 1, 1e-3, 0)):
        sq.squat_build_subspace(s, q, r, lam, g)
        assert sq.squat_subspace_select_key_kernel(s, False) == want, (r, g, lam)
    sq.squat_build_subspace(s, q, 8, 1e-3, 1)
    sq.squat_subspace_import(s, np.zeros((cfg.n_kv_heads, D, D), np.float32))
    assert sq.squat_subspace_select_key_kernel(s, False) == 0
    s.close()
