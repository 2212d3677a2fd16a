"""GPU parity: the key quantizer, driven with update matrices imported from the oracle
(isolates step 2 from step 1), through the C ABI.  Comparison protocol: see parity.py."""
import numpy as np
import pytest
import torch

import oracle
import squat_inputs as si
import paper_2503_24358_b200 as sq
from parity import (alloc_key_outputs, compare_key_unit, oracle_mats, rtn_per_channel_f32, to_torch)

pytestmark = pytest.mark.gpu

D = 128


def _run_keys(cfg, k_np, W32, bits, G):
    """k_np [B,H,T,d] generator output; W32 [H,d,d] float32.  Returns unpacked codes, scale, zero, deq."""
    B, H, T, d = k_np.shape
    s = sq.Subspace(H, d)
    sq.squat_subspace_import(s, W32)
    k = to_torch(k_np, cfg.dtype)
    codes, scales, zeros = alloc_key_outputs(B, H, T, d, bits, G)
    sq.squat_quantize_keys(s, k, bits, G, codes, scales, zeros)
    deq = torch.empty((B, H, T, d), dtype=torch.float32, device="cuda")
    sq.squat_dequantize(sq.SQUAT_KEYS, codes, scales, zeros, B, H, T, d, bits, G, deq)
    torch.cuda.synchronize()
    s.close()
    un = oracle.unpack(codes.cpu().numpy().reshape(B * H * T, -1), d, bits).reshape(B, H, T, d)
    return un, scales.cpu().numpy(), zeros.cpu().numpy(), deq.cpu().numpy(), codes


def _compare_all_units(cfg, k_np, W32, mats, bits, G, got, min_raw=0.999):
    un, sc, zr, deq, _ = got
    B, H, T, d = k_np.shape
    tot = {"elements": 0, "raw_equal": 0, "ties": 0}
    for b in range(B):
        for h in range(H):
            K64 = si.to_f32(k_np[b, h], cfg.dtype).astype(np.float64)
            st = compare_key_unit(K64, W32[h].astype(np.float64), G, bits, un[b, h], sc[b, h], zr[b, h], deq[b, h],
                                  mats[h]["Qhat"] if mats else None)
            for key in tot:
                tot[key] += st[key]
    assert tot["raw_equal"] >= min_raw * tot["elements"], tot
    return tot


def _oracle_W32(cfg, heads, n_tokens=None, **kw):
    mats = [oracle_mats(cfg, h, n_tokens, **kw) for h in heads]
    return np.stack([m["W"] for m in mats]).astype(np.float32), mats


def test_keys_config0_full():
    cfg = si.get_config(0)
    W32, mats = _oracle_W32(cfg, range(cfg.n_kv_heads))
    k_np = si.gen_keys(cfg)
    got = _run_keys(cfg, k_np, W32, cfg.bits, cfg.group_size)
    _compare_all_units(cfg, k_np, W32, mats, cfg.bits, cfg.group_size, got)


def test_keys_config1_full():
    cfg = si.get_config(1)
    W32, mats = _oracle_W32(cfg, range(cfg.n_kv_heads))
    k_np = si.gen_keys(cfg)
    got = _run_keys(cfg, k_np, W32, cfg.bits, cfg.group_size)
    tot = _compare_all_units(cfg, k_np, W32, mats, cfg.bits, cfg.group_size, got)
    print("config1 imported-W:", tot)


@pytest.mark.parametrize("bits,G,r,g", [(4, 32, 32, 1), (2, 64, 8, 1), (2, 128, 32, 1), (4, 128, 64, 1),
                                        (2, 32, 16, 32), (2, 32, 40, 64), (4, 64, 5, 64)])
def test_keys_variants_bf16(bits, G, r, g):
    # bits x group size x rank x block size g; 3 heads, batch 3, 2048 tokens: 2.36 M elements per variant, enough
    # for the 99.9 % bar on the raw identical fraction to mean something (one tie moves about 400 elements)
    cfg = si.get_config(1).with_(batch=3, n_kv_heads=3, n_q_heads=3, n_tokens=2048)
    W32, mats = _oracle_W32(cfg, range(3), rank_r=r, g=g)
    k_np = si.gen_keys(cfg)
    got = _run_keys(cfg, k_np, W32, bits, G)
    tot = _compare_all_units(cfg, k_np, W32, mats, bits, G, got, min_raw=0.999)
    print(f"variant bits={bits} G={G} r={r} g={g}:", tot)


RAGGED_SHAPES = [
    (32, 160, 1, 2),     # 5 groups per head: the second 128-token tile has one group, its other three warps idle along
    (32, 96, 3, 3),      # 9 groups per head across 3 batch entries: tiles mix batch entries, the last one is ragged
    (64, 192, 1, 2),     # 3 groups of 64: tile 1 holds one team and a spare one
    (128, 128, 5, 1),    # 5 groups of 128 = 5 tiles: two rounds, the second with one tile slot in use
    (32, 32, 1, 5),      # one group per head: every tile ragged, every round a new head
    (32, 160, 4, 40),    # 200 tiles of 40 heads on 148 CTAs: some CTAs' rounds run across a head boundary (two images staged)
    (32, 64, 1, 170),    # 170 one-tile heads: a CTA's two tiles belong to different heads
]


def test_keys_ragged_tiles_and_rounds():
    # the kernel works in tiles of 128 tokens (4 warps) and rounds of up to 4 tiles that may span two heads.
    # Every shape goes through the element-by-element protocol on its own; the shapes are small by nature, so the
    # 99.9 % bar on the raw identical fraction is applied to all of them together (4.9 M elements)
    bits = 2
    pool = {"elements": 0, "raw_equal": 0, "ties": 0}
    for G, T, B, H in RAGGED_SHAPES:
        cfg = si.get_config(1).with_(batch=B, n_kv_heads=H, n_q_heads=H, n_tokens=T)
        W32, mats = _oracle_W32(cfg, range(H), n_tokens=max(T, 256))
        k_np = si.gen_keys(cfg)
        sq.squat_get_device_status(clear=True)
        got = _run_keys(cfg, k_np, W32, bits, G)
        assert not (sq.squat_get_device_status(clear=True) & sq.FLAG_DEVICE_TIMEOUT), (G, T, B, H)
        tot = _compare_all_units(cfg, k_np, W32, mats, bits, G, got, min_raw=0.0)
        for key in pool:
            pool[key] += tot[key]
    print("ragged shapes pooled:", pool)
    assert pool["raw_equal"] >= 0.999 * pool["elements"], pool


def test_keys_zero_update_reduces_to_round_to_nearest():
    # r = 0 / lambda = 0: W = 0 and the kernel must reproduce plain per-channel round-to-nearest
    # (Section 3.3).  Scales and zeros are bit-exact against the binary32 computation; codes may differ
    # from it only at rounding ties (the kernel multiplies by a 1-ulp reciprocal), which the replay
    # protocol checks element by element against the fp64 oracle.
    for cfg in (si.get_config(0), si.get_config(1).with_(n_kv_heads=4, n_q_heads=4, n_tokens=1024)):
        k_np = si.gen_keys(cfg)
        B, H, T, d = k_np.shape
        for bits, G in ((2, 32), (4, 64), (2, 128)):
            W0 = np.zeros((H, d, d), np.float32)
            got = _run_keys(cfg, k_np, W0, bits, G)
            un, sc, zr, deq, _ = got
            _compare_all_units(cfg, k_np, W0, None, bits, G, got, min_raw=0.999)
            for h in range(H):
                c, s, z = rtn_per_channel_f32(si.to_f32(k_np[0, h], cfg.dtype), G, bits)
                assert np.array_equal(sc[0, h].view(np.uint32), s.view(np.uint32))
                assert np.array_equal(zr[0, h].view(np.uint32), z.view(np.uint32))
                assert (un[0, h] != c).mean() < 5e-3      # coarse bf16 data has many exact ties at 4 bits


def test_keys_window_calls_equal_one_call():
    # quantizing a prompt whole or window by window (any split at multiples of G) gives identical bytes,
    # also when the windows are written into a larger cache through the output strides
    cfg = si.get_config(1).with_(batch=2, n_kv_heads=4, n_q_heads=4, n_tokens=512)
    W32, _ = _oracle_W32(cfg, range(4))
    k_np = si.gen_keys(cfg)
    B, H, T, d, bits, G = 2, 4, 512, D, 2, 32
    s = sq.Subspace(H, d)
    sq.squat_subspace_import(s, W32)
    k = to_torch(k_np, cfg.dtype)
    whole = alloc_key_outputs(B, H, T, d, bits, G)
    sq.squat_quantize_keys(s, k, bits, G, *whole)
    parts = [torch.zeros_like(t) for t in whole]
    for lo, hi in ((0, 128), (128, 160), (160, 512)):
        sq.squat_quantize_keys(s, k[:, :, lo:hi], bits, G, parts[0][:, :, lo:], parts[1][:, :, lo // G:],
                               parts[2][:, :, lo // G:], out_stride_b=H * T, out_stride_h=T)
    torch.cuda.synchronize()
    for a, b in zip(whole, parts):
        assert torch.equal(a, b)
    s.close()


def test_keys_constant_channel_and_status_flag():
    cfg = si.get_config(0).with_(n_kv_heads=1, n_q_heads=1, n_tokens=64)
    W32, mats = _oracle_W32(cfg, range(1))
    k_np = si.gen_keys(cfg).copy()
    k_np[..., 0] = 2.5                   # channel 0 is never corrected, so its groups stay constant
    sq.squat_get_device_status(clear=True)
    got = _run_keys(cfg, k_np, W32, 2, 32)
    _compare_all_units(cfg, k_np, W32, mats, 2, 32, got)
    assert got[1][0, 0, 0, 0] == 0.0 and got[2][0, 0, 0, 0] == np.float32(2.5)
    assert sq.squat_get_device_status(clear=True) & sq.FLAG_ZERO_RANGE


def test_keys_shape_errors():
    s = sq.Subspace(4, D)
    k = torch.zeros((1, 4, 48, D), dtype=torch.bfloat16, device="cuda")
    outs = alloc_key_outputs(1, 4, 64, D, 2, 32)
    with pytest.raises(sq.SquatError) as e:
        sq.squat_quantize_keys(s, k, 2, 32, *outs)          # 48 tokens: not a multiple of G
    assert e.value.status == 2
    k8 = torch.zeros((1, 8, 64, D), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sq.SquatError) as e:
        sq.squat_quantize_keys(s, k8, 2, 32, *alloc_key_outputs(1, 8, 64, D, 2, 32))    # heads != handle
    assert e.value.status == 2
    s.close()
