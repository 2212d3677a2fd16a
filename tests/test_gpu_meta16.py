"""GPU parity of the 16-bit-metadata cache (scale and zero-point stored as IEEE binary16): values and dequantize
bit-exact against the oracle's binary32 / binary16 sequence, keys against the float64 oracle under the replay
protocol extended to rounding ties of the metadata (parity.compare_key_unit_meta16).  Through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import squat_inputs as si
import paper_2503_24358_b200 as sq
from parity import compare_key_unit, oracle_mats, to_torch

pytestmark = pytest.mark.gpu

D = 128


def _alloc(B, H, T, bits, G, keys):
    codes = torch.empty((B, H, T, D * bits // 8), dtype=torch.uint8, device="cuda")
    shape = (B, H, T // G, D) if keys else (B, H, T, D // G)
    return codes, torch.empty(shape, dtype=torch.float16, device="cuda"), torch.empty(shape, dtype=torch.float16, device="cuda")


@pytest.mark.parametrize("bits,G,dtype", [(2, 32, "bf16"), (4, 64, "bf16"), (2, 128, "f32"), (4, 32, "f32")])
def test_values_with_16_bit_metadata_are_bit_exact(bits, G, dtype):
    rng = np.random.default_rng(bits * 100 + G)
    B, H, T = 2, 3, 160
    V = (rng.standard_normal((B, H, T, D)) * 2.5 + 0.9).astype(np.float32)
    V[0, 0, 3, :G] = 1.25                                    # a constant group: range 0, codes 0
    V[1, 2, 7, :] += 300.0                                   # a large offset: the rounded zero-point is off by up to 0.125
    V[0, 1, 9, G:2 * G] *= 1e-7                              # a range whose binary16 scale is subnormal or 0
    if dtype == "bf16":
        V = torch.from_numpy(V).to(torch.bfloat16).float().numpy()
    v = torch.from_numpy(V).cuda().to(torch.bfloat16 if dtype == "bf16" else torch.float32)
    codes, scales, zeros = _alloc(B, H, T, bits, G, keys=False)
    sq.squat_get_device_status(clear=True)
    sq.squat_quantize_values(v, bits, G, codes, scales, zeros)
    torch.cuda.synchronize()
    ref = oracle.quant_values_f32(V.reshape(-1, D), G, bits, meta16=True)
    got_codes = oracle.unpack(codes.cpu().numpy().reshape(-1, D * bits // 8), D, bits)
    assert np.array_equal(scales.float().cpu().numpy().reshape(-1, D // G), ref["scale"])
    assert np.array_equal(zeros.float().cpu().numpy().reshape(-1, D // G), ref["zero"])
    assert np.array_equal(got_codes, ref["codes"])
    assert sq.squat_get_device_status(clear=True) & sq.FLAG_ZERO_RANGE
    # dequantize from the 16-bit metadata: fma(code, scale, zero) rounded once to float32
    out = torch.empty((B, H, T, D), dtype=torch.float32, device="cuda")
    sq.squat_dequantize(sq.SQUAT_VALUES, codes, scales, zeros, B, H, T, D, bits, G, out)
    torch.cuda.synchronize()
    want = (ref["codes"].astype(np.float64).reshape(-1, D // G, G) * ref["scale"].astype(np.float64)[..., None]
            + ref["zero"].astype(np.float64)[..., None]).astype(np.float32).reshape(B, H, T, D)
    assert np.array_equal(out.cpu().numpy(), want)
    # and the float32-metadata path of the same library is untouched by the variant
    c32, s32, z32 = codes.clone(), torch.empty(scales.shape, device="cuda"), torch.empty(zeros.shape, device="cuda")
    sq.squat_quantize_values(v, bits, G, c32, s32, z32)
    torch.cuda.synchronize()
    ref32 = oracle.quant_values_f32(V.reshape(-1, D), G, bits)
    assert np.array_equal(s32.cpu().numpy().reshape(-1, D // G), ref32["scale"])
    assert np.array_equal(oracle.unpack(c32.cpu().numpy().reshape(-1, D * bits // 8), D, bits), ref32["codes"])
    sq.squat_get_device_status(clear=True)                  # the constant group set the zero-range flag again: leave none behind


def _run_keys16(cfg, k_np, W32, bits, G):
    B, H, T, d = k_np.shape
    s = sq.Subspace(H, d)
    sq.squat_subspace_import(s, W32)
    k = to_torch(k_np, cfg.dtype)
    codes, scales, zeros = _alloc(B, H, T, bits, G, keys=True)
    sq.squat_quantize_keys(s, k, bits, G, codes, scales, zeros)
    deq = torch.empty((B, H, T, d), dtype=torch.float32, device="cuda")
    sq.squat_dequantize(sq.SQUAT_KEYS, codes, scales, zeros, B, H, T, d, bits, G, deq)
    torch.cuda.synchronize()
    s.close()
    un = oracle.unpack(codes.cpu().numpy().reshape(B * H * T, -1), d, bits).reshape(B, H, T, d)
    return un, scales.float().cpu().numpy(), zeros.float().cpu().numpy(), deq.cpu().numpy()


def _compare(cfg, k_np, W32, mats, bits, G, got, min_raw):
    un, sc, zr, deq = got
    B, H, T, d = k_np.shape
    tot = {"elements": 0, "raw_equal": 0, "ties": 0, "meta_ties": 0}
    for b in range(B):
        for h in range(H):
            K64 = si.to_f32(k_np[b, h], cfg.dtype).astype(np.float64)
            st = compare_key_unit(K64, W32[h].astype(np.float64), G, bits, un[b, h], sc[b, h], zr[b, h], deq[b, h],
                                  mats[h]["Qhat"] if mats else None, meta16=True)
            for key in tot:
                tot[key] += st[key]
    assert tot["raw_equal"] >= min_raw * tot["elements"], tot
    return tot


def test_keys_with_16_bit_metadata_config0_full():
    cfg = si.get_config(0)
    mats = [oracle_mats(cfg, h) for h in range(cfg.n_kv_heads)]
    W32 = np.stack([m["W"] for m in mats]).astype(np.float32)
    k_np = si.gen_keys(cfg)
    got = _run_keys16(cfg, k_np, W32, cfg.bits, cfg.group_size)
    print("config0 16-bit metadata:", _compare(cfg, k_np, W32, mats, cfg.bits, cfg.group_size, got, 0.99))


@pytest.mark.parametrize("bits,G,r,g", [(2, 32, 32, 1), (4, 64, 8, 1), (2, 128, 32, 1), (2, 32, 16, 32)])
def test_keys_with_16_bit_metadata_variants_bf16(bits, G, r, g):
    cfg = si.get_config(1).with_(batch=2, n_kv_heads=3, n_q_heads=3, n_tokens=512)
    mats = [oracle_mats(cfg, h, rank_r=r, g=g) for h in range(3)]
    W32 = np.stack([m["W"] for m in mats]).astype(np.float32)
    k_np = si.gen_keys(cfg)
    got = _run_keys16(cfg, k_np, W32, bits, G)
    print("16-bit metadata:", _compare(cfg, k_np, W32, mats, bits, G, got, 0.99))


def test_keys_with_16_bit_metadata_zero_update_is_round_to_nearest_on_the_stored_grid():
    # W = 0: every (group, channel) independent; the kernel's exact-tie path must reproduce the oracle bit for bit
    cfg = si.get_config(1).with_(batch=1, n_kv_heads=2, n_q_heads=2, n_tokens=256)
    k_np = si.gen_keys(cfg)
    W32 = np.zeros((2, D, D), np.float32)
    un, sc, zr, deq = _run_keys16(cfg, k_np, W32, 2, 32)
    for h in range(2):
        K64 = si.to_f32(k_np[0, h], cfg.dtype).astype(np.float64)
        o = oracle.quant_keys(K64, 32, 2, meta16=True)
        assert np.array_equal(o["scale"], sc[0, h]) and np.array_equal(o["zero"], zr[0, h])
        assert np.array_equal(o["codes"], un[0, h])


def test_keys_with_16_bit_metadata_workload1_four_heads_full_length():
    # 4 heads of the Llama-2-7B-shaped workload at full length (524 288 elements per head): the 99.9 % bar on the raw
    # (pre-replay) fraction, and how many metadata ties the protocol had to resolve
    cfg = si.get_config(1).with_(n_kv_heads=4, n_q_heads=4)
    mats = [oracle_mats(cfg, h) for h in range(4)]
    W32 = np.stack([m["W"] for m in mats]).astype(np.float32)
    k_np = si.gen_keys(cfg)
    got = _run_keys16(cfg, k_np, W32, cfg.bits, cfg.group_size)
    tot = _compare(cfg, k_np, W32, mats, cfg.bits, cfg.group_size, got, 0.999)
    print("workload 1 (4 heads) 16-bit metadata:", tot)
