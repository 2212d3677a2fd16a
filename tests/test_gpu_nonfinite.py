"""Non-finite inputs: a NaN or an infinity among the keys or values must raise SQUAT_FLAG_NONFINITE in the device
status word, the call must return normally, and every group that holds no such element must come out exactly as
it does without it.  (The group that holds one has no meaningful grid: its codes are unspecified.)  No address,
loop bound or wait in the kernels depends on the data, so these inputs cannot fault or hang them."""
import numpy as np
import pytest
import torch

import squat_inputs as si
import paper_2503_24358_b200 as sq
from parity import alloc_key_outputs, alloc_value_outputs, to_torch

pytestmark = pytest.mark.gpu

D = 128


@pytest.mark.parametrize("bad", [float("nan"), float("inf"), float("-inf")])
@pytest.mark.parametrize("dtype,G", [("bf16", 32), ("f32", 128)])
def test_keys_nonfinite_sets_flag_and_spares_other_groups(bad, dtype, G):
    cfg = si.get_config(1 if dtype == "bf16" else 0).with_(batch=1, n_kv_heads=2, n_q_heads=2, n_tokens=512)
    B, H, T, bits = 1, 2, 512, 2
    s = sq.Subspace(H, D)
    sq.squat_build_subspace(s, to_torch(si.gen_queries(cfg), cfg.dtype), 8, cfg.lam, 1)
    k = to_torch(si.gen_keys(cfg), cfg.dtype)
    clean = alloc_key_outputs(B, H, T, D, bits, G)
    sq.squat_get_device_status(clear=True)
    sq.squat_quantize_keys(s, k, bits, G, *clean)
    assert sq.squat_get_device_status(clear=True) & sq.FLAG_NONFINITE == 0
    tok, ch, head = 3 * G + 5, 40, 1                     # one element in group 3 of head 1
    k2 = k.clone()
    k2[0, head, tok, ch] = bad
    dirty = alloc_key_outputs(B, H, T, D, bits, G)
    sq.squat_quantize_keys(s, k2, bits, G, *dirty)
    torch.cuda.synchronize()
    flags = sq.squat_get_device_status(clear=True)
    assert flags & sq.FLAG_NONFINITE, hex(flags)
    assert flags & sq.FLAG_DEVICE_TIMEOUT == 0
    grp = tok // G
    keep_tok = torch.ones((H, T), dtype=torch.bool, device="cuda")
    keep_tok[head, grp * G:(grp + 1) * G] = False
    keep_grp = torch.ones((H, T // G), dtype=torch.bool, device="cuda")
    keep_grp[head, grp] = False
    assert torch.equal(clean[0][0][keep_tok], dirty[0][0][keep_tok])
    assert torch.equal(clean[1][0][keep_grp], dirty[1][0][keep_grp])
    assert torch.equal(clean[2][0][keep_grp], dirty[2][0][keep_grp])
    # channels before the bad one are quantized before it is ever touched: the same in the bad group too
    words = ch * bits // 8
    assert torch.equal(clean[0][0, head, grp * G:(grp + 1) * G, :words], dirty[0][0, head, grp * G:(grp + 1) * G, :words])
    s.close()


@pytest.mark.parametrize("bad", [float("nan"), float("inf"), float("-inf")])
@pytest.mark.parametrize("dtype,G,m16", [("bf16", 32, False), ("f32", 64, False), ("bf16", 128, True)])
def test_values_nonfinite_sets_flag_and_spares_other_groups(bad, dtype, G, m16):
    cfg = si.get_config(1 if dtype == "bf16" else 0).with_(batch=2, n_kv_heads=2, n_q_heads=2, n_tokens=96)
    B, H, T, bits = 2, 2, 96, 4
    v = to_torch(si.gen_values(cfg), cfg.dtype)

    def outs():
        c, sc, z = alloc_value_outputs(B, H, T, D, bits, G)
        return (c, sc.to(torch.float16), z.to(torch.float16)) if m16 else (c, sc, z)

    clean = outs()
    sq.squat_get_device_status(clear=True)
    sq.squat_quantize_values(v, bits, G, *clean)
    assert sq.squat_get_device_status(clear=True) & sq.FLAG_NONFINITE == 0
    b, h, tok, ch = 1, 0, 17, 70
    v2 = v.clone()
    v2[b, h, tok, ch] = bad
    dirty = outs()
    sq.squat_quantize_values(v2, bits, G, *dirty)
    torch.cuda.synchronize()
    flags = sq.squat_get_device_status(clear=True)
    assert flags & sq.FLAG_NONFINITE, hex(flags)
    q = ch // G
    keep = torch.ones((B, H, T, D // G), dtype=torch.bool, device="cuda")
    keep[b, h, tok, q] = False
    assert torch.equal(clean[1][keep], dirty[1][keep]) and torch.equal(clean[2][keep], dirty[2][keep])
    cb = G * bits // 8                                    # code bytes per group
    cg_clean = clean[0].view(B, H, T, D // G, cb)
    cg_dirty = dirty[0].view(B, H, T, D // G, cb)
    assert torch.equal(cg_clean[keep], cg_dirty[keep])
    assert int(cg_dirty[b, h, tok, q].max()) == 0          # the group with the bad element: codes 0


def test_handle_is_bound_to_its_device_and_exactness_travels_with_the_matrices():
    # the number of leading blocks that take the exact rounding decision is stored on the device by the kernel that
    # packs the update matrices: importing W = 0 after a build (and the other way round) must switch it in stream order
    cfg = si.get_config(0)
    H, T, bits, G = cfg.n_kv_heads, cfg.n_tokens, cfg.bits, cfg.group_size
    k = to_torch(si.gen_keys(cfg), cfg.dtype)
    s = sq.Subspace(H, D)
    a = alloc_key_outputs(1, H, T, D, bits, G)
    sq.squat_quantize_keys(s, k, bits, G, *a)                       # fresh handle: W = 0
    sq.squat_build_subspace(s, to_torch(si.gen_queries(cfg), cfg.dtype), cfg.rank_r, cfg.lam, 1)
    sq.squat_subspace_import(s, np.zeros((H, D, D), np.float32))    # back to W = 0
    b = alloc_key_outputs(1, H, T, D, bits, G)
    sq.squat_quantize_keys(s, k, bits, G, *b)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    s.close()
