"""GPU parity at the full sizes of workloads 2, 3 and 4, in the launch configuration bench.py uses, on
sampled (batch, head) units the oracle can afford; plus the host-buffer entry point.  Workloads 0 and 1
are compared in full in test_gpu_keys.py / test_gpu_subspace.py."""
import numpy as np
import pytest
import torch

import oracle
import squat_inputs as si
import paper_2503_24358_b200 as sq
from parity import (alloc_key_outputs, alloc_value_outputs, compare_key_unit, oracle_mats, to_torch)

pytestmark = pytest.mark.gpu

D = 128


def _check_units(cfg, units, k_np, v_np, kc, ks, kz, vc, vs, vz, bits, G, mats_cache, rank_r=None, tok_lo=0, n_tok=None,
                 n_prompt=None):
    """Compares the sampled units; key outputs may sit at token offset tok_lo of a longer cache."""
    T = k_np.shape[2] if n_tok is None else n_tok
    deq = torch.empty((1, 1, T, D), dtype=torch.float32, device="cuda")
    tot = {"elements": 0, "raw_equal": 0, "ties": 0}
    for b, h in units:
        key = (h, rank_r)
        if key not in mats_cache:
            mats_cache[key] = oracle_mats(cfg, h, n_prompt, rank_r=rank_r)
        m = mats_cache[key]
        c_u = kc[b, h, tok_lo:tok_lo + T].contiguous()
        s_u = ks[b, h, tok_lo // G:(tok_lo + T) // G].contiguous()
        z_u = kz[b, h, tok_lo // G:(tok_lo + T) // G].contiguous()
        sq.squat_dequantize(sq.SQUAT_KEYS, c_u, s_u, z_u, 1, 1, T, D, bits, G, deq)
        torch.cuda.synchronize()
        K64 = si.to_f32(k_np[b, h], cfg.dtype).astype(np.float64)
        st = compare_key_unit(K64, m["W"], G, bits, oracle.unpack(c_u.cpu().numpy(), D, bits), s_u.cpu().numpy(),
                              z_u.cpu().numpy(), deq[0, 0].cpu().numpy(), m["Qhat"])
        for k_ in tot:
            tot[k_] += st[k_]
        if v_np is not None:
            ref = oracle.quant_values_f32(si.to_f32(v_np[b, h], cfg.dtype), G, bits)
            assert np.array_equal(vc[b, h, tok_lo:tok_lo + T].cpu().numpy(), oracle.pack(ref["codes"], bits))
            assert np.array_equal(vs[b, h, tok_lo:tok_lo + T].cpu().numpy(), ref["scale"])
            assert np.array_equal(vz[b, h, tok_lo:tok_lo + T].cpu().numpy(), ref["zero"])
    return tot


def test_workload2_gqa_full_size():
    cfg = si.get_config(2)                       # batch 16, 32 q heads on 8 KV heads, 8192 tokens
    B, H, T, bits, G = cfg.batch, cfg.n_kv_heads, cfg.n_tokens, cfg.bits, cfg.group_size
    s = sq.Subspace(H, D)
    sq.squat_build_subspace(s, to_torch(si.gen_queries(cfg), cfg.dtype), cfg.rank_r, cfg.lam, cfg.block_g)
    k_np, v_np = si.gen_keys(cfg), si.gen_values(cfg)
    k, v = to_torch(k_np, cfg.dtype), to_torch(v_np, cfg.dtype)
    kc, ks, kz = alloc_key_outputs(B, H, T, D, bits, G)
    vc, vs, vz = alloc_value_outputs(B, H, T, D, bits, G)
    sq.squat_quantize_keys(s, k, bits, G, kc, ks, kz)
    sq.squat_quantize_values(v, bits, G, vc, vs, vz)
    torch.cuda.synchronize()
    tot = _check_units(cfg, [(0, 0), (7, 3), (15, 7)], k_np, v_np, kc, ks, kz, vc, vs, vz, bits, G, {})
    print("workload 2 sampled units:", tot)
    assert tot["raw_equal"] >= 0.999 * tot["elements"], tot
    assert sq.squat_get_device_status(clear=True) == 0
    s.close()


def test_workload3_decode_append_stream():
    # subspace from the 2048-token prompt, then 32 windows of 128 tokens appended into a 4096-token cache
    cfg = si.get_config(3)
    B, H, bits, G = cfg.batch, cfg.n_kv_heads, cfg.bits, cfg.group_size
    W, NW = cfg.decode_window_len, cfg.decode_windows
    Tc = W * NW
    s = sq.Subspace(H, D)
    sq.squat_build_subspace(s, to_torch(si.gen_queries(cfg), cfg.dtype), cfg.rank_r, cfg.lam, cfg.block_g)
    kc, ks, kz = alloc_key_outputs(B, H, Tc, D, bits, G)
    vc, vs, vz = alloc_value_outputs(B, H, Tc, D, bits, G)
    sampled = {0: None, 13: None, 22: None, 31: None}  # windows whose content is generated and checked
    k = v = None
    for w in range(NW):
        if w in sampled or k is None:
            k_np = si.gen_keys(cfg, n_tokens=W, segment=1 + w)
            v_np = si.gen_values(cfg, n_tokens=W, segment=1 + w)
            k, v = to_torch(k_np, cfg.dtype), to_torch(v_np, cfg.dtype)
            if w in sampled:
                sampled[w] = (k_np, v_np)
        # every window is one call of each quantizer on [64, 32, 128, 128]; the others reuse the last tensors
        sq.squat_quantize_keys(s, k, bits, G, kc[:, :, w * W:], ks[:, :, w * W // G:], kz[:, :, w * W // G:],
                               out_stride_b=H * Tc, out_stride_h=Tc)
        sq.squat_quantize_values(v, bits, G, vc[:, :, w * W:], vs[:, :, w * W:], vz[:, :, w * W:],
                                 out_stride_b=H * Tc, out_stride_h=Tc)
    torch.cuda.synchronize()
    cache, tot_all = {}, {"elements": 0, "raw_equal": 0, "ties": 0}
    for w, (k_np, v_np) in sampled.items():
        # every head once per sampled window, the batch entry moving with head and window: 4 x 32 units of
        # 128 x 128 elements = 2.1 M compared elements
        units = [((7 * h + 5 * w) % B, h) for h in range(H)]
        tot = _check_units(cfg, units, k_np, v_np, kc, ks, kz, vc, vs, vz, bits, G, cache, tok_lo=w * W, n_tok=W)
        for k_ in tot_all:
            tot_all[k_] += tot[k_]
    print("workload 3 sampled windows/units:", tot_all)
    assert tot_all["elements"] >= 2_000_000
    assert tot_all["raw_equal"] >= 0.999 * tot_all["elements"], tot_all
    s.close()


def test_workload4_long_context_sweep():
    # batch 4, 32 heads, 32768 tokens: every (bits, r, G) point of the sweep on the full tensors
    cfg = si.get_config(4)
    B, H, T = cfg.batch, cfg.n_kv_heads, cfg.n_tokens
    q = to_torch(si.gen_queries(cfg), cfg.dtype)
    k_np = si.gen_keys(cfg)
    k = to_torch(k_np, cfg.dtype)
    s = sq.Subspace(H, D)
    cache = {}
    units = [(0, 5), (3, 30)]
    built_r = None
    for bits, r, G in sorted(cfg.sweep, key=lambda p: p[1]):
        if r != built_r:
            sq.squat_build_subspace(s, q, r, cfg.lam, cfg.block_g)
            built_r = r
        kc, ks, kz = alloc_key_outputs(B, H, T, D, bits, G)
        sq.squat_quantize_keys(s, k, bits, G, kc, ks, kz)
        torch.cuda.synchronize()
        tot = _check_units(cfg, units, k_np, None, kc, ks, kz, None, None, None, bits, G, cache, rank_r=r)
        print(f"workload 4 point bits={bits} r={r} G={G}:", tot)
        assert tot["raw_equal"] >= 0.999 * tot["elements"], (bits, r, G, tot)
        del kc, ks, kz
    # values: one pass per (bits, G) on the full tensor, two sampled units each
    del k
    v_np = si.gen_values(cfg)
    v = to_torch(v_np, cfg.dtype)
    for bits, G in sorted({(b, g) for b, _, g in cfg.sweep}):
        vc, vs, vz = alloc_value_outputs(B, H, T, D, bits, G)
        sq.squat_quantize_values(v, bits, G, vc, vs, vz)
        torch.cuda.synchronize()
        for b, h in units:
            ref = oracle.quant_values_f32(si.to_f32(v_np[b, h], cfg.dtype), G, bits)
            assert np.array_equal(vc[b, h].cpu().numpy(), oracle.pack(ref["codes"], bits))
            assert np.array_equal(vs[b, h].cpu().numpy(), ref["scale"]) and np.array_equal(vz[b, h].cpu().numpy(), ref["zero"])
    s.close()


def test_host_buffer_entry_equals_device_calls():
    # squat_write_path_host = H2D copies + build + keys + values + D2H copies: byte-identical results
    for cfg in (si.get_config(0), si.get_config(1).with_(batch=2, n_kv_heads=4, n_q_heads=8, n_tokens=512)):
        B, H, T, bits, G = cfg.batch, cfg.n_kv_heads, cfg.n_tokens, cfg.bits, cfg.group_size
        q_np, k_np, v_np = si.gen_queries(cfg), si.gen_keys(cfg), si.gen_values(cfg)
        s = sq.Subspace(H, D)
        sq.squat_build_subspace(s, to_torch(q_np, cfg.dtype), cfg.rank_r, cfg.lam, cfg.block_g)
        kc, ks, kz = alloc_key_outputs(B, H, T, D, bits, G)
        vc, vs, vz = alloc_value_outputs(B, H, T, D, bits, G)
        sq.squat_quantize_keys(s, to_torch(k_np, cfg.dtype), bits, G, kc, ks, kz)
        sq.squat_quantize_values(to_torch(v_np, cfg.dtype), bits, G, vc, vs, vz)
        torch.cuda.synchronize()
        host_in = [to_torch(a, cfg.dtype, device="cpu").pin_memory() for a in (q_np, k_np, v_np)]
        host_out = [torch.empty_like(t, device="cpu").pin_memory() for t in (kc, ks, kz, vc, vs, vz)]
        tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
        ws = torch.empty(sq.squat_write_path_workspace_bytes(tdt, B, cfg.n_q_heads, H, T, D, bits, G), dtype=torch.uint8,
                         device="cuda")
        s2 = sq.Subspace(H, D)
        sq.squat_write_path_host(s2, *host_in, cfg.rank_r, cfg.lam, cfg.block_g, bits, G, *host_out, ws)
        for dev_t, host_t in zip((kc, ks, kz, vc, vs, vz), host_out):
            assert torch.equal(dev_t.cpu(), host_t)
        with pytest.raises(sq.SquatError):
            sq.squat_write_path_host(s2, *host_in, cfg.rank_r, cfg.lam, cfg.block_g, bits, G, *host_out, ws[:1024])
        s.close()
        s2.close()


def test_host_buffer_entry_variants_equal_device_calls():
    # the same entry with 16-bit metadata and / or step 1 by the block power method: byte-identical to the device calls
    cfg = si.get_config(1).with_(batch=2, n_kv_heads=4, n_q_heads=8, n_tokens=512)
    B, H, T, bits, G = cfg.batch, cfg.n_kv_heads, cfg.n_tokens, cfg.bits, cfg.group_size
    q_np, k_np, v_np = si.gen_queries(cfg), si.gen_keys(cfg), si.gen_values(cfg)
    x0 = torch.from_numpy(si.gen_start_block(cfg.seed, D, cfg.rank_r))
    tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    ws = torch.empty(sq.squat_write_path_workspace_bytes(tdt, B, cfg.n_q_heads, H, T, D, bits, G), dtype=torch.uint8,
                     device="cuda")
    host_in = [to_torch(a, cfg.dtype, device="cpu").pin_memory() for a in (q_np, k_np, v_np)]
    for m16 in (False, True):
        for power in (False, True):
            if not m16 and not power:
                continue                                            # the plain entry: covered above
            s = sq.Subspace(H, D)
            if power:
                sq.squat_build_subspace_power(s, to_torch(q_np, cfg.dtype), cfg.rank_r, cfg.lam, x0.cuda(), 2, cfg.block_g)
            else:
                sq.squat_build_subspace(s, to_torch(q_np, cfg.dtype), cfg.rank_r, cfg.lam, cfg.block_g)
            kc, ks, kz = alloc_key_outputs(B, H, T, D, bits, G)
            vc, vs, vz = alloc_value_outputs(B, H, T, D, bits, G)
            if m16:
                ks, kz, vs, vz = (t.to(torch.float16) for t in (ks, kz, vs, vz))
            sq.squat_quantize_keys(s, to_torch(k_np, cfg.dtype), bits, G, kc, ks, kz)
            sq.squat_quantize_values(to_torch(v_np, cfg.dtype), bits, G, vc, vs, vz)
            torch.cuda.synchronize()
            host_out = [torch.empty_like(t, device="cpu").pin_memory() for t in (kc, ks, kz, vc, vs, vz)]
            s2 = sq.Subspace(H, D)
            sq.squat_write_path_host(s2, *host_in, cfg.rank_r, cfg.lam, cfg.block_g, bits, G, *host_out, ws,
                                     start_block=x0 if power else None, power_iters=2)
            for dev_t, host_t in zip((kc, ks, kz, vc, vs, vz), host_out):
                assert torch.equal(dev_t.cpu(), host_t), (m16, power)
            s.close()
            s2.close()
    sq.squat_get_device_status(clear=True)


def test_append_window_host_equals_device_calls():
    # squat_append_window_host = H2D copies of one decode window + keys + values + D2H copies, with the update matrices
    # the handle already holds (nothing is rebuilt): byte-identical to the device calls, both metadata types
    cfg = si.get_config(3).with_(batch=3, n_kv_heads=4, n_q_heads=4, n_tokens=256)
    B, H, bits, G, W = cfg.batch, cfg.n_kv_heads, cfg.bits, cfg.group_size, 128
    s = sq.Subspace(H, D)
    sq.squat_build_subspace(s, to_torch(si.gen_queries(cfg), cfg.dtype), cfg.rank_r, cfg.lam, cfg.block_g)
    ws = torch.empty(sq.squat_write_path_workspace_bytes(torch.bfloat16, B, H, H, W, D, bits, G), dtype=torch.uint8, device="cuda")
    for seg, m16 in ((1, False), (2, True)):
        k_np, v_np = si.gen_keys(cfg, n_tokens=W, segment=seg), si.gen_values(cfg, n_tokens=W, segment=seg)
        kc, ks, kz = alloc_key_outputs(B, H, W, D, bits, G)
        vc, vs, vz = alloc_value_outputs(B, H, W, D, bits, G)
        if m16:
            ks, kz, vs, vz = (t.to(torch.float16) for t in (ks, kz, vs, vz))
        sq.squat_quantize_keys(s, to_torch(k_np, cfg.dtype), bits, G, kc, ks, kz)
        sq.squat_quantize_values(to_torch(v_np, cfg.dtype), bits, G, vc, vs, vz)
        torch.cuda.synchronize()
        host_in = [to_torch(a, cfg.dtype, device="cpu").pin_memory() for a in (k_np, v_np)]
        host_out = [torch.empty_like(t, device="cpu").pin_memory() for t in (kc, ks, kz, vc, vs, vz)]
        sq.squat_append_window_host(s, *host_in, bits, G, *host_out, ws)
        for dev_t, host_t in zip((kc, ks, kz, vc, vs, vz), host_out):
            assert torch.equal(dev_t.cpu(), host_t), m16
    with pytest.raises(sq.SquatError):
        sq.squat_append_window_host(s, *host_in, bits, G, *host_out, ws[:1024])
    sq.squat_get_device_status(clear=True)
    s.close()


def test_write_path_captures_into_a_cuda_graph_and_replays_identically():
    # no call of the write path allocates, synchronises or touches the host: the whole step records into a CUDA graph
    cfg = si.get_config(0)
    B, H, T, d, bits, G = cfg.batch, cfg.n_kv_heads, cfg.n_tokens, cfg.head_dim, cfg.bits, cfg.group_size
    q, k, v = (to_torch(x, cfg.dtype) for x in (si.gen_queries(cfg), si.gen_keys(cfg), si.gen_values(cfg)))
    s = sq.Subspace(H, d)
    kc, ks, kz = alloc_key_outputs(B, H, T, d, bits, G)
    vc, vs, vz = alloc_value_outputs(B, H, T, d, bits, G)
    kd = torch.empty((B, H, T, d), dtype=torch.float32, device="cuda")

    def step():
        sq.squat_build_subspace(s, q, cfg.rank_r, cfg.lam, cfg.block_g)
        sq.squat_quantize_keys(s, k, bits, G, kc, ks, kz)
        sq.squat_quantize_values(v, bits, G, vc, vs, vz)
        sq.squat_dequantize(sq.SQUAT_KEYS, kc, ks, kz, B, H, T, d, bits, G, kd)

    step()                                              # eager: reference outputs (and one-time set-up outside the capture)
    torch.cuda.synchronize()
    ref = [t.clone() for t in (kc, ks, kz, vc, vs, vz, kd)]
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        step()
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()
    for t in (kc, ks, kz, vc, vs, vz, kd):
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    for got, want in zip((kc, ks, kz, vc, vs, vz, kd), ref):
        assert torch.equal(got, want)
    assert sq.squat_get_device_status(clear=True) & sq.FLAG_DEVICE_TIMEOUT == 0
    s.close()
