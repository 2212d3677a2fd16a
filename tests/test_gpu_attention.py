"""GPU parity: one decode step of attention over the packed cache (squat_decode_attention) against the
oracle (dequantize, append the residual buffer, softmax(q K^T / sqrt(d)) V in float64), through the C ABI.

The caches are made by the ORACLE's quantizers and packer, so the reader is checked independently of the GPU
writer; one test reads a cache written by the GPU write path.  Tolerance: the kernel works in float32 (scores,
exponentials, weighted sums over up to a few thousand tokens): 3e-5 absolute on outputs of order 1 for queries
of unit scale.  A float32 score carries an absolute error proportional to the magnitude of the products it sums,
i.e. to the scale of the query, and the softmax turns an absolute score error into a relative error of the
weights; so for a query whose root-mean-square element is rho > 1 (the raw prompt queries of workload 0: rho
about 4) the bar is 3e-5 * rho."""
import math

import numpy as np
import pytest
import torch

import oracle
import squat_inputs as si
import paper_2503_24358_b200 as sq
from parity import alloc_key_outputs, alloc_value_outputs, to_torch

pytestmark = pytest.mark.gpu

D = 128
ATOL = 3e-5


def _oracle_cache(seed, B, H, T, bits, G, outlier=True):
    """Random keys/values, quantized and packed by the oracle.  Returns device tensors and the unpacked pieces."""
    rng = np.random.default_rng(seed)
    K = rng.standard_normal((B, H, T, D))
    if outlier:
        K[..., 7] *= 8.0
    V = rng.standard_normal((B, H, T, D))
    kc = np.zeros((B, H, T, D * bits // 8), np.uint8)
    vc = np.zeros_like(kc)
    ks = np.zeros((B, H, T // G, D), np.float32)
    kz = np.zeros_like(ks)
    vs = np.zeros((B, H, T, D // G), np.float32)
    vz = np.zeros_like(vs)
    units = {}
    for b in range(B):
        for h in range(H):
            kq = oracle.quant_keys(K[b, h], G, bits)
            vq = oracle.quant_values_f64(V[b, h], G, bits)
            kc[b, h], vc[b, h] = oracle.pack(kq["codes"], bits), oracle.pack(vq["codes"], bits)
            ks[b, h], kz[b, h], vs[b, h], vz[b, h] = kq["scale"], kq["zero"], vq["scale"], vq["zero"]
            units[b, h] = (kq, vq)
    dev = lambda a: torch.from_numpy(a).cuda()
    return (dev(kc), dev(ks), dev(kz), dev(vc), dev(vs), dev(vz)), units


def _run(q, cache, H, T, bits, G, k_res=None, v_res=None, scale=0.0, **kw):
    B, Hq, _ = q.shape
    out = torch.empty((B, Hq, D), dtype=torch.float32, device="cuda")
    ws = torch.empty(sq.squat_decode_attention_workspace_bytes(B, Hq, T), dtype=torch.uint8, device="cuda")
    sq.squat_decode_attention(q, *cache, H, T, bits, G, out, ws, k_res, v_res, scale, **kw)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64)


def _check(out, q_used, units, H, G, k_res=None, v_res=None, T=None):
    B, Hq, _ = q_used.shape
    qpk = Hq // H
    worst = 0.0
    for b in range(B):
        for h in range(H):
            kq, vq = units[b, h]
            n = kq["codes"].shape[0] if T is None else T
            ref = oracle.decode_attention_over_cache(
                q_used[b, h * qpk:(h + 1) * qpk], kq["codes"][:n], kq["scale"][:n // G], kq["zero"][:n // G],
                vq["codes"][:n], vq["scale"][:n], vq["zero"][:n], G,
                None if k_res is None else k_res[b, h], None if v_res is None else v_res[b, h]) if n else \
                oracle.attention_decode(q_used[b, h * qpk:(h + 1) * qpk], k_res[b, h], v_res[b, h])
            rho = max(1.0, float(np.sqrt(np.mean(q_used[b, h * qpk:(h + 1) * qpk] ** 2, axis=-1)).max()))
            err = np.abs(out[b, h * qpk:(h + 1) * qpk] - ref).max() / rho
            worst = max(worst, err)
    assert worst <= ATOL, worst
    return worst


def test_attention_mha_small_f32():
    B, H, T, bits, G = 2, 2, 256, 2, 32
    cache, units = _oracle_cache(0, B, H, T, bits, G)
    q = torch.randn(B, H, D, generator=torch.Generator().manual_seed(1)).cuda()
    out = _run(q, cache, H, T, bits, G)
    print("max err", _check(out, q.double().cpu().numpy(), units, H, G))


@pytest.mark.parametrize("bits,G,qpk,T,R,res_dtype", [
    (2, 32, 4, 2112, 32, torch.bfloat16),        # 3 token chunks, the last one ragged; bf16 residual buffer
    (4, 64, 2, 1088, 128, torch.float32),        # 4-bit codes, two query heads per KV head, full residual buffer
    (2, 128, 1, 1024, 0, torch.float32),         # exactly one chunk, no residual buffer
    (4, 32, 8, 96, 5, torch.float32),            # 8 query heads per KV head: two passes over the cache
    (2, 64, 3, 192, 1, torch.bfloat16),          # a query-head count that is not a power of two
])
def test_attention_variants(bits, G, qpk, T, R, res_dtype):
    B, H = 2, 2
    cache, units = _oracle_cache(10 + bits + G + qpk, B, H, T, bits, G)
    g = torch.Generator().manual_seed(T + R)
    q = torch.randn(B, H * qpk, D, generator=g).to(torch.bfloat16).cuda()
    k_res = v_res = None
    if R:
        k_res = torch.randn(B, H, R, D, generator=g).to(res_dtype).cuda()
        v_res = torch.randn(B, H, R, D, generator=g).to(res_dtype).cuda()
    out = _run(q, cache, H, T, bits, G, k_res, v_res)
    kr = None if k_res is None else k_res.double().cpu().numpy()
    vr = None if v_res is None else v_res.double().cpu().numpy()
    print("max err", _check(out, q.double().cpu().numpy(), units, H, G, kr, vr))


def test_attention_residual_buffer_only_and_prefix_of_a_longer_cache():
    B, H, T, bits, G = 1, 2, 512, 2, 32
    cache, units = _oracle_cache(3, B, H, T, bits, G)
    g = torch.Generator().manual_seed(9)
    q = torch.randn(B, H, D, generator=g).cuda()
    k_res, v_res = torch.randn(B, H, 16, D, generator=g).cuda(), torch.randn(B, H, 16, D, generator=g).cuda()
    kr, vr = k_res.double().cpu().numpy(), v_res.double().cpu().numpy()
    # nothing quantized yet: only the residual buffer
    out = _run(q, cache, H, 0, bits, G, k_res, v_res)
    _check(out, q.double().cpu().numpy(), units, H, G, kr, vr, T=0)
    # the first 192 tokens of the 512-token cache (strides say where the heads start)
    out = _run(q, cache, H, 192, bits, G, k_res, v_res, cache_stride_b=H * T, cache_stride_h=T)
    _check(out, q.double().cpu().numpy(), units, H, G, kr, vr, T=192)


def test_attention_closed_forms_and_scale_argument():
    B, H, T, bits, G = 1, 1, 128, 2, 32
    cache, units = _oracle_cache(4, B, H, T, bits, G)
    kq, vq = units[0, 0]
    Vd = oracle.dequant_values(vq["codes"], vq["scale"], vq["zero"], G)
    # zero query: every weight is 1 / n, the output is the mean of the dequantized values
    out = _run(torch.zeros(1, 1, D).cuda(), cache, H, T, bits, G)
    assert np.abs(out[0, 0] - Vd.mean(axis=0)).max() <= ATOL
    # an explicit scale of 1 / sqrt(d) is the default
    q = torch.randn(1, 1, D, generator=torch.Generator().manual_seed(2)).cuda()
    a, b = _run(q, cache, H, T, bits, G), _run(q, cache, H, T, bits, G, scale=1.0 / math.sqrt(D))
    assert np.array_equal(a, b)
    # twice the scale equals twice the query
    c, d2 = _run(q, cache, H, T, bits, G, scale=2.0 / math.sqrt(D)), _run(2 * q, cache, H, T, bits, G)
    assert np.abs(c - d2).max() <= ATOL


def test_attention_reads_what_the_gpu_write_path_wrote():
    cfg = si.get_config(0)                                   # fp32, 8 heads, 256 tokens, r = 8
    B, H, T, bits, G = cfg.batch, cfg.n_kv_heads, cfg.n_tokens, cfg.bits, cfg.group_size
    qp, k, v = (to_torch(x, cfg.dtype) for x in (si.gen_queries(cfg), si.gen_keys(cfg), si.gen_values(cfg)))
    s = sq.Subspace(H, D)
    sq.squat_build_subspace(s, qp, cfg.rank_r, cfg.lam, cfg.block_g)
    kc, ks, kz = alloc_key_outputs(B, H, T, D, bits, G)
    vc, vs, vz = alloc_value_outputs(B, H, T, D, bits, G)
    sq.squat_quantize_keys(s, k, bits, G, kc, ks, kz)
    sq.squat_quantize_values(v, bits, G, vc, vs, vz)
    q = qp[:, -1, :].reshape(1, cfg.n_q_heads, D).contiguous()     # the newest prompt token's queries
    out = _run(q, (kc, ks, kz, vc, vs, vz), H, T, bits, G)
    units = {}
    for h in range(H):
        units[0, h] = ({"codes": oracle.unpack(kc[0, h].cpu().numpy(), D, bits), "scale": ks[0, h].cpu().numpy(),
                        "zero": kz[0, h].cpu().numpy()},
                       {"codes": oracle.unpack(vc[0, h].cpu().numpy(), D, bits), "scale": vs[0, h].cpu().numpy(),
                        "zero": vz[0, h].cpu().numpy()})
    _check(out, q.double().cpu().numpy(), units, H, G)
    s.close()


def test_attention_argument_errors():
    B, H, T, bits, G = 1, 1, 64, 2, 32
    cache, _ = _oracle_cache(5, B, H, T, bits, G)
    q = torch.zeros(B, H, D).cuda()
    out = torch.empty((B, H, D), dtype=torch.float32, device="cuda")
    ws = torch.empty(sq.squat_decode_attention_workspace_bytes(B, H, T), dtype=torch.uint8, device="cuda")
    with pytest.raises(sq.SquatError):                       # tokens not a multiple of the group size
        sq.squat_decode_attention(q, *cache, H, 48, bits, G, out, ws)
    with pytest.raises(sq.SquatError):                       # unsupported code width
        sq.squat_decode_attention(q, *cache, H, T, 3, G, out, ws)
    with pytest.raises(sq.SquatError):                       # nothing to attend to
        sq.squat_decode_attention(q, *cache, H, 0, bits, G, out, ws)
    with pytest.raises(sq.SquatError):                       # workspace too small
        sq.squat_decode_attention(q, *cache, H, T, bits, G, out, ws[:16])
    big = torch.zeros(B, H, 129, D).cuda()
    with pytest.raises(sq.SquatError):                       # residual buffer beyond the supported length
        sq.squat_decode_attention(q, *cache, H, T, bits, G, out, ws, big, big)


# ---------------------------------------------------------------------------------------------------------
# Keys stored before the rotary position embedding (Section 4, the "pre" variant): the reader turns every
# dequantized key row at its position.  Oracle: dequantize, rope_rows at first_pos + t, attention in float64.

def _run_pre(q, cache, H, T, bits, G, first_pos, table_positions, k_res=None, v_res=None, base=10000.0):
    B, Hq, _ = q.shape
    out = torch.empty((B, Hq, D), dtype=torch.float32, device="cuda")
    ws = torch.empty(sq.squat_decode_attention_workspace_bytes(B, Hq, T), dtype=torch.uint8, device="cuda")
    table = sq.squat_rope_table(table_positions, base).cuda()
    sq.squat_decode_attention_pre_rope(q, *cache, H, T, bits, G, out, ws, table, table_positions, first_pos, k_res, v_res)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64)


def _check_pre(out, q_used, units, H, G, first_pos, k_res=None, v_res=None, T=None, base=10000.0):
    B, Hq, _ = q_used.shape
    qpk = Hq // H
    worst = 0.0
    for b in range(B):
        for h in range(H):
            kq, vq = units[b, h]
            n = kq["codes"].shape[0] if T is None else T
            ref = oracle.decode_attention_over_pre_rope_cache(
                q_used[b, h * qpk:(h + 1) * qpk], kq["codes"][:n], kq["scale"][:n // G], kq["zero"][:n // G],
                vq["codes"][:n], vq["scale"][:n], vq["zero"][:n], G, first_pos,
                None if k_res is None else k_res[b, h], None if v_res is None else v_res[b, h], base)
            worst = max(worst, np.abs(out[b, h * qpk:(h + 1) * qpk] - ref).max())
    assert worst <= ATOL, worst
    return worst


@pytest.mark.parametrize("bits,G,qpk,T,R,first_pos,res_dtype", [
    (2, 32, 1, 256, 0, 0, torch.float32),          # MHA, cache from position 0, no residual buffer
    (2, 32, 4, 2112, 32, 4096, torch.bfloat16),    # GQA 4:1, 3 chunks with a ragged one, positions 4096 .. 6239
    (4, 64, 2, 1088, 128, 32, torch.float32),      # 4-bit codes, full residual buffer
    (2, 128, 8, 128, 5, 8064, torch.float32),      # two passes over the cache (8 query heads per KV head)
    (4, 32, 3, 96, 1, 0, torch.bfloat16),
])
def test_pre_rope_reader_matches_the_oracle(bits, G, qpk, T, R, first_pos, res_dtype):
    B, H = 2, 2
    cache, units = _oracle_cache(40 + bits + G + qpk, B, H, T, bits, G)
    g = torch.Generator().manual_seed(T + R + first_pos)
    q = torch.randn(B, H * qpk, D, generator=g).to(torch.bfloat16).cuda()
    k_res = v_res = None
    if R:
        k_res = torch.randn(B, H, R, D, generator=g).to(res_dtype).cuda()
        v_res = torch.randn(B, H, R, D, generator=g).to(res_dtype).cuda()
    out = _run_pre(q, cache, H, T, bits, G, first_pos, first_pos + T + R, k_res, v_res)
    kr = None if k_res is None else k_res.double().cpu().numpy()
    vr = None if v_res is None else v_res.double().cpu().numpy()
    print("max err", _check_pre(out, q.double().cpu().numpy(), units, H, G, first_pos, kr, vr))


def test_pre_rope_reader_special_cases():
    B, H, T, bits, G = 1, 2, 512, 2, 32
    cache, units = _oracle_cache(7, B, H, T, bits, G)
    g = torch.Generator().manual_seed(11)
    q = torch.randn(B, H, D, generator=g).cuda()
    k_res, v_res = torch.randn(B, H, 16, D, generator=g).cuda(), torch.randn(B, H, 16, D, generator=g).cuda()
    kr, vr = k_res.double().cpu().numpy(), v_res.double().cpu().numpy()
    qn = q.double().cpu().numpy()
    # another base (Llama-3.1 uses 500000)
    out = _run_pre(q, cache, H, T, bits, G, 64, 1024, k_res, v_res, base=500000.0)
    _check_pre(out, qn, units, H, G, 64, kr, vr, base=500000.0)
    # only the residual buffer, at positions 96 ..
    out = _run_pre(q, cache, H, 0, bits, G, 96, 256, k_res, v_res)
    _check_pre(out, qn, units, H, G, 96, kr, vr, T=0)
    # a prefix of a longer cache
    out = torch.empty((B, H, D), dtype=torch.float32, device="cuda")
    ws = torch.empty(sq.squat_decode_attention_workspace_bytes(B, H, 192), dtype=torch.uint8, device="cuda")
    table = sq.squat_rope_table(1024).cuda()
    sq.squat_decode_attention_pre_rope(q, *cache, H, 192, bits, G, out, ws, table, 1024, 0, k_res, v_res,
                                       cache_stride_b=H * T, cache_stride_h=T)
    torch.cuda.synchronize()
    _check_pre(out.cpu().numpy().astype(np.float64), qn, units, H, G, 0, kr, vr, T=192)
    # the embedding matters: read as if the keys had been stored after it, the result differs
    plain = _run(q, cache, H, T, bits, G, k_res, v_res)
    pre = _run_pre(q, cache, H, T, bits, G, 0, 1024, k_res, v_res)
    assert np.abs(plain - pre).max() > 1e-3
    # argument errors: first_pos not a multiple of 32, table too short
    with pytest.raises(sq.SquatError):
        sq.squat_decode_attention_pre_rope(q, *cache, H, T, bits, G, out, ws, table, 1024, 8, k_res, v_res)
    with pytest.raises(sq.SquatError):
        sq.squat_decode_attention_pre_rope(q, *cache, H, T, bits, G, out, ws, table, 1024, 512, k_res, v_res)


# ---------------------------------------------------------------------------------------------------------
# The readers over a cache with 16-bit (binary16) scales and zero-points, built by the oracle's 16-bit variants.

def _oracle_cache16(seed, B, H, T, bits, G):
    rng = np.random.default_rng(seed)
    K = rng.standard_normal((B, H, T, D))
    K[..., 7] *= 8.0
    V = rng.standard_normal((B, H, T, D))
    kc = np.zeros((B, H, T, D * bits // 8), np.uint8)
    vc = np.zeros_like(kc)
    ks = np.zeros((B, H, T // G, D), np.float16)
    kz = np.zeros_like(ks)
    vs = np.zeros((B, H, T, D // G), np.float16)
    vz = np.zeros_like(vs)
    units = {}
    for b in range(B):
        for h in range(H):
            kq = oracle.quant_keys(K[b, h], G, bits, meta16=True)
            vq = oracle.quant_values_f32(V[b, h].astype(np.float32), G, bits, meta16=True)
            kc[b, h], vc[b, h] = oracle.pack(kq["codes"], bits), oracle.pack(vq["codes"], bits)
            ks[b, h], kz[b, h] = kq["scale"].astype(np.float16), kq["zero"].astype(np.float16)      # exact: binary16 values
            vs[b, h], vz[b, h] = vq["scale"].astype(np.float16), vq["zero"].astype(np.float16)
            assert np.array_equal(ks[b, h].astype(np.float32), kq["scale"])
            units[b, h] = (kq, vq)
    dev = lambda a: torch.from_numpy(a).cuda()
    return (dev(kc), dev(ks), dev(kz), dev(vc), dev(vs), dev(vz)), units


@pytest.mark.parametrize("bits,G,qpk,T,R", [(2, 32, 1, 256, 0), (2, 32, 4, 2112, 32), (4, 64, 2, 1088, 128), (2, 128, 8, 128, 5)])
def test_readers_over_a_cache_with_16_bit_metadata(bits, G, qpk, T, R):
    B, H = 2, 2
    cache, units = _oracle_cache16(70 + bits + G + qpk, B, H, T, bits, G)
    g = torch.Generator().manual_seed(T + R)
    q = torch.randn(B, H * qpk, D, generator=g).to(torch.bfloat16).cuda()
    k_res = v_res = None
    if R:
        k_res = torch.randn(B, H, R, D, generator=g).cuda()
        v_res = torch.randn(B, H, R, D, generator=g).cuda()
    kr = None if k_res is None else k_res.double().cpu().numpy()
    vr = None if v_res is None else v_res.double().cpu().numpy()
    qn = q.double().cpu().numpy()
    out = _run(q, cache, H, T, bits, G, k_res, v_res)                          # keys stored after the rotary embedding
    print("max err", _check(out, qn, units, H, G, kr, vr))
    out = _run_pre(q, cache, H, T, bits, G, 64, 64 + T + R, k_res, v_res)      # keys stored before it
    print("max err (pre)", _check_pre(out, qn, units, H, G, 64, kr, vr))
