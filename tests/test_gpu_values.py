"""GPU parity: value quantization (bit-exact) and dequantization, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import squat_inputs as si
import paper_2503_24358_b200 as sq
from parity import alloc_value_outputs, from_torch_bf16, to_torch

pytestmark = pytest.mark.gpu


def _check_values(v_np, dtype, bits, G, v_dev=None):
    """v_np: generator output [B,H,T,d]; compares every unit with the oracle, bit for bit."""
    B, H, T, d = v_np.shape
    v = to_torch(v_np, dtype) if v_dev is None else v_dev
    codes, scales, zeros = alloc_value_outputs(B, H, T, d, bits, G)
    sq.squat_quantize_values(v, bits, G, codes, scales, zeros)
    torch.cuda.synchronize()
    v32 = si.to_f32(v_np, dtype).reshape(B * H * T, d)
    ref = oracle.quant_values_f32(v32, G, bits)
    got_codes = oracle.unpack(codes.cpu().numpy().reshape(B * H * T, -1), d, bits)
    assert np.array_equal(got_codes, ref["codes"])
    assert np.array_equal(codes.cpu().numpy().reshape(B * H * T, -1), oracle.pack(ref["codes"], bits))
    assert np.array_equal(scales.cpu().numpy().reshape(-1, d // G).view(np.uint32), ref["scale"].view(np.uint32))
    assert np.array_equal(zeros.cpu().numpy().reshape(-1, d // G).view(np.uint32), ref["zero"].view(np.uint32))
    return codes, scales, zeros, ref


@pytest.mark.parametrize("bits,G", [(2, 32), (4, 32), (2, 64), (4, 128), (2, 128), (4, 64)])
def test_values_config0_f32(bits, G):
    cfg = si.get_config(0)
    _check_values(si.gen_values(cfg), cfg.dtype, bits, G)


@pytest.mark.parametrize("bits,G", [(2, 32), (4, 32), (2, 128)])
def test_values_config1_bf16_full(bits, G):
    cfg = si.get_config(1)
    _check_values(si.gen_values(cfg), cfg.dtype, bits, G)       # 131072 tokens: full size, all elements


@pytest.mark.parametrize("T", [1, 3, 33, 257])
def test_values_ragged_token_counts(T):
    cfg = si.get_config(1).with_(batch=2, n_kv_heads=3)
    _check_values(si.gen_values(cfg, n_tokens=T), cfg.dtype, 2, 32)


def test_values_empty_input_is_a_no_op():
    v = torch.empty((1, 4, 0, 128), dtype=torch.bfloat16, device="cuda")
    codes, scales, zeros = alloc_value_outputs(1, 4, 0, 128, 2, 32)
    n0 = sq.squat_kernel_launch_count()
    sq.squat_quantize_values(v, 2, 32, codes, scales, zeros)
    assert sq.squat_kernel_launch_count() == n0


def test_values_strided_input_and_cache_sized_output():
    # input: a [B,T,H,d] tensor viewed as [B,H,T,d]; output: written into a longer cache at a token offset
    cfg = si.get_config(1).with_(batch=2, n_kv_heads=4)
    T, Tcache, off, d, bits, G = 64, 256, 96, 128, 2, 32
    v_np = si.gen_values(cfg, n_tokens=T)
    v_bthd = to_torch(np.ascontiguousarray(v_np.transpose(0, 2, 1, 3)), cfg.dtype)
    v = v_bthd.permute(0, 2, 1, 3)
    assert not v.is_contiguous()
    codes = torch.zeros((2, 4, Tcache, d * bits // 8), dtype=torch.uint8, device="cuda")
    scales = torch.zeros((2, 4, Tcache, d // G), dtype=torch.float32, device="cuda")
    zeros = torch.zeros_like(scales)
    sq.squat_quantize_values(v, bits, G, codes[:, :, off:], scales[:, :, off:], zeros[:, :, off:],
                             out_stride_b=4 * Tcache, out_stride_h=Tcache)
    torch.cuda.synchronize()
    ref = oracle.quant_values_f32(si.to_f32(v_np, cfg.dtype).reshape(-1, d), G, bits)
    got = codes[:, :, off:off + T].contiguous().cpu().numpy().reshape(-1, d * bits // 8)
    assert np.array_equal(got, oracle.pack(ref["codes"], bits))
    assert np.array_equal(scales[:, :, off:off + T].contiguous().cpu().numpy().reshape(-1, d // G), ref["scale"])
    assert not codes[:, :, :off].any() and not codes[:, :, off + T:].any()      # nothing outside the window


def test_values_exact_ties_and_constant_groups():
    # hand-made rows: exact ties (round half to even) and a constant group (scale 0, flag raised)
    d, G = 128, 32
    row = np.zeros(d, dtype=np.float32)
    row[:8] = [0.0, 3.0, 0.5, 1.5, 2.5, 1.0, 2.0, 0.25]
    row[32:64] = 7.0                                     # constant group
    row[64:96] = np.linspace(-1, 1, 32, dtype=np.float32)
    row[96:] = np.arange(32, dtype=np.float32) * 0.1
    v_np = np.tile(row, (1, 1, 5, 1))
    sq.squat_get_device_status(clear=True)
    codes, scales, zeros, ref = _check_values(v_np, "f32", 2, G)
    assert ref["codes"][0, :8].tolist() == [0, 3, 0, 2, 2, 1, 2, 0]
    assert scales[0, 0, 0, 1].item() == 0.0
    assert sq.squat_get_device_status(clear=True) & sq.FLAG_ZERO_RANGE


def test_values_near_tie_fallback_is_exercised():
    # bf16 data sits on a coarse grid, so many elements are exact or near rounding ties; the
    # exact-division fallback must make them agree with the binary32 sequence bit for bit
    rng = np.random.default_rng(11)
    v = (rng.integers(-64, 64, size=(1, 2, 4096, 128)) / 16.0).astype(np.float32)
    _check_values(si.f32_to_bf16_bits(v), "bf16", 2, 32)
    _check_values(v, "f32", 4, 32)


@pytest.mark.parametrize("kind", ["values", "keys"])
@pytest.mark.parametrize("bits,G,out_dtype", [(2, 32, torch.float32), (4, 64, torch.float32), (2, 128, torch.bfloat16), (4, 32, torch.bfloat16)])
def test_dequantize_matches_oracle(kind, bits, G, out_dtype):
    rng = np.random.default_rng(bits + G)
    B, H, T, d = 2, 3, 256, 128
    codes_np = rng.integers(0, 2 ** bits, (B * H * T, d), dtype=np.uint8)
    packed = torch.from_numpy(oracle.pack(codes_np, bits).reshape(B, H, T, -1)).cuda()
    if kind == "values":
        sc = rng.random((B * H * T, d // G), dtype=np.float32) + 0.01
        zr = rng.standard_normal((B * H * T, d // G)).astype(np.float32)
        ref = oracle.dequant_values(codes_np, sc, zr, G)
        k = sq.SQUAT_VALUES
        shp = (B, H, T, d // G)
    else:
        sc = rng.random((B * H * T // G, d), dtype=np.float32) + 0.01
        zr = rng.standard_normal((B * H * T // G, d)).astype(np.float32)
        ref = oracle.dequant_keys(codes_np, sc, zr, G)
        k = sq.SQUAT_KEYS
        shp = (B, H, T // G, d)
    out = torch.empty((B, H, T, d), dtype=out_dtype, device="cuda")
    sq.squat_dequantize(k, packed, torch.from_numpy(sc.reshape(shp)).cuda(), torch.from_numpy(zr.reshape(shp)).cuda(),
                        B, H, T, d, bits, G, out)
    torch.cuda.synchronize()
    ref32 = ref.astype(np.float32)                    # the exact value rounded once to float32
    if out_dtype == torch.float32:
        assert np.array_equal(out.cpu().numpy().reshape(-1, d), ref32)
    else:
        assert np.array_equal(from_torch_bf16(out).reshape(-1, d), si.bf16_bits_to_f32(si.f32_to_bf16_bits(ref32)))


def test_quantize_dequantize_roundtrip_error_bound():
    cfg = si.get_config(1)
    v_np = si.gen_values(cfg, n_tokens=512)
    B, H, T, d = v_np.shape
    codes, scales, zeros, _ = _check_values(v_np, cfg.dtype, 2, 32)
    out = torch.empty((B, H, T, d), dtype=torch.float32, device="cuda")
    sq.squat_dequantize(sq.SQUAT_VALUES, codes, scales, zeros, B, H, T, d, 2, 32, out)
    err = (out.cpu().numpy() - si.to_f32(v_np, cfg.dtype)).reshape(B, H, T, d // 32, 32)
    bound = 0.5 * scales.cpu().numpy()[..., None] * (1 + 1e-6)
    assert np.all(np.abs(err) <= bound)


@pytest.mark.parametrize("d,G,bits", [(64, 32, 2), (64, 64, 4), (256, 32, 2), (256, 128, 4)])
def test_values_and_dequantize_other_head_dims(d, G, bits):
    # the value quantizer and the dequantizer are not tied to d = 128: spans of 32 channels, 8 channels per thread
    rng = np.random.default_rng(d + G + bits)
    B, H, T = 2, 5, 70
    v_np = rng.standard_normal((B, H, T, d)).astype(np.float32)
    codes, scales, zeros, ref = _check_values(v_np, "f32", bits, G)
    out = torch.empty((B, H, T, d), dtype=torch.float32, device="cuda")
    sq.squat_dequantize(sq.SQUAT_VALUES, codes, scales, zeros, B, H, T, d, bits, G, out)
    torch.cuda.synchronize()
    want = oracle.dequant_values(ref["codes"], ref["scale"], ref["zero"], G).astype(np.float32)
    assert np.array_equal(out.cpu().numpy().reshape(-1, d), want)
    # key layout (groups of G tokens per channel) at the same head dimension
    Tk = 2 * G
    codes_np = rng.integers(0, 2 ** bits, (B * H * Tk, d), dtype=np.uint8)
    sc = rng.random((B * H * Tk // G, d), dtype=np.float32) + 0.01
    zr = rng.standard_normal((B * H * Tk // G, d)).astype(np.float32)
    packed = torch.from_numpy(oracle.pack(codes_np, bits).reshape(B, H, Tk, -1)).cuda()
    outk = torch.empty((B, H, Tk, d), dtype=torch.float32, device="cuda")
    sq.squat_dequantize(sq.SQUAT_KEYS, packed, torch.from_numpy(sc.reshape(B, H, Tk // G, d)).cuda(),
                        torch.from_numpy(zr.reshape(B, H, Tk // G, d)).cuda(), B, H, Tk, d, bits, G, outk)
    torch.cuda.synchronize()
    assert np.array_equal(outk.cpu().numpy().reshape(-1, d), oracle.dequant_keys(codes_np, sc, zr, G).astype(np.float32))


def test_values_many_heads_and_batches():
    # batch and heads are grid dimensions of both kernels: more of them than SMs, few tokens each
    rng = np.random.default_rng(11)
    B, H, T, d, bits, G = 37, 200, 3, 128, 2, 32
    v_np = rng.standard_normal((B, H, T, d)).astype(np.float32)
    codes, scales, zeros, ref = _check_values(v_np, "f32", bits, G)
    out = torch.empty((B, H, T, d), dtype=torch.float32, device="cuda")
    sq.squat_dequantize(sq.SQUAT_VALUES, codes, scales, zeros, B, H, T, d, bits, G, out)
    torch.cuda.synchronize()
    want = oracle.dequant_values(ref["codes"], ref["scale"], ref["zero"], G).astype(np.float32)
    assert np.array_equal(out.cpu().numpy().reshape(-1, d), want)

