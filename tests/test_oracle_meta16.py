"""CPU pins of the oracle's 16-bit-metadata variants (scale and zero-point stored as IEEE binary16; the "KV size"
columns of Tables 1-2 imply this storage) -- against things other than itself: numpy's own float16 conversion,
a numpy restatement of the value quantizer on float32 / float16 arrays, the r = 0 reduction of the key quantizer,
dequantize-quantize idempotence, and the size formula of the packed cache."""
import numpy as np
import pytest

import oracle

D = 128


def test_half_round_is_numpys_float16_conversion():
    rng = np.random.default_rng(0)
    x = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * np.float32(10.0) ** rng.integers(-8, 5, 20000).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 65504.0, 65519.99, 65520.0, 70000.0, -65520.0, 6.1035156e-05, 6.0975552e-05,
                  5.9604645e-08, 2.9802322e-08, 2.9802326e-08, 8.9406967e-08, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11,
                  2049.0, 2051.0, np.inf, -np.inf], dtype=np.float32)])
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).astype(np.float32)
    got = oracle.half_round(x)
    assert np.array_equal(got, want)
    # ties go to even: 1 + 2^-11 lies half way between 1 and 1 + 2^-10 -> 1; 1 + 3 * 2^-11 -> 1 + 2^-9
    assert oracle.half_round(np.float32(1.0 + 2.0 ** -11)) == 1.0
    assert oracle.half_round(np.float32(1.0 + 3 * 2.0 ** -11)) == np.float32(1.0 + 2.0 ** -9)


@pytest.mark.parametrize("bits,G", [(2, 32), (4, 64), (2, 128)])
def test_values_with_16_bit_metadata_match_a_numpy_restatement(bits, G):
    rng = np.random.default_rng(1)
    V = (rng.standard_normal((40, D)) * 3 + 0.7).astype(np.float32)
    out = oracle.quant_values_f32(V, G, bits, meta16=True)
    L = np.float32((1 << bits) - 1)
    Vg = V.reshape(40, D // G, G)
    m, M = Vg.min(axis=2), Vg.max(axis=2)
    delta = ((M - m) / L).astype(np.float32).astype(np.float16).astype(np.float32)      # binary32 division, then binary16
    z = m.astype(np.float16).astype(np.float32)
    t = ((Vg - z[..., None]).astype(np.float32) / delta[..., None]).astype(np.float32)
    codes = np.clip(np.rint(t), 0, L).astype(np.uint8).reshape(40, D)
    assert np.array_equal(out["scale"], delta) and np.array_equal(out["zero"], z)
    assert np.array_equal(out["codes"], codes)
    # the stored values are binary16 numbers; the float32 variant's are generally not
    assert np.array_equal(out["scale"].astype(np.float16).astype(np.float32), out["scale"])
    plain = oracle.quant_values_f32(V, G, bits)
    assert not np.array_equal(plain["scale"], out["scale"])
    assert np.abs(plain["scale"] - out["scale"]).max() <= 2.0 ** -11 * np.abs(plain["scale"]).max()


def test_keys_with_16_bit_metadata_r0_is_round_to_nearest_on_the_stored_grid():
    # W = None: no correction -> every (group, channel) is independent: plain asymmetric quantization against
    # the binary16-rounded scale and zero-point, codes clamped
    rng = np.random.default_rng(2)
    n, G, bits = 96, 32, 2
    K = rng.standard_normal((n, D)) * 2 + 1.3
    out = oracle.quant_keys(K, G, bits, meta16=True)
    L = (1 << bits) - 1
    Kg = K.reshape(n // G, G, D)
    m, M = Kg.min(axis=1), Kg.max(axis=1)
    z = m.astype(np.float32).astype(np.float16).astype(np.float32)
    s = ((M - m) / L).astype(np.float32).astype(np.float16).astype(np.float32)
    assert np.array_equal(out["zero"], z) and np.array_equal(out["scale"], s)
    assert np.array_equal(out["raw_zero"], m.astype(np.float32)) and np.array_equal(out["raw_scale"], ((M - m) / L).astype(np.float32))
    t = (Kg - z[:, None, :].astype(np.float64)) / s[:, None, :].astype(np.float64)
    codes = np.clip(np.rint(t), 0, L).astype(np.uint8).reshape(n, D)
    assert np.array_equal(out["codes"], codes)
    Khat = codes.reshape(n // G, G, D) * s[:, None, :].astype(np.float64) + z[:, None, :].astype(np.float64)
    assert np.abs(out["Khat"] - Khat.reshape(n, D)).max() == 0.0
    # error of the 16-bit variant stays within half a step plus the metadata rounding (2^-11 relative of |zero| and range)
    bound = 0.5 * s[:, None, :] + 2.0 ** -10 * (np.abs(z)[:, None, :] + L * s[:, None, :])
    assert np.all(np.abs(out["Khat"].reshape(n // G, G, D) - Kg) <= bound + 1e-12)


def test_forced_metadata_replaces_single_group_channel_pairs():
    rng = np.random.default_rng(3)
    n, G, bits = 64, 32, 2
    K = rng.standard_normal((n, D))
    W = np.tril(rng.standard_normal((D, D)) * 0.05, -1)
    base = oracle.quant_keys(K, G, bits, W, meta16=True)
    fs = np.full((n // G, D), np.nan, np.float32)
    fz = np.full((n // G, D), np.nan, np.float32)
    assert np.array_equal(oracle.quant_keys(K, G, bits, W, meta16=True, force_meta=(fs, fz))["codes"], base["codes"])
    # move the zero-point of (group 1, channel 5) one binary16 step down: that pair's stored value changes, earlier
    # channels and the other group are untouched, later channels of group 1 may change through the feedback
    z = base["zero"][1, 5]
    fz[1, 5] = np.nextafter(np.float16(z), np.float16(-np.inf)).astype(np.float32)
    moved = oracle.quant_keys(K, G, bits, W, meta16=True, force_meta=(fs, fz))
    assert moved["zero"][1, 5] == fz[1, 5] and moved["zero"][1, 5] != z
    assert np.array_equal(moved["codes"][:G], base["codes"][:G])
    assert np.array_equal(moved["codes"][G:, :5], base["codes"][G:, :5])
    assert np.array_equal(moved["zero"][:, :5], base["zero"][:, :5])


def test_dequantize_then_quantize_is_idempotent_with_16_bit_metadata():
    rng = np.random.default_rng(4)
    n, G, bits = 64, 32, 2
    K = rng.standard_normal((n, D)) * 1.7 - 0.4
    a = oracle.quant_keys(K, G, bits, meta16=True)
    Kd = oracle.dequant_keys(a["codes"], a["scale"], a["zero"], G)
    b = oracle.quant_keys(Kd, G, bits, meta16=True)
    assert np.array_equal(a["codes"], b["codes"])
    assert np.array_equal(a["scale"], b["scale"]) and np.array_equal(a["zero"], b["zero"])


def test_cache_size_ratio_with_16_bit_metadata_is_the_papers_18_75_percent():
    # 2-bit codes + binary16 scale and zero per 32 elements, against 16-bit elements (the "KV size" columns of
    # Tables 1-2 report 19.1-21.4 % including the full-precision residual tokens)
    bits, G = 2, 32
    ratio = (bits + 2 * 16 / G) / 16
    assert ratio == 0.1875
    assert (bits + 2 * 32 / G) / 16 == 0.25          # the float32-metadata layout of the default path
