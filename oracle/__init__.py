"""ctypes front end of the CPU oracle (oracle/squat_oracle.c)  --  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It marshals numpy arrays into the C functions and adds nothing to their
arithmetic.  It never imports the CUDA package.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "squat_oracle.c")
_LIB = os.path.join(_HERE, "libsquat_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE: no contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-frounding-math",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.sqo_kv_cache_bytes.restype = ctypes.c_longlong
        _lib.sqo_kv_cache_bytes.argtypes = [ctypes.c_longlong] * 6
    return _lib


def _p(a, ty):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ty))


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


_D, _F, _U8, _I16 = ctypes.c_double, ctypes.c_float, ctypes.c_uint8, ctypes.c_int16


def gram(Qc):
    Qc = np.ascontiguousarray(Qc, dtype=np.float64)
    N, d = Qc.shape
    M = np.empty((d, d), dtype=np.float64)
    _check(_load().sqo_gram(_p(Qc, _D), ctypes.c_long(N), d, _p(M, _D)), "gram")
    return M


def jacobi_eig(A):
    """Eigenvalues (descending) and eigenvectors (rows) of a symmetric matrix."""
    A = np.array(A, dtype=np.float64, order="C", copy=True)
    d = A.shape[0]
    mu = np.empty(d, dtype=np.float64)
    V = np.empty((d, d), dtype=np.float64)
    _check(_load().sqo_jacobi_eig(_p(A, _D), d, _p(mu, _D), _p(V, _D)), "jacobi_eig")
    return mu, V


def query_subspace(Qc, r):
    """Returns (Qhat [r, d], mu [d], V [d, d] rows = eigenvectors of Qc^T Qc)."""
    Qc = np.ascontiguousarray(Qc, dtype=np.float64)
    N, d = Qc.shape
    Qhat = np.zeros((r, d), dtype=np.float64)
    mu = np.empty(d, dtype=np.float64)
    V = np.empty((d, d), dtype=np.float64)
    _check(_load().sqo_query_subspace(_p(Qc, _D), ctypes.c_long(N), d, r, _p(Qhat, _D), _p(mu, _D), _p(V, _D)),
           "query_subspace")
    return Qhat, mu, V


def update_matrices(Qhat, d, lam, g=1, want_chain=False):
    """Returns dict with W, P, P_inv and (optionally) the list Ainv[1..T]."""
    Qhat = np.ascontiguousarray(Qhat, dtype=np.float64).reshape(-1, d)
    r = Qhat.shape[0]
    W = np.empty((d, d), dtype=np.float64)
    P = np.empty((d, d), dtype=np.float64)
    Pinv = np.empty((d, d), dtype=np.float64)
    T = d // g
    chain = None
    if want_chain:
        chain = np.empty(sum((t * g) ** 2 for t in range(1, T + 1)), dtype=np.float64)
    _check(_load().sqo_update_matrices(_p(Qhat, _D) if r else None, r, d, ctypes.c_double(lam), g,
                                       _p(W, _D), _p(P, _D), _p(Pinv, _D), _p(chain, _D)), "update_matrices")
    out = {"W": W, "P": P, "P_inv": Pinv}
    if want_chain:
        mats, off = {}, 0
        for t in range(1, T + 1):
            m = t * g
            mats[t] = chain[off:off + m * m].reshape(m, m).copy()
            off += m * m
        out["Ainv"] = mats
    return out


def half_round(x):
    """float32 array rounded to the nearest binary16 value (ties to even), as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    lib = _load()
    lib.sqo_half_round.restype = ctypes.c_float
    lib.sqo_half_round.argtypes = [ctypes.c_float]
    return np.array([lib.sqo_half_round(float(v)) for v in x.ravel()], dtype=np.float32).reshape(x.shape)


def quant_keys(K, G, bits, W=None, force=None, want_tval=False, meta16=False, force_meta=None):
    """Algorithm 1 Quant on [n, d] keys. Returns dict(codes, scale, zero, Khat[, tval]).  meta16: scale and zero are
    stored as binary16 (returned as float32 arrays holding those values; raw_scale / raw_zero are the float32 values
    before that rounding); force_meta = (scale, zero) float32 arrays [n/G, d] with NaN where nothing is forced."""
    K = np.ascontiguousarray(K, dtype=np.float64)
    n, d = K.shape
    codes = np.empty((n, d), dtype=np.uint8)
    scale = np.empty((n // G, d), dtype=np.float32)
    zero = np.empty((n // G, d), dtype=np.float32)
    Khat = np.empty((n, d), dtype=np.float64)
    tval = np.empty((n, d), dtype=np.float64) if want_tval else None
    if W is not None:
        W = np.ascontiguousarray(W, dtype=np.float64)
        assert W.shape == (d, d)
    if force is not None:
        force = np.ascontiguousarray(force, dtype=np.int16)
        assert force.shape == (n, d)
    raw_s = np.empty_like(scale) if meta16 else None
    raw_z = np.empty_like(zero) if meta16 else None
    fs = fz = None
    if force_meta is not None:
        fs = np.ascontiguousarray(force_meta[0], dtype=np.float32)
        fz = np.ascontiguousarray(force_meta[1], dtype=np.float32)
        assert fs.shape == scale.shape and fz.shape == zero.shape
    _check(_load().sqo_quant_keys_m16(_p(K, _D), ctypes.c_long(n), d, G, bits, _p(W, _D), _p(codes, _U8),
                                      _p(scale, _F), _p(zero, _F), _p(Khat, _D), _p(tval, _D), _p(force, _I16),
                                      1 if meta16 else 0, _p(raw_s, _F), _p(raw_z, _F), _p(fs, _F), _p(fz, _F)),
           "quant_keys")
    out = {"codes": codes, "scale": scale, "zero": zero, "Khat": Khat}
    if meta16:
        out["raw_scale"], out["raw_zero"] = raw_s, raw_z
    if want_tval:
        out["tval"] = tval
    return out


def quant_values_f32(V, G, bits, meta16=False):
    V = np.ascontiguousarray(V, dtype=np.float32)
    n, d = V.shape
    codes = np.empty((n, d), dtype=np.uint8)
    scale = np.empty((n, d // G), dtype=np.float32)
    zero = np.empty((n, d // G), dtype=np.float32)
    fn = _load().sqo_quant_values_f32_m16 if meta16 else _load().sqo_quant_values_f32
    _check(fn(_p(V, _F), ctypes.c_long(n), d, G, bits, _p(codes, _U8), _p(scale, _F), _p(zero, _F)), "quant_values_f32")
    return {"codes": codes, "scale": scale, "zero": zero}


def quant_values_f64(V, G, bits):
    V = np.ascontiguousarray(V, dtype=np.float64)
    n, d = V.shape
    codes = np.empty((n, d), dtype=np.uint8)
    scale = np.empty((n, d // G), dtype=np.float32)
    zero = np.empty((n, d // G), dtype=np.float32)
    _check(_load().sqo_quant_values_f64(_p(V, _D), ctypes.c_long(n), d, G, bits, _p(codes, _U8), _p(scale, _F),
                                        _p(zero, _F)), "quant_values_f64")
    return {"codes": codes, "scale": scale, "zero": zero}


def dequant_keys(codes, scale, zero, G):
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    n, d = codes.shape
    scale = np.ascontiguousarray(scale, dtype=np.float32)
    zero = np.ascontiguousarray(zero, dtype=np.float32)
    out = np.empty((n, d), dtype=np.float64)
    _check(_load().sqo_dequant_keys(_p(codes, _U8), _p(scale, _F), _p(zero, _F), ctypes.c_long(n), d, G, _p(out, _D)),
           "dequant_keys")
    return out


def dequant_values(codes, scale, zero, G):
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    n, d = codes.shape
    scale = np.ascontiguousarray(scale, dtype=np.float32)
    zero = np.ascontiguousarray(zero, dtype=np.float32)
    out = np.empty((n, d), dtype=np.float64)
    _check(_load().sqo_dequant_values(_p(codes, _U8), _p(scale, _F), _p(zero, _F), ctypes.c_long(n), d, G,
                                      _p(out, _D)), "dequant_values")
    return out


def pack(codes, bits):
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    n, d = codes.shape
    packed = np.empty((n, d * bits // 8), dtype=np.uint8)
    _check(_load().sqo_pack(_p(codes, _U8), ctypes.c_long(n), d, bits, _p(packed, _U8)), "pack")
    return packed


def unpack(packed, d, bits):
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    n = packed.shape[0]
    codes = np.empty((n, d), dtype=np.uint8)
    _check(_load().sqo_unpack(_p(packed, _U8), ctypes.c_long(n), d, bits, _p(codes, _U8)), "unpack")
    return codes


def attention_decode(q, K, V):
    """One decode step over cached rows K, V [n, d] for the query vectors q [nq, d] (Section 2)."""
    q = np.ascontiguousarray(np.atleast_2d(q), dtype=np.float64)
    K = np.ascontiguousarray(K, dtype=np.float64)
    V = np.ascontiguousarray(V, dtype=np.float64)
    nq, d = q.shape
    n = K.shape[0]
    out = np.empty((nq, d), dtype=np.float64)
    _check(_load().sqo_attention_decode(_p(q, _D), nq, _p(K, _D), _p(V, _D), ctypes.c_long(n), d, _p(out, _D)),
           "attention_decode")
    return out


def decode_attention_over_cache(q, k_codes, k_scale, k_zero, v_codes, v_scale, v_zero, G, k_res=None, v_res=None):
    """What a decode step computes for one (batch, KV head): the quantized part of the cache is
    dequantized (codes [n, d] unpacked), the residual buffer's full-precision rows are appended, then
    attention_decode.  Marshalling only: every number comes from the C functions."""
    Kd = dequant_keys(k_codes, k_scale, k_zero, G)
    Vd = dequant_values(v_codes, v_scale, v_zero, G)
    if k_res is not None and len(k_res):
        Kd = np.concatenate([Kd, np.asarray(k_res, dtype=np.float64)], axis=0)
        Vd = np.concatenate([Vd, np.asarray(v_res, dtype=np.float64)], axis=0)
    return attention_decode(q, Kd, Vd)


def rope_rows(X, pos, base=10000.0):
    """Rotary position embedding of the rows X [n, d] at integer positions pos [n] (Section 4, the variant
    that stores keys before the embedding); returns a new array."""
    X = np.array(X, dtype=np.float64, order="C", copy=True)
    n, d = X.shape
    pos = np.ascontiguousarray(pos, dtype=np.int64)
    assert pos.shape == (n,)
    posl = (ctypes.c_long * n)(*[int(v) for v in pos])
    _check(_load().sqo_rope_rows(_p(X, _D), ctypes.c_long(n), d, posl, ctypes.c_double(base)), "rope_rows")
    return X


def decode_attention_over_pre_rope_cache(q, k_codes, k_scale, k_zero, v_codes, v_scale, v_zero, G, first_pos,
                                         k_res=None, v_res=None, base=10000.0):
    """decode_attention_over_cache for a cache whose keys were quantized BEFORE the rotary embedding: cached
    token t (and then the residual rows) sits at position first_pos + t; its dequantized key row is rotated
    there, the query comes already rotated at its own position.  Marshalling only."""
    Kd = dequant_keys(k_codes, k_scale, k_zero, G) if len(k_codes) else np.zeros((0, np.asarray(q).shape[-1]))
    Vd = dequant_values(v_codes, v_scale, v_zero, G) if len(v_codes) else np.zeros_like(Kd)
    if k_res is not None and len(k_res):
        Kd = np.concatenate([Kd, np.asarray(k_res, dtype=np.float64)], axis=0)
        Vd = np.concatenate([Vd, np.asarray(v_res, dtype=np.float64)], axis=0)
    Kr = rope_rows(Kd, first_pos + np.arange(Kd.shape[0]), base)
    return attention_decode(q, Kr, Vd)


def kv_cache_bytes(batch, seq_len, layers, heads, head_dim, bytes_per_param):
    return int(_load().sqo_kv_cache_bytes(batch, seq_len, layers, heads, head_dim, bytes_per_param))


def build_W(Qc, r, lam, g=1):
    """Convenience: stacked queries -> assembled update matrix W (steps O1 + O2)."""
    d = Qc.shape[1]
    Qhat, mu, V = query_subspace(Qc, r)
    mats = update_matrices(Qhat, d, lam, g)
    mats.update({"Qhat": Qhat, "mu": mu, "V": V})
    return mats


def power_subspace(M, X0, iters):
    """Block power method for the query subspace (the accelerator the paper names for line 5 of Algorithm 1;
    the paper gives no steps, these are the textbook ones):  X <- orth(M X), `iters` times from the start
    block X0 [d, r] (iters = 0: X = orth(X0)), then Rayleigh-Ritz on span(X): B = X^T M X = S diag(theta) S^T,
    Ritz vectors u_i = X s_i.  Returns (Qhat [r, d] with rows sqrt(theta_i) u_i^T, theta descending, X), so
    that Qhat^T Qhat = X B X^T, the compression of M to the iterated subspace, takes the place of the rank-r
    truncation of M.  Library steps: numpy's Householder QR and symmetric eigensolver."""
    M = np.asarray(M, dtype=np.float64)
    X = np.asarray(X0, dtype=np.float64)
    d, r = X.shape
    if M.shape != (d, d):
        raise ValueError("M must be [d, d] and X0 [d, r]")
    if iters == 0:
        X, _ = np.linalg.qr(X)
    for _ in range(iters):
        Y = M @ X
        X, _ = np.linalg.qr(Y)
    B = X.T @ (M @ X)
    B = 0.5 * (B + B.T)
    theta, S = np.linalg.eigh(B)
    theta, S = theta[::-1], S[:, ::-1]
    U = X @ S
    Qhat = np.sqrt(np.maximum(theta, 0.0))[:, None] * U.T
    return np.ascontiguousarray(Qhat), theta.copy(), X


def build_W_power(Qc, X0, iters, lam, g=1):
    """Stacked queries -> update matrix W with the block power method in place of the SVD."""
    d = Qc.shape[1]
    M = gram(Qc)
    Qhat, theta, X = power_subspace(M, X0, iters)
    mats = update_matrices(Qhat, d, lam, g)
    mats.update({"Qhat": Qhat, "theta": theta, "X": X, "M": M})
    return mats
