"""Thin ctypes binding of libsquat.so: argument marshalling only.

Every function has the name of the C entry point it calls (include/squat.h) and takes
torch tensors where the C function takes device pointers.  Nothing here computes: all
steps of the write path run in the library's CUDA kernels.  If the shared library is
missing or does not load, every call raises -- there is no fallback.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# SQUAT_LIBRARY selects another build of the same library (the bounds-checked one, libsquat_checked.so)
LIB_PATH = os.environ.get("SQUAT_LIBRARY") or os.path.join(_HERE, "libsquat.so")

SQUAT_F32, SQUAT_BF16 = 0, 1
SQUAT_KEYS, SQUAT_VALUES = 0, 1
FLAG_NONFINITE, FLAG_ZERO_RANGE, FLAG_NO_CONVERGE, FLAG_DEVICE_TIMEOUT, FLAG_BOUNDS = 1, 2, 4, 8, 16

EXPORTED_SYMBOLS = (
    "squat_subspace_create", "squat_subspace_destroy", "squat_build_subspace", "squat_subspace_export",
    "squat_subspace_import", "squat_subspace_eig_sweeps", "squat_quantize_keys", "squat_quantize_values", "squat_dequantize",
    "squat_write_path_workspace_bytes", "squat_write_path_host", "squat_get_device_status",
    "squat_kernel_launch_count", "squat_status_string", "squat_last_cuda_error", "squat_gram_static",
    "squat_decode_attention_workspace_bytes", "squat_decode_attention",
    "squat_rope_table_floats", "squat_rope_table_fill", "squat_decode_attention_pre_rope",
    "squat_decode_attention_ex", "squat_build_subspace_from_gram", "squat_build_subspace_power", "squat_write_path_host_ex", "squat_build_subspace_power_from_gram", "squat_quantize_keys_m16", "squat_quantize_values_m16", "squat_dequantize_m16",
    "squat_fp32_peak_probe", "squat_append_window_host", "squat_subspace_select_key_kernel", "squat_checked_selftest",
)

_lib = None


class SquatError(RuntimeError):
    def __init__(self, status, where):
        lib = _load()
        msg = lib.squat_status_string(status).decode()
        if status == 5:
            msg += " (" + lib.squat_last_cuda_error().decode() + ")"
        super().__init__(f"{where}: {msg} [status {status}]")
        self.status = status


def _load():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2503_24358_b200.build` "
                               "(there is no CPU fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        c = ctypes
        vp, i, ll, dbl = c.c_void_p, c.c_int, c.c_longlong, c.c_double
        lib.squat_subspace_create.argtypes = [i, i, c.POINTER(vp)]
        lib.squat_subspace_destroy.argtypes = [vp]
        lib.squat_build_subspace.argtypes = [vp, vp, i, i, i, ll, ll, i, dbl, i, vp]
        lib.squat_subspace_export.argtypes = [vp, vp, vp, vp, vp, vp]
        lib.squat_subspace_import.argtypes = [vp, vp, vp]
        lib.squat_subspace_eig_sweeps.argtypes = [vp, vp, vp]
        lib.squat_quantize_keys.argtypes = [vp, vp, i, i, i, i, i, ll, ll, ll, i, i, vp, vp, vp, ll, ll, vp]
        lib.squat_quantize_values.argtypes = [vp, i, i, i, i, i, ll, ll, ll, i, i, vp, vp, vp, ll, ll, vp]
        lib.squat_dequantize.argtypes = [i, vp, vp, vp, i, i, i, i, i, i, ll, ll, vp, i, vp]
        lib.squat_write_path_workspace_bytes.argtypes = [i] * 8
        lib.squat_write_path_workspace_bytes.restype = c.c_size_t
        lib.squat_write_path_host.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, dbl, i, i, i,
                                              vp, vp, vp, vp, vp, vp, vp, c.c_size_t, vp]
        lib.squat_write_path_host_ex.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, dbl, i, i, i,
                                                 vp, vp, vp, vp, vp, vp, i, vp, i, vp, c.c_size_t, vp]
        lib.squat_gram_static.argtypes = [vp, i, i, i, i, i, ll, ll, vp, vp]
        lib.squat_decode_attention_workspace_bytes.argtypes = [i, i, i]
        lib.squat_decode_attention_workspace_bytes.restype = c.c_size_t
        lib.squat_decode_attention.argtypes = [vp, i, i, i, i, i, vp, vp, vp, vp, vp, vp, i, ll, ll, i, i, vp, vp, i, i,
                                               c.c_float, vp, vp, c.c_size_t, vp]
        lib.squat_quantize_keys_m16.argtypes = lib.squat_quantize_keys.argtypes
        lib.squat_quantize_values_m16.argtypes = lib.squat_quantize_values.argtypes
        lib.squat_dequantize_m16.argtypes = lib.squat_dequantize.argtypes
        lib.squat_build_subspace_from_gram.argtypes = [vp, vp, i, dbl, i, vp]
        lib.squat_build_subspace_power.argtypes = [vp, vp, i, i, i, ll, ll, i, dbl, i, vp, ll, i, vp]
        lib.squat_build_subspace_power_from_gram.argtypes = [vp, vp, i, dbl, i, vp, ll, i, vp]
        lib.squat_rope_table_floats.argtypes = [i]
        lib.squat_rope_table_floats.restype = c.c_size_t
        lib.squat_rope_table_fill.argtypes = [dbl, i, i, vp]
        lib.squat_decode_attention_pre_rope.argtypes = [vp, i, i, i, i, i, vp, vp, vp, vp, vp, vp, i, ll, ll, i, i, vp, vp, i, i,
                                                        c.c_float, vp, i, ll, vp, vp, c.c_size_t, vp]
        lib.squat_decode_attention_ex.argtypes = [vp, i, i, i, i, i, vp, vp, vp, vp, vp, vp, i, i, ll, ll, i, i, vp, vp, i, i,
                                                  c.c_float, vp, i, ll, vp, vp, c.c_size_t, vp]
        lib.squat_append_window_host.argtypes = [vp, vp, vp, i, i, i, i, i, i, i, vp, vp, vp, vp, vp, vp, i, vp, c.c_size_t, vp]
        lib.squat_subspace_select_key_kernel.argtypes = [vp, i, c.POINTER(i)]
        lib.squat_checked_selftest.argtypes = [vp, c.POINTER(i)]
        lib.squat_fp32_peak_probe.argtypes = [i, i, vp, c.POINTER(ll), vp]
        lib.squat_get_device_status.argtypes = [vp, c.POINTER(c.c_uint), i]
        lib.squat_kernel_launch_count.restype = c.c_ulonglong
        lib.squat_status_string.argtypes = [i]
        lib.squat_status_string.restype = c.c_char_p
        lib.squat_last_cuda_error.restype = c.c_char_p
        _lib = lib
    return _lib


def _check(status, where):
    if status != 0:
        raise SquatError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SQUAT_F32
    if t.dtype == torch.bfloat16:
        return SQUAT_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream(stream=None):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dev(t: torch.Tensor, name: str):
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


class Subspace:
    """Owner of a squat_subspace handle (the per-layer update matrices of every KV head)."""

    def __init__(self, n_kv_heads: int, head_dim: int = 128):
        self._h = ctypes.c_void_p()
        self.n_kv_heads, self.head_dim = n_kv_heads, head_dim
        _check(_load().squat_subspace_create(n_kv_heads, head_dim, ctypes.byref(self._h)), "squat_subspace_create")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            _load().squat_subspace_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self):
        return self._h


def squat_build_subspace(s: Subspace, q: torch.Tensor, rank_r: int, lam: float, block_g: int = 1, stream=None):
    """q: [n_q_heads, n_tokens, d] prompt queries of the first sample (last dim contiguous)."""
    if q.dim() != 3 or q.stride(2) != 1 or q.shape[2] != s.head_dim:
        raise ValueError("q must be [n_q_heads, n_tokens, head_dim] with contiguous last dim")
    _check(_load().squat_build_subspace(s.handle, _dev(q, "q"), _dtype_code(q), q.shape[0], q.shape[1],
                                        q.stride(0), q.stride(1), rank_r, float(lam), block_g, _stream(stream)),
           "squat_build_subspace")


def squat_subspace_export(s: Subspace, want=("W",), stream=None):
    """Returns a dict of numpy arrays: W [H,d,d] f32, gram [H,d,d] f64, eigval [H,d], eigvec [H,d,d]."""
    import numpy as np
    H, d = s.n_kv_heads, s.head_dim
    bufs = {
        "W": np.empty((H, d, d), np.float32) if "W" in want else None,
        "gram": np.empty((H, d, d), np.float64) if "gram" in want else None,
        "eigval": np.empty((H, d), np.float64) if "eigval" in want else None,
        "eigvec": np.empty((H, d, d), np.float64) if "eigvec" in want else None,
    }
    ptr = lambda a: None if a is None else a.ctypes.data_as(ctypes.c_void_p)
    _check(_load().squat_subspace_export(s.handle, _stream(stream), ptr(bufs["W"]), ptr(bufs["gram"]),
                                         ptr(bufs["eigval"]), ptr(bufs["eigvec"])), "squat_subspace_export")
    return {k: v for k, v in bufs.items() if v is not None}


def squat_subspace_import(s: Subspace, W, stream=None):
    """W: numpy [H, d, d] float32, row j' column j (block strictly lower triangular)."""
    import numpy as np
    W = np.ascontiguousarray(W, dtype=np.float32)
    if W.shape != (s.n_kv_heads, s.head_dim, s.head_dim):
        raise ValueError("W must be [n_kv_heads, d, d]")
    _check(_load().squat_subspace_import(s.handle, W.ctypes.data_as(ctypes.c_void_p), _stream(stream)),
           "squat_subspace_import")


def squat_subspace_eig_sweeps(s: Subspace, stream=None):
    """Jacobi sweeps the eigensolver ran for each head in the last build (diagnostic)."""
    import numpy as np
    out = np.zeros(s.n_kv_heads, dtype=np.int32)
    _check(_load().squat_subspace_eig_sweeps(s.handle, _stream(stream), out.ctypes.data_as(ctypes.c_void_p)),
           "squat_subspace_eig_sweeps")
    return out


def _check_bhtd(x, name):
    if x.dim() != 4 or x.stride(3) != 1:
        raise ValueError(f"{name} must be [batch, heads, tokens, head_dim] with contiguous last dim")


def _meta16(scales: torch.Tensor, zeros: torch.Tensor) -> bool:
    """float16 scale / zero tensors select the entry points of the 16-bit-metadata cache."""
    if scales.dtype != zeros.dtype or scales.dtype not in (torch.float32, torch.float16):
        raise ValueError("scales and zeros must both be float32 or both float16")
    return scales.dtype == torch.float16


def squat_quantize_keys(s: Subspace, k: torch.Tensor, bits: int, group_size: int, codes: torch.Tensor,
                        scales: torch.Tensor, zeros: torch.Tensor, out_stride_b: int = None,
                        out_stride_h: int = None, stream=None):
    """k [B,H,T,d] -> codes (uint8), scales, zeros (float32, or float16 for the 16-bit-metadata cache), written in place.

    out strides are in tokens; by default the outputs are dense [B,H,T,...]."""
    _check_bhtd(k, "k")
    B, H, T, d = k.shape
    osh = T if out_stride_h is None else out_stride_h
    osb = H * osh if out_stride_b is None else out_stride_b
    fn = _load().squat_quantize_keys_m16 if _meta16(scales, zeros) else _load().squat_quantize_keys
    _check(fn(s.handle, _dev(k, "k"), _dtype_code(k), B, H, T, d, k.stride(0), k.stride(1),
                                       k.stride(2), bits, group_size, _dev(codes, "codes"), _dev(scales, "scales"),
                                       _dev(zeros, "zeros"), osb, osh, _stream(stream)), "squat_quantize_keys")


def squat_quantize_values(v: torch.Tensor, bits: int, group_size: int, codes: torch.Tensor, scales: torch.Tensor,
                          zeros: torch.Tensor, out_stride_b: int = None, out_stride_h: int = None, stream=None):
    _check_bhtd(v, "v")
    B, H, T, d = v.shape
    osh = T if out_stride_h is None else out_stride_h
    osb = H * osh if out_stride_b is None else out_stride_b
    fn = _load().squat_quantize_values_m16 if _meta16(scales, zeros) else _load().squat_quantize_values
    _check(fn(_dev(v, "v"), _dtype_code(v), B, H, T, d, v.stride(0), v.stride(1),
                                         v.stride(2), bits, group_size, _dev(codes, "codes"), _dev(scales, "scales"),
                                         _dev(zeros, "zeros"), osb, osh, _stream(stream)), "squat_quantize_values")


def squat_dequantize(kind: int, codes: torch.Tensor, scales: torch.Tensor, zeros: torch.Tensor, batch: int,
                     n_kv_heads: int, n_tokens: int, head_dim: int, bits: int, group_size: int, out: torch.Tensor,
                     in_stride_b: int = None, in_stride_h: int = None, stream=None):
    ish = n_tokens if in_stride_h is None else in_stride_h
    isb = n_kv_heads * ish if in_stride_b is None else in_stride_b
    if not out.is_contiguous():
        raise ValueError("out must be contiguous")
    fn = _load().squat_dequantize_m16 if _meta16(scales, zeros) else _load().squat_dequantize
    _check(fn(kind, _dev(codes, "codes"), _dev(scales, "scales"), _dev(zeros, "zeros"), batch,
                                    n_kv_heads, n_tokens, head_dim, bits, group_size, isb, ish, _dev(out, "out"),
                                    _dtype_code(out), _stream(stream)), "squat_dequantize")


def squat_write_path_workspace_bytes(dtype: torch.dtype, batch, n_q_heads, n_kv_heads, n_tokens, head_dim, bits,
                                     group_size) -> int:
    code = SQUAT_F32 if dtype == torch.float32 else SQUAT_BF16
    return int(_load().squat_write_path_workspace_bytes(code, batch, n_q_heads, n_kv_heads, n_tokens, head_dim, bits,
                                                        group_size))


def squat_write_path_host(s: Subspace, q, k, v, rank_r, lam, block_g, bits, group_size, k_codes, k_scales, k_zeros,
                          v_codes, v_scales, v_zeros, workspace: torch.Tensor, stream=None, start_block=None,
                          power_iters: int = 2):
    """q, k, v and the six outputs are HOST tensors (pinned for speed); workspace is a CUDA uint8 tensor.  float16
    scale / zero tensors select the 16-bit metadata variant (all four of them then); a HOST float64 start_block
    [d, rank_r] selects step 1 by the block power method with power_iters multiplications."""
    for name, t in (("q", q), ("k", k), ("v", v), ("k_codes", k_codes), ("k_scales", k_scales), ("k_zeros", k_zeros),
                    ("v_codes", v_codes), ("v_scales", v_scales), ("v_zeros", v_zeros)):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous host tensor")
    B, H, T, d = k.shape
    hp = lambda t: ctypes.c_void_p(t.data_ptr())
    meta = (k_scales, k_zeros, v_scales, v_zeros)
    m16 = all(t.dtype == torch.float16 for t in meta)
    if not m16 and not all(t.dtype == torch.float32 for t in meta):
        raise ValueError("scales and zero-points must be all float32 or all float16")
    if not m16 and start_block is None:
        _check(_load().squat_write_path_host(s.handle, hp(q), hp(k), hp(v), _dtype_code(k), B, q.shape[0], H, T, d, rank_r,
                                             float(lam), block_g, bits, group_size, hp(k_codes), hp(k_scales), hp(k_zeros),
                                             hp(v_codes), hp(v_scales), hp(v_zeros), _dev(workspace, "workspace"),
                                             workspace.numel() * workspace.element_size(), _stream(stream)),
               "squat_write_path_host")
        return
    x0 = None
    if start_block is not None:
        if start_block.is_cuda or start_block.dtype != torch.float64 or not start_block.is_contiguous() or \
                tuple(start_block.shape) != (d, rank_r):
            raise ValueError("start_block must be a contiguous host float64 tensor [d, rank_r]")
        x0 = hp(start_block)
    _check(_load().squat_write_path_host_ex(s.handle, hp(q), hp(k), hp(v), _dtype_code(k), B, q.shape[0], H, T, d, rank_r,
                                            float(lam), block_g, bits, group_size, hp(k_codes), hp(k_scales), hp(k_zeros),
                                            hp(v_codes), hp(v_scales), hp(v_zeros), int(m16), x0, int(power_iters),
                                            _dev(workspace, "workspace"),
                                            workspace.numel() * workspace.element_size(), _stream(stream)),
           "squat_write_path_host_ex")


def squat_append_window_host(s: Subspace, k, v, bits, group_size, k_codes, k_scales, k_zeros, v_codes, v_scales, v_zeros,
                             workspace: torch.Tensor, stream=None):
    """One decode window from HOST tensors (pinned for speed): k, v [B, H, T, d] go up, are quantized with the update
    matrices the handle holds, and the six outputs come back.  float16 scale / zero tensors select 16-bit metadata;
    workspace: CUDA uint8 tensor of squat_write_path_workspace_bytes(dtype, B, H, H, T, d, bits, group_size)."""
    for name, t in (("k", k), ("v", v), ("k_codes", k_codes), ("k_scales", k_scales), ("k_zeros", k_zeros),
                    ("v_codes", v_codes), ("v_scales", v_scales), ("v_zeros", v_zeros)):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous host tensor")
    B, H, T, d = k.shape
    hp = lambda t: ctypes.c_void_p(t.data_ptr())
    meta = (k_scales, k_zeros, v_scales, v_zeros)
    m16 = all(t.dtype == torch.float16 for t in meta)
    if not m16 and not all(t.dtype == torch.float32 for t in meta):
        raise ValueError("scales and zero-points must be all float32 or all float16")
    _check(_load().squat_append_window_host(s.handle, hp(k), hp(v), _dtype_code(k), B, H, T, d, bits, group_size,
                                            hp(k_codes), hp(k_scales), hp(k_zeros), hp(v_codes), hp(v_scales), hp(v_zeros),
                                            int(m16), _dev(workspace, "workspace"),
                                            workspace.numel() * workspace.element_size(), _stream(stream)),
           "squat_append_window_host")


def squat_subspace_select_key_kernel(s: "Subspace", prefer_dense: bool = False) -> int:
    """Chooses the kernel squat_quantize_keys runs on this handle (True: always the dense one; False: the rank-r form
    where the last build prepared it).  Returns the rank the rank-r form is prepared for (0: not prepared)."""
    r = ctypes.c_int(0)
    _check(_load().squat_subspace_select_key_kernel(s.handle, 1 if prefer_dense else 0, ctypes.byref(r)),
           "squat_subspace_select_key_kernel")
    return int(r.value)


def squat_checked_selftest(stream=None) -> bool:
    """True iff the loaded library is the bounds-checked build and its check caught a one-byte overrun (formed, never
    accessed); raises SquatError (status 3) on the normal build."""
    det = ctypes.c_int(0)
    _check(_load().squat_checked_selftest(_stream(stream), ctypes.byref(det)), "squat_checked_selftest")
    return bool(det.value)


def squat_fp32_peak_probe(packed: bool, iters: int, sink: torch.Tensor, stream=None) -> int:
    """Launches the FP32 multiply-add probe kernel (a measurement aid; time it with CUDA events around this call).
    sink: a CUDA float32 tensor of at least one element.  Returns the floating-point operations of the launch."""
    flops = ctypes.c_longlong(0)
    _check(_load().squat_fp32_peak_probe(1 if packed else 0, int(iters), _dev(sink, "sink"), ctypes.byref(flops),
                                         _stream(stream)), "squat_fp32_peak_probe")
    return int(flops.value)


def squat_gram_static(q: torch.Tensor, n_kv_heads: int, gram_out: torch.Tensor, stream=None):
    """Gram matrices of the stacked queries into gram_out [n_kv_heads, d, d] (float64, CUDA) without any
    allocation: for callers that cannot call cudaMalloc (allocator callbacks, frozen allocators, processes
    whose device memory is fully handed out).  At most 64 KV heads; calls must not overlap on the GPU."""
    if q.dim() != 3 or q.stride(2) != 1:
        raise ValueError("q must be [n_q_heads, n_tokens, head_dim] with contiguous last dim")
    if gram_out.dtype != torch.float64 or not gram_out.is_contiguous():
        raise ValueError("gram_out must be a contiguous float64 tensor")
    _check(_load().squat_gram_static(_dev(q, "q"), _dtype_code(q), q.shape[0], n_kv_heads, q.shape[1], q.shape[2],
                                     q.stride(0), q.stride(1), _dev(gram_out, "gram_out"), _stream(stream)),
           "squat_gram_static")


def squat_build_subspace_from_gram(s: "Subspace", gram: torch.Tensor, rank_r: int, lam: float, block_g: int = 1, stream=None):
    """Eigen-decomposition and update matrices from Gram matrices [n_kv_heads, d, d] (float64, CUDA) the caller has
    summed over the prompt's tokens, e.g. across the ranks that hold them."""
    if gram.dtype != torch.float64 or not gram.is_contiguous():
        raise ValueError("gram must be a contiguous float64 tensor")
    _check(_load().squat_build_subspace_from_gram(s.handle, _dev(gram, "gram"), int(rank_r), ctypes.c_double(lam),
                                                  int(block_g), _stream(stream)), "squat_build_subspace_from_gram")


def squat_build_subspace_power(s: "Subspace", q: torch.Tensor, rank_r: int, lam: float, start_block: torch.Tensor,
                               iters: int = 2, block_g: int = 1, stream=None):
    """Step 1 with the block power method: q as for squat_build_subspace; start_block [d, rank_r] (one block for all
    heads) or [n_kv_heads, d, rank_r], float64, CUDA, contiguous; iters multiplications by the Gram matrix."""
    if q.dim() != 3 or q.stride(2) != 1 or q.shape[2] != s.head_dim:
        raise ValueError("q must be [n_q_heads, n_tokens, head_dim] with contiguous last dim")
    ptr, stride_h = _start_block_args(s, start_block, rank_r)
    _check(_load().squat_build_subspace_power(s.handle, _dev(q, "q"), _dtype_code(q), q.shape[0], q.shape[1],
                                              q.stride(0), q.stride(1), int(rank_r), ctypes.c_double(lam), int(block_g),
                                              ptr, stride_h, int(iters), _stream(stream)),
           "squat_build_subspace_power")


def token_shard(n_tokens: int, rank: int, world: int, multiple: int = 32):
    """[start, stop) of the prompt tokens rank `rank` of `world` holds when a prompt is spread over ranks: contiguous,
    boundaries at multiples of `multiple` (the quantization group size, so that no group straddles two ranks), sizes as
    even as that allows.  n_tokens must be a multiple of `multiple`."""
    if n_tokens % multiple or not 0 <= rank < world:
        raise ValueError("n_tokens must be a multiple of the group size and 0 <= rank < world")
    units = n_tokens // multiple
    lo = units * rank // world
    hi = units * (rank + 1) // world
    return lo * multiple, hi * multiple


def _start_block_args(s: "Subspace", start_block: torch.Tensor, rank_r: int):
    if start_block.dtype != torch.float64 or not start_block.is_contiguous():
        raise ValueError("start_block must be a contiguous float64 tensor")
    if tuple(start_block.shape) == (s.head_dim, rank_r):
        stride_h = 0
    elif tuple(start_block.shape) == (s.n_kv_heads, s.head_dim, rank_r):
        stride_h = s.head_dim * rank_r
    else:
        raise ValueError("start_block must be [d, rank_r] or [n_kv_heads, d, rank_r]")
    return (_dev(start_block, "start_block") if rank_r > 0 else None), stride_h


def squat_build_subspace_power_from_gram(s: "Subspace", gram: torch.Tensor, rank_r: int, lam: float,
                                         start_block: torch.Tensor, iters: int = 2, block_g: int = 1, stream=None):
    """The block power build from Gram matrices [n_kv_heads, d, d] (float64, CUDA) the caller has summed over the
    prompt's tokens; start_block as for squat_build_subspace_power."""
    if gram.dtype != torch.float64 or not gram.is_contiguous():
        raise ValueError("gram must be a contiguous float64 tensor")
    ptr, stride_h = _start_block_args(s, start_block, rank_r)
    _check(_load().squat_build_subspace_power_from_gram(s.handle, _dev(gram, "gram"), int(rank_r), ctypes.c_double(lam),
                                                        int(block_g), ptr, stride_h, int(iters), _stream(stream)),
           "squat_build_subspace_power_from_gram")


def squat_build_subspace_sharded(s: "Subspace", q_local: torch.Tensor, rank_r: int, lam: float, block_g: int = 1,
                                 gram_buf: torch.Tensor = None, group=None, stream=None, start_block: torch.Tensor = None,
                                 power_iters: int = 2):
    """Step 1 for a prompt whose tokens are spread over the ranks of a torch.distributed group: Gram matrices of
    the local tokens (q_local [n_q_heads, local_tokens, d]; a rank may hold none), one all-reduce (sum) of
    n_kv_heads * d * d float64, then the eigen-decomposition (or, with a start_block every rank passes alike, the
    block power iteration) and the update matrices on every rank.  Without an initialised process group this is the
    single-GPU build through the same two calls.

    The whole sequence runs on `stream` (torch's current stream when None): the collective is issued with that stream
    current, so it starts after the Gram kernels and the build starts after it.  Limits inherited from
    squat_gram_static: at most 64 KV heads, and one shared scratch array in the library -- two sharded builds (two
    layers, say) must not overlap on the GPU, so do not run them on different streams at the same time."""
    import torch.distributed as dist
    H = s.n_kv_heads
    if q_local.dim() != 3 or q_local.shape[0] % H != 0:
        raise ValueError("q_local must be [n_q_heads, local_tokens, d] with n_q_heads a multiple of the handle's KV heads")
    if stream is None:
        stream = torch.cuda.current_stream()
    with torch.cuda.stream(stream):
        if gram_buf is None:
            gram_buf = torch.empty((H, q_local.shape[2], q_local.shape[2]), dtype=torch.float64, device=q_local.device)
        if q_local.shape[1] > 0:
            squat_gram_static(q_local, H, gram_buf, stream)
        else:
            gram_buf.zero_()
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
            dist.all_reduce(gram_buf, op=dist.ReduceOp.SUM, group=group)
        if start_block is not None:
            squat_build_subspace_power_from_gram(s, gram_buf, rank_r, lam, start_block, power_iters, block_g, stream)
        else:
            squat_build_subspace_from_gram(s, gram_buf, rank_r, lam, block_g, stream)
    return gram_buf


def squat_decode_attention_workspace_bytes(batch: int, n_q_heads: int, n_tokens: int) -> int:
    return int(_load().squat_decode_attention_workspace_bytes(batch, n_q_heads, n_tokens))


def squat_decode_attention(q: torch.Tensor, k_codes, k_scales, k_zeros, v_codes, v_scales, v_zeros, n_kv_heads: int,
                           n_tokens: int, bits: int, group_size: int, out: torch.Tensor, workspace: torch.Tensor,
                           k_res: torch.Tensor = None, v_res: torch.Tensor = None, softmax_scale: float = 0.0,
                           cache_stride_b: int = None, cache_stride_h: int = None, stream=None):
    """One decode step of attention over the packed cache.  q [B, Hq, d]; the cache tensors as the write path
    produced them; k_res / v_res [B, H, R, d] the full-precision residual buffer (optional); out [B, Hq, d]
    float32; workspace a CUDA uint8 tensor of squat_decode_attention_workspace_bytes(...)."""
    if q.dim() != 3 or not q.is_contiguous() or not out.is_contiguous() or out.dtype != torch.float32:
        raise ValueError("q must be contiguous [batch, n_q_heads, d]; out contiguous float32")
    B, Hq, d = q.shape
    csh = n_tokens if cache_stride_h is None else cache_stride_h
    csb = n_kv_heads * csh if cache_stride_b is None else cache_stride_b
    n_res = 0 if k_res is None else k_res.shape[2]
    if n_res and (not k_res.is_contiguous() or not v_res.is_contiguous() or k_res.dtype != v_res.dtype):
        raise ValueError("k_res and v_res must be contiguous [batch, n_kv_heads, n_res, d] of one dtype")
    opt = lambda t, n: _dev(t, n) if t is not None and t.numel() else None
    if k_scales is not None and k_scales.dtype == torch.float16:         # a cache with 16-bit scales and zero-points
        for t in (k_zeros, v_scales, v_zeros):
            if t.dtype != torch.float16:
                raise ValueError("scales and zero-points must all be float16 or all float32")
        _check(_load().squat_decode_attention_ex(
            _dev(q, "q"), _dtype_code(q), B, Hq, n_kv_heads, d, opt(k_codes, "k_codes"), opt(k_scales, "k_scales"),
            opt(k_zeros, "k_zeros"), opt(v_codes, "v_codes"), opt(v_scales, "v_scales"), opt(v_zeros, "v_zeros"), 1, n_tokens,
            csb, csh, bits, group_size, opt(k_res, "k_res"), opt(v_res, "v_res"), _dtype_code(k_res) if n_res else SQUAT_F32,
            n_res, float(softmax_scale), None, 0, 0, _dev(out, "out"), _dev(workspace, "workspace"),
            workspace.numel() * workspace.element_size(), _stream(stream)), "squat_decode_attention_ex")
        return
    _check(_load().squat_decode_attention(_dev(q, "q"), _dtype_code(q), B, Hq, n_kv_heads, d, opt(k_codes, "k_codes"),
                                          opt(k_scales, "k_scales"), opt(k_zeros, "k_zeros"), opt(v_codes, "v_codes"),
                                          opt(v_scales, "v_scales"), opt(v_zeros, "v_zeros"), n_tokens, csb, csh, bits,
                                          group_size, opt(k_res, "k_res"), opt(v_res, "v_res"),
                                          _dtype_code(k_res) if n_res else SQUAT_F32, n_res, float(softmax_scale),
                                          _dev(out, "out"), _dev(workspace, "workspace"),
                                          workspace.numel() * workspace.element_size(), _stream(stream)),
           "squat_decode_attention")


def squat_rope_table(n_positions: int, base: float = 10000.0, head_dim: int = 128) -> torch.Tensor:
    """The rotary tables squat_decode_attention_pre_rope reads, as a CPU float32 tensor (the caller moves it to the
    device): filled by the library on the host in float64."""
    lib = _load()
    lib.squat_rope_table_floats.restype = ctypes.c_size_t
    n = int(lib.squat_rope_table_floats(int(n_positions)))
    t = torch.empty(n, dtype=torch.float32)
    _check(lib.squat_rope_table_fill(ctypes.c_double(base), int(head_dim), int(n_positions),
                                     ctypes.c_void_p(t.data_ptr())), "squat_rope_table_fill")
    return t


def squat_decode_attention_pre_rope(q: torch.Tensor, k_codes, k_scales, k_zeros, v_codes, v_scales, v_zeros,
                                    n_kv_heads: int, n_tokens: int, bits: int, group_size: int, out: torch.Tensor,
                                    workspace: torch.Tensor, rope_table: torch.Tensor, table_positions: int,
                                    first_pos: int = 0, k_res: torch.Tensor = None, v_res: torch.Tensor = None,
                                    softmax_scale: float = 0.0, cache_stride_b: int = None, cache_stride_h: int = None,
                                    stream=None):
    """squat_decode_attention over a cache whose keys (and residual keys) were stored before the rotary position
    embedding: cached token t sits at position first_pos + t.  rope_table: squat_rope_table(table_positions) on the
    device."""
    if q.dim() != 3 or not q.is_contiguous() or not out.is_contiguous() or out.dtype != torch.float32:
        raise ValueError("q must be contiguous [batch, n_q_heads, d]; out contiguous float32")
    if rope_table.dtype != torch.float32 or not rope_table.is_contiguous():
        raise ValueError("rope_table must be a contiguous float32 tensor")
    B, Hq, d = q.shape
    csh = n_tokens if cache_stride_h is None else cache_stride_h
    csb = n_kv_heads * csh if cache_stride_b is None else cache_stride_b
    n_res = 0 if k_res is None else k_res.shape[2]
    if n_res and (not k_res.is_contiguous() or not v_res.is_contiguous() or k_res.dtype != v_res.dtype):
        raise ValueError("k_res and v_res must be contiguous [batch, n_kv_heads, n_res, d] of one dtype")
    opt = lambda t, n: _dev(t, n) if t is not None and t.numel() else None
    if k_scales is not None and k_scales.dtype == torch.float16:         # a cache with 16-bit scales and zero-points
        _check(_load().squat_decode_attention_ex(
            _dev(q, "q"), _dtype_code(q), B, Hq, n_kv_heads, d, opt(k_codes, "k_codes"), opt(k_scales, "k_scales"),
            opt(k_zeros, "k_zeros"), opt(v_codes, "v_codes"), opt(v_scales, "v_scales"), opt(v_zeros, "v_zeros"), 1, n_tokens,
            csb, csh, bits, group_size, opt(k_res, "k_res"), opt(v_res, "v_res"), _dtype_code(k_res) if n_res else SQUAT_F32,
            n_res, float(softmax_scale), _dev(rope_table, "rope_table"), int(table_positions), int(first_pos),
            _dev(out, "out"), _dev(workspace, "workspace"), workspace.numel() * workspace.element_size(), _stream(stream)),
            "squat_decode_attention_ex")
        return
    _check(_load().squat_decode_attention_pre_rope(
        _dev(q, "q"), _dtype_code(q), B, Hq, n_kv_heads, d, opt(k_codes, "k_codes"), opt(k_scales, "k_scales"),
        opt(k_zeros, "k_zeros"), opt(v_codes, "v_codes"), opt(v_scales, "v_scales"), opt(v_zeros, "v_zeros"), n_tokens,
        ctypes.c_longlong(csb), ctypes.c_longlong(csh), bits, group_size, opt(k_res, "k_res"), opt(v_res, "v_res"),
        _dtype_code(k_res) if n_res else SQUAT_F32, n_res, ctypes.c_float(softmax_scale), _dev(rope_table, "rope_table"),
        int(table_positions), ctypes.c_longlong(first_pos), _dev(out, "out"), _dev(workspace, "workspace"),
        ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)), "squat_decode_attention_pre_rope")


def squat_get_device_status(clear: bool = True, stream=None) -> int:
    flags = ctypes.c_uint(0)
    _check(_load().squat_get_device_status(_stream(stream), ctypes.byref(flags), 1 if clear else 0),
           "squat_get_device_status")
    return flags.value


def squat_kernel_launch_count() -> int:
    return int(_load().squat_kernel_launch_count())
