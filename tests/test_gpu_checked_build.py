"""The bounds-checked build of the library (libsquat_checked.so, -DSQUAT_CHECKED): the key and value kernels test every
global, shared-memory and tensor-memory address they form, and the shared-memory windows of the matrix descriptors
they hand to the tensor core, against the buffer or region it belongs to; a violation sets SQUAT_FLAG_BOUNDS and the
access is skipped.  It stands in for a memory checker.  Small, ragged and strided cases run through it in a child
process (the library is chosen when the package is first used): no violation may be reported and every output must
equal, byte for byte, what the normal build produces in this process."""
import hashlib
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import squat_inputs as si

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
D = 128


def run_cases():
    """Runs the cases with whatever library the process has loaded; returns {case: [digest of every output, flags]}."""
    import paper_2503_24358_b200 as sq
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from parity import alloc_key_outputs, alloc_value_outputs, to_torch
    out = {}

    def digest(ts):
        torch.cuda.synchronize()
        return [hashlib.sha256(t.contiguous().cpu().numpy().tobytes()).hexdigest() for t in ts]

    cases = [  # (name, base config, batch, heads, tokens, bits, G, rank, meta16)
        ("dense f32 config 0", 0, 1, 8, 256, 2, 32, 32, False),
        ("dense ragged tiles", 1, 3, 3, 96, 2, 32, 32, False),
        ("dense one group per head", 1, 1, 5, 32, 4, 32, 16, False),
        ("dense G=64", 1, 1, 2, 192, 2, 64, 24, False),
        ("dense G=128 m16", 1, 5, 1, 128, 4, 128, 40, True),
        ("dense two images per round", 1, 1, 170, 64, 2, 32, 32, False),
        ("rank-r form", 1, 3, 2, 160, 2, 32, 8, False),
        ("rank-r form G=128 m16", 1, 2, 2, 256, 4, 128, 5, True),
        ("rank-r form f32 G=64", 0, 1, 3, 192, 2, 64, 3, False),
    ]
    for name, ci, B, H, T, bits, G, r, m16 in cases:
        cfg = si.get_config(ci).with_(batch=B, n_kv_heads=H, n_q_heads=H, n_tokens=T)
        s = sq.Subspace(H, D)
        sq.squat_get_device_status(clear=True)
        sq.squat_build_subspace(s, to_torch(si.gen_queries(cfg, n_tokens=max(T, 256)), cfg.dtype), r, cfg.lam, 1)
        k, v = to_torch(si.gen_keys(cfg), cfg.dtype), to_torch(si.gen_values(cfg), cfg.dtype)
        # outputs sit at a token offset of a longer cache: strided stores
        Tc, off = T + 2 * G, G
        kc, ks, kz = alloc_key_outputs(B, H, Tc, D, bits, G)
        vc, vs, vz = alloc_value_outputs(B, H, Tc, D, bits, G)
        for t in (kc, ks, kz, vc, vs, vz):
            t.zero_()
        if m16:
            ks, kz, vs, vz = (t.to(torch.float16) for t in (ks, kz, vs, vz))
        sq.squat_quantize_keys(s, k, bits, G, kc[:, :, off:], ks[:, :, off // G:], kz[:, :, off // G:],
                               out_stride_b=H * Tc, out_stride_h=Tc)
        sq.squat_quantize_values(v, bits, G, vc[:, :, off:], vs[:, :, off:], vz[:, :, off:], out_stride_b=H * Tc, out_stride_h=Tc)
        d = digest((kc, ks, kz, vc, vs, vz))
        out[name] = d + [int(sq.squat_get_device_status(clear=True))]
        s.close()
    return out


def test_checked_build_reports_no_violation_and_equals_the_normal_build():
    from paper_2503_24358_b200 import build as sq_build
    lib = sq_build.build(checked=True)
    env = dict(os.environ, SQUAT_LIBRARY=lib, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    code = ("import json, sys; sys.path.insert(0, %r); import test_gpu_checked_build as t; import paper_2503_24358_b200 as sq; "
            "assert sq.LIB_PATH.endswith('libsquat_checked.so'); assert sq.squat_checked_selftest(); print('RESULT ' + json.dumps(t.run_cases()))" % os.path.join(ROOT, "tests"))
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    checked = json.loads([ln for ln in r.stdout.splitlines() if ln.startswith("RESULT ")][-1][7:])
    import paper_2503_24358_b200 as sq
    assert sq.LIB_PATH.endswith("libsquat.so")
    with pytest.raises(sq.SquatError):
        sq.squat_checked_selftest()                       # the normal build has no checks to test
    normal = run_cases()
    assert set(checked) == set(normal)
    for name in normal:
        assert checked[name][-1] & sq.FLAG_BOUNDS == 0, (name, hex(checked[name][-1]))
        assert checked[name][-1] & sq.FLAG_DEVICE_TIMEOUT == 0, name
        assert checked[name][:-1] == normal[name][:-1], name
