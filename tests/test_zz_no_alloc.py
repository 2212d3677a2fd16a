"""GPU test of the allocation-free Gram entry point, squat_gram_static.

Who needs it: callers that cannot allocate device memory where they need this step -- code inside an
allocator or memory-pool callback, code running while the framework's allocator is frozen, or a process
whose device memory a serving engine has already claimed in full.  The entry keeps its intermediate
partial sums in a fixed array inside the library instead of cudaMalloc'ed scratch.

The check: through the C ABI, its output must equal what the existing entry (squat_build_subspace, whose
Gram stage uses scratch owned by the subspace handle) produces for the same queries, on two calls in a
row with different inputs -- the second, smaller call must not see anything the first left in the
shared array.  This file sorts last so that every other test has run before it.
"""
import numpy as np
import pytest
import torch

import squat_inputs as si
import paper_2503_24358_b200 as sq
from parity import to_torch

pytestmark = pytest.mark.gpu

REL_TOL = 1e-12          # same bound the subspace tests use for the Gram matrix (summation order differs)


def _reference_gram(cfg, q):
    s = sq.Subspace(cfg.n_kv_heads, 128)
    sq.squat_build_subspace(s, q, 8, 1e-3, 1)
    g = sq.squat_subspace_export(s, ("gram",))["gram"]
    s.close()
    return g


def test_gram_static_matches_the_allocating_entry_twice_in_a_row():
    first = si.get_config(1).with_(n_kv_heads=32, n_q_heads=32, n_tokens=1024)      # 32 heads, 2 chunks each
    second = si.get_config(2).with_(n_kv_heads=4, n_q_heads=16, n_tokens=160)       # GQA, fewer units, ragged rows
    third = si.get_config(0).with_(n_kv_heads=64, n_q_heads=64, n_tokens=96)        # float32 queries; 64 heads: every unit of the scratch, one chunk each
    for i, cfg in enumerate((first, second, third)):
        q = to_torch(si.gen_queries(cfg), cfg.dtype)
        out = torch.full((cfg.n_kv_heads, 128, 128), float("nan"), dtype=torch.float64, device="cuda")
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        free_before = torch.cuda.mem_get_info()[0]       # the driver's own count of free device memory: sees any cudaMalloc
        sq.squat_gram_static(q, cfg.n_kv_heads, out)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        if i > 0:                                        # (the very first call of a process may load the kernels' module)
            assert torch.cuda.mem_get_info()[0] == free_before
        got = out.cpu().numpy()
        ref = _reference_gram(cfg, q)
        assert np.isfinite(got).all()
        assert np.abs(got - ref).max() <= REL_TOL * np.abs(ref).max()
        assert np.array_equal(got, got.transpose(0, 2, 1))


def test_gram_static_rejects_sizes_beyond_its_scratch():
    q = torch.zeros((65, 64, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((65, 128, 128), dtype=torch.float64, device="cuda")
    n0 = sq.squat_kernel_launch_count()
    with pytest.raises(sq.SquatError) as e:
        sq.squat_gram_static(q, 65, out)                 # 65 KV heads > 64 units of scratch
    assert e.value.status == 3
    assert sq.squat_kernel_launch_count() == n0          # nothing was launched
