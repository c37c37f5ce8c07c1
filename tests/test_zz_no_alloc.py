"""The allocation-free entry point against the context-based one.

Some callers of this library cannot allocate device memory (they run inside an
arena that owns the device heap, or in a section where cudaMalloc's implicit
synchronisation is not allowed), so they cannot create a context.
``lacache_full_recompute_static`` serves them from a fixed array inside the
library.  This file checks, through the C ABI, that it returns what
``lacache_full_recompute`` returns, on two calls in a row (the second call finds
the first call's leftovers in the shared array), and that it refuses sizes
beyond its fixed scratch.  It is named to be collected last.
"""
import numpy as np
import pytest
import torch

from paper_2607_16339_b200 import binding
from paper_2607_16339_b200.workloads import SyntheticSchedule, small_workload

from lacache_testlib import TOL_CACHED_VS_FULL, make_ctx, new_outputs, to_dev

pytestmark = pytest.mark.gpu

_set_up = [False]     # the first call on a device loads the library's device image (the fixed array with it)


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_static_entry_point_matches_context_entry_point(dtype):
    shapes = [dict(prompt_lens=(211,), gen_len=64, block_len=32, hq=4, hkv=2, d=128),
              dict(prompt_lens=(57,), gen_len=32, block_len=16, hq=2, hkv=2, d=64 if dtype == "fp32" else 128)]
    dt = binding.DTYPE_BF16 if dtype == "bf16" else binding.DTYPE_FP32
    for i, kw in enumerate(shapes):      # two calls in a row, different sizes: the array is shared
        wl = small_workload(dtype=dtype, steps=1, scale_mode="inv_sqrt_d" if dtype == "fp32" else "per_head_u(0.5,2)", **kw)
        sch = SyntheticSchedule(wl, seed=20 + i)
        q, k, v = (to_dev(a, wl) for a in (sch.q, sch.k, sch.v))
        ctx = make_ctx(wl, engine=binding.ENGINE_SIMT)
        ref, ref_lse = new_outputs(wl)
        ctx.full_recompute(q, k, v, ref, ref_lse)
        torch.cuda.synchronize()
        for rep in range(2):             # and the same size twice (the second finds its tables in place)
            out, lse = new_outputs(wl)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            binding.full_recompute_static(dt, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.rope_theta, q, k, v, out, lse)
            torch.cuda.synchronize()
            if _set_up[0]:
                assert torch.cuda.mem_get_info()[0] == free_before      # nothing was allocated on the device
            _set_up[0] = True
            assert torch.isfinite(out).all()
            assert (out - ref).abs().max().item() <= TOL_CACHED_VS_FULL[dtype]
            assert (lse - ref_lse).abs().max().item() <= 1e-5
        ctx.destroy()


def test_static_entry_point_rejects_oversize_and_bad_arguments():
    x = torch.zeros(16, 2, 128, dtype=torch.bfloat16, device="cuda")
    o = torch.zeros(16, 2, 128, device="cuda")
    lib = binding.load()
    import ctypes
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    # too many tokens / too many elements for the fixed scratch: refused before anything launches
    for n_tok, hq in ((4097, 2), (4096, 16)):
        st = lib.lacache_full_recompute_static(0, n_tok, hq, hq, 128, 1e4, 0.0, p(x), p(x), p(x), p(o), None, None)
        assert st == binding.ERR_SHAPE
        assert b"static scratch limit" in lib.lacache_last_error(None)
    assert lib.lacache_full_recompute_static(0, 16, 2, 2, 96, 1e4, 0.0, p(x), p(x), p(x), p(o), None, None) == binding.ERR_UNSUPPORTED
    assert lib.lacache_full_recompute_static(0, 16, 2, 2, 128, 1e4, 0.0, None, p(x), p(x), p(o), None, None) == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()
