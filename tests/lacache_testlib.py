"""Helpers shared by the GPU parity tests (marshalling and comparison only)."""
import numpy as np
import torch

import oracle
from paper_2607_16339_b200 import binding
from paper_2607_16339_b200.workloads import SyntheticSchedule

TOL = {"bf16": (2e-2, 2e-3), "fp32": (1e-5, 1e-5)}   # (max abs, mean abs) vs the fp64 oracle
TOL_CACHED_VS_FULL = {"bf16": 1e-3, "fp32": 1e-5}     # GPU cached path vs GPU full recompute


def torch_dtype(wl):
    return torch.bfloat16 if wl.dtype == "bf16" else torch.float32


def to_dev(a, wl):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda().to(torch_dtype(wl)).contiguous()


def advance_to_block(sch, b):
    """Bring the full arrays to the state at the start of block b: every
    earlier block holds its last draw."""
    wl = sch.wl
    for bb in range(b):
        sch.begin_block(bb)
        sch.draw_step(bb, wl.steps_per_block)
    return sch.begin_block(b)


def sample_rows(wl, sch, b, n_fixed=192, seed=0):
    """All block rows, rows next to tile / block / sequence edges, and a seeded
    sample of fixed rows."""
    cu = wl.cu_seqlens
    rows = set(int(r) for r in sch.block_rows(b))
    for s in range(wl.batch):
        lo, hi = int(cu[s]), int(cu[s + 1])
        bs = lo + wl.prompt_lens[s] + b * wl.block_len
        for e in (lo, hi - 1, bs - 1, bs + wl.block_len, lo + 127, lo + 128, hi - 2):
            if lo <= e < hi:
                rows.add(e)
    rng = np.random.default_rng(seed)
    rows.update(int(r) for r in rng.choice(wl.total_tokens, size=min(n_fixed, wl.total_tokens), replace=False))
    return np.array(sorted(rows), dtype=np.int32)


def check_against_oracle(wl, sch, out, lse, rows=None, what=""):
    scale = wl.head_dim ** -0.5
    ref, rlse = oracle.attention(sch.q, sch.k, sch.v, wl.cu_seqlens, wl.rope_theta, scale, rows=rows)
    o = out.detach().cpu().numpy().astype(np.float64)
    ls = lse.detach().cpu().numpy().astype(np.float64)
    if rows is not None:
        o, ls = o[rows], ls[rows]
    assert np.isfinite(o).all(), what
    err = np.abs(o - ref)
    tmax, tmean = TOL[wl.dtype]
    assert err.max() <= tmax, "%s: max abs err %.4g > %.4g" % (what, err.max(), tmax)
    assert err.mean() <= tmean, "%s: mean abs err %.4g > %.4g" % (what, err.mean(), tmean)
    lerr = np.abs(ls - rlse).max()
    assert lerr <= max(tmax, 1e-4), "%s: lse err %.4g" % (what, lerr)
    return err.max(), err.mean()


def make_ctx(wl, **kw):
    return binding.Context.from_workload(wl, **kw)


def new_outputs(wl):
    T = wl.total_tokens
    out = torch.full((T, wl.n_q_heads, wl.head_dim), float("nan"), device="cuda")
    lse = torch.full((T, wl.n_q_heads), float("nan"), device="cuda")
    return out, lse
