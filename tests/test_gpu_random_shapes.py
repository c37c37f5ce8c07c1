"""GPU parity over seeded random shapes and launch plans.

The fixed cases elsewhere were chosen by hand, and hand-chosen shapes give most CTAs a single unit of
work: the paths a CTA takes for its second and later units (tiles that come through a tensor map instead
of being rotated in place, barrier phases that wrap, unit tables, split launches) then go untested.  Each
case here draws a batch shape, a head layout, a block length and the library's planning knobs (few CTAs,
so that every role of every CTA walks many units; a forced role split) from a seeded generator and runs
the whole path -- build, steps, full recompute, cached state, and the incremental build with its advances
-- against the fp64 oracle and against itself.  The knobs are the library's documented experiment
knobs, read when a context is created."""
import numpy as np
import pytest

from paper_2607_16339_b200 import binding
from paper_2607_16339_b200.workloads import small_workload

from test_gpu_parity import _run_points
from test_gpu_incremental import _run as _run_generation

pytestmark = pytest.mark.gpu

HEADS = [(2, 2), (4, 4), (4, 2), (6, 2), (8, 2), (8, 1), (14, 2), (3, 1), (12, 4)]


def draw_case(seed):
    rng = np.random.default_rng(7000 + seed)
    hq, hkv = HEADS[int(rng.integers(len(HEADS)))]
    block_len = int(rng.choice([16, 32, 48, 64]))
    batch = int(rng.integers(1, 5))
    prompts = tuple(int(x) for x in rng.choice([0, 3, 40, 95, 96, 130, 257, 390, 520], size=batch))
    n_blocks = int(rng.integers(2, 5))
    mode = int(rng.integers(3))      # 0: one bf16 plane (small scores), 1: split bf16 planes, 2: one fp16 plane
    plain = mode == 0
    wl_kw = dict(prompt_lens=prompts, gen_len=n_blocks * block_len, block_len=block_len, steps=int(rng.integers(1, 3)),
                 hq=hq, hkv=hkv, scale_mode="inv_sqrt_d" if plain else "per_head_u(0.5,2)")
    knobs = {}
    max_ctas = rng.choice([0, 0, 3, 7, 20])
    if max_ctas:
        knobs["LACACHE_MAX_CTAS"] = str(int(max_ctas))
    stream_ctas = rng.choice([0, 0, 1, 2])
    if stream_ctas:
        knobs["LACACHE_STREAM_CTAS"] = str(int(stream_ctas))
    if rng.integers(4) == 0:
        knobs["LACACHE_NO_QCOMP"] = "1"
    if rng.integers(4) == 0:
        knobs["LACACHE_DEEP_UNITS"] = str(int(rng.choice([1, 2, 5])))
    ctx_kw = dict(precision_mode=(binding.PRECISION_PLAIN, binding.PRECISION_SPLIT, binding.PRECISION_FP16)[mode],
                  cache_granularity=binding.GRANULARITY_TILE if rng.integers(3) == 0 else binding.GRANULARITY_TOKEN)
    return wl_kw, knobs, ctx_kw


@pytest.mark.parametrize("seed", range(64))
def test_random_shape_and_plan(seed, monkeypatch):
    wl_kw, knobs, ctx_kw = draw_case(seed)
    for k, v in knobs.items():
        monkeypatch.setenv(k, v)
    what = "seed %d: %r %r %r" % (seed, wl_kw, knobs, ctx_kw)
    try:
        _run_points(small_workload(name="random-%d" % seed, **wl_kw), "tc", seed=seed, **ctx_kw)
        if ctx_kw["cache_granularity"] == binding.GRANULARITY_TOKEN:
            _run_generation(small_workload(name="random-gen-%d" % seed, **wl_kw), seed=100 + seed,
                            precision_mode=ctx_kw["precision_mode"])
    except AssertionError as e:
        raise AssertionError("%s\n%s" % (what, e)) from e
    finally:
        for k in knobs:
            monkeypatch.delenv(k)
