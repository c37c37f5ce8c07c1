"""GPU parity tests of the tile-granular variant (Algorithm 1 as printed: the Q_overlap / K_overlap
predicates are taken per tile, and only key tiles that lie wholly in the fixed set are cached).

`out` and `lse` have the same definition as with token-granular caching, so the oracle is the same
full-sequence attention; what differs is WHAT is cached, which the state test below checks against the
oracle's Eq. 2-6 state over the tile-level key set.  Tiles are 128 tokens, counted from the start of
each sequence."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_16339_b200 import binding
from paper_2607_16339_b200.workloads import WORKLOADS, SyntheticSchedule, parity_points, small_workload

from lacache_testlib import advance_to_block, make_ctx, new_outputs, sample_rows, to_dev
from test_gpu_parity import SMALL, _run_points

pytestmark = pytest.mark.gpu

TILE = 128


def overlap_mask(wl, b):
    """1 for every token of a tile that overlaps block b of its sequence (derived here, independently of
    the library: tiles of 128 tokens from the start of the sequence, the last one clipped)."""
    cu = wl.cu_seqlens
    mask = np.zeros(wl.total_tokens, dtype=np.int32)
    for s, P in enumerate(wl.prompt_lens):
        n = int(cu[s + 1] - cu[s])
        first, last = P + b * wl.block_len, P + (b + 1) * wl.block_len - 1     # positions of the block
        lo, hi = (first // TILE) * TILE, min(n, (last // TILE + 1) * TILE)
        mask[cu[s] + lo:cu[s] + hi] = 1
    return mask


@pytest.mark.parametrize("case", sorted(SMALL))
def test_small_cases_tile_granular(case):
    wl = small_workload(name=case, dtype="bf16", d=128, **SMALL[case])
    _run_points(wl, "tc", seed=5, cache_granularity=binding.GRANULARITY_TILE)


def test_long_ragged_batch_tile_granular():
    """Prompts that put the block at every offset inside a tile (and across two tiles) over the blocks
    of a generation; per-head scales up to 2."""
    wl = small_workload(name="tile-ragged", prompt_lens=(700, 333, 61, 128), gen_len=192, block_len=32, steps=2,
                        hq=4, hkv=2)
    _run_points(wl, "tc", seed=3, cache_granularity=binding.GRANULARITY_TILE)
    wl = small_workload(name="tile-blk64", prompt_lens=(420, 95), gen_len=192, block_len=64, steps=1, hq=4, hkv=4)
    _run_points(wl, "tc", seed=4, cache_granularity=binding.GRANULARITY_TILE)


def test_tile_granular_with_plain_operands():
    wl = small_workload(name="tile-plain", prompt_lens=(700, 333, 61, 128), gen_len=192, block_len=32, steps=2,
                        hq=4, hkv=2, scale_mode="inv_sqrt_d")
    _run_points(wl, "tc", seed=3, cache_granularity=binding.GRANULARITY_TILE, precision_mode=binding.PRECISION_PLAIN)


def test_cached_state_is_the_tile_level_state():
    """What the tile-granular build caches: for every row outside the tiles that overlap the block, the
    state of Eq. 2-6 over exactly the keys outside those tiles (compared through O~/l and m + log l: the
    triple itself is not unique).  A token-granular context caches more keys, so the two differ."""
    wl = small_workload(prompt_lens=(300, 150, 40), gen_len=96, block_len=32, steps=1, hq=4, hkv=2, d=128)
    sch = SyntheticSchedule(wl, seed=2)
    T = wl.total_tokens
    for b in (0, 1, 2):
        sch = SyntheticSchedule(wl, seed=2)
        q, k, v = advance_to_block(sch, b)
        mask = overlap_mask(wl, b)
        assert mask.sum() > sch.is_block(b).sum()          # the tiles hold more than the block
        rm, rl, ro = oracle.build_state(q, k, v, wl.cu_seqlens, mask, wl.rope_theta, wl.head_dim ** -0.5)
        states = {}
        for gran in (binding.GRANULARITY_TILE, binding.GRANULARITY_TOKEN):
            ctx = make_ctx(wl, engine=binding.ENGINE_TCGEN05, cache_granularity=gran)
            ctx.build(b, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
            m = torch.empty(T, wl.n_q_heads, device="cuda"); l = torch.empty_like(m)
            o = torch.empty(T, wl.n_q_heads, wl.head_dim, device="cuda")
            ctx.export_state(m, l, o)
            torch.cuda.synchronize()
            assert ctx.poll_status()[0] == 0
            states[gran] = tuple(x.cpu().numpy().astype(np.float64) for x in (m, l, o))
            ctx.destroy()
        keep = mask == 0
        m, l, o = (x[keep] for x in states[binding.GRANULARITY_TILE])
        has_keys = rl[keep] > 0                              # a sequence that fits in the overlapping tiles caches nothing
        assert np.array_equal(l > 0, has_keys)
        got = (o / np.where(l > 0, l, 1.0)[..., None])[has_keys]
        ref = (ro[keep] / np.where(has_keys, rl[keep], 1.0)[..., None])[has_keys]
        assert np.abs(got - ref).max() <= 2e-2
        assert np.abs((m + np.log(np.where(l > 0, l, 1.0)))[has_keys] - (rm[keep] + np.log(np.where(has_keys, rl[keep], 1.0)))[has_keys]).max() <= 2e-2
        # the token-granular state of the same rows covers more keys: a larger log normaliser
        mt, lt, _ = (x[keep] for x in states[binding.GRANULARITY_TOKEN])
        assert ((mt + np.log(lt))[has_keys] >= (m + np.log(np.where(l > 0, l, 1.0)))[has_keys] - 1e-3).all()
        assert ((mt + np.log(lt))[has_keys] > (m + np.log(np.where(l > 0, l, 1.0)))[has_keys] + 1e-6).any()


@pytest.mark.parametrize("cfg", [2, 4])
def test_full_size_configs_tile_granular(cfg):
    wl = WORKLOADS[cfg]
    blocks = sorted({b for b, _ in parity_points(wl)})
    _run_points(wl, "tc", seed=0, blocks=blocks, rows_fn=sample_rows, check_full=True, check_state=False,
                cache_granularity=binding.GRANULARITY_TILE)


def test_tile_granular_limits():
    wl = small_workload(prompt_lens=(40,), gen_len=64, block_len=32, steps=1, hq=2, hkv=2, d=128)
    sch = SyntheticSchedule(wl, seed=1)
    ctx = make_ctx(wl, cache_granularity=binding.GRANULARITY_TILE)
    q, k, v = (to_dev(a, wl) for a in sch.begin_block(0))
    with pytest.raises(binding.LacacheError) as e:
        ctx.build_incremental(0, q, k, v)
    assert e.value.status == binding.ERR_UNSUPPORTED
    # the whole sequence fits in the tile that overlaps the block: nothing is cached, a step still serves every row
    ctx.build(0, q, k, v)
    out, lse = new_outputs(wl)
    qb, kb, vb = (to_dev(a, wl) for a in sch.draw_step(0, 1))
    ctx.step(qb, kb, vb, out, lse)
    torch.cuda.synchronize()
    assert ctx.poll_status()[0] == 0
    from lacache_testlib import check_against_oracle
    check_against_oracle(wl, sch, out, lse, None, "one tile")
    ctx.destroy()
    with pytest.raises(binding.LacacheError) as e:
        make_ctx(small_workload(dtype="fp32", prompt_lens=(40,), gen_len=64, block_len=32, hq=2, hkv=2, d=64),
                 cache_granularity=binding.GRANULARITY_TILE)
    assert e.value.status == binding.ERR_UNSUPPORTED
