"""GPU parity tests: the CUDA path (through the C ABI) against the fp64 oracle,
element by element on the same seeded inputs, plus the structural checks of
the cache (immutability, cached == full recompute, bit-exact integer metadata).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_16339_b200 import binding
from paper_2607_16339_b200.workloads import WORKLOADS, SyntheticSchedule, parity_points, small_workload

from lacache_testlib import (TOL, TOL_CACHED_VS_FULL, advance_to_block, check_against_oracle, make_ctx,
                             new_outputs, sample_rows, to_dev)

pytestmark = pytest.mark.gpu

ENGINES = {"simt": binding.ENGINE_SIMT, "tc": binding.ENGINE_TCGEN05}


def _small_cases():
    c = {}
    # several row tiles, ragged batch, block straddling 64/128 boundaries
    c["ragged3"] = dict(prompt_lens=(200, 77, 130), gen_len=128, block_len=32, steps=2, hq=4, hkv=4)
    # GQA, block of 64
    c["gqa"] = dict(prompt_lens=(190,), gen_len=128, block_len=64, steps=2, hq=8, hkv=2, scale_mode="inv_sqrt_d")
    # no prompt at all: the first block has an empty prefix
    c["noprompt"] = dict(prompt_lens=(0, 5), gen_len=96, block_len=32, steps=1, hq=2, hkv=1)
    # one block covers the whole generation (empty suffix); odd prompt length
    c["oneblock"] = dict(prompt_lens=(131,), gen_len=32, block_len=32, steps=2, hq=2, hkv=2)
    # key outliers as in the long-generation config
    c["outliers"] = dict(prompt_lens=(300,), gen_len=64, block_len=32, steps=1, hq=4, hkv=4, outlier_frac=0.02)
    # GQA with a 32-row block (pipelined merge role: the block's keys of a KV head serve its query heads)
    c["gqa32"] = dict(prompt_lens=(150, 61), gen_len=64, block_len=32, steps=2, hq=8, hkv=2)
    # tiny block
    c["blk16"] = dict(prompt_lens=(50, 64), gen_len=48, block_len=16, steps=1, hq=2, hkv=2)
    return c


SMALL = _small_cases()


def _engines_for(dtype, d):
    return ["simt", "tc"] if (dtype == "bf16" and d == 128) else ["simt"]


def _run_points(wl, engine, seed, blocks=None, rows_fn=None, check_full=True, check_state=True, **ctx_kw):
    sch = SyntheticSchedule(wl, seed=seed)
    ctx = make_ctx(wl, engine=ENGINES[engine], **ctx_kw)
    out, lse = new_outputs(wl)
    fout, flse = new_outputs(wl)
    blocks = list(range(wl.n_blocks)) if blocks is None else blocks
    worst = 0.0
    T = wl.total_tokens
    cur = 0
    for b in blocks:
        # bring the arrays to the start of block b
        for bb in range(cur, b):
            sch.begin_block(bb)
            sch.draw_step(bb, wl.steps_per_block)
        cur = b
        q, k, v = sch.begin_block(b)
        ctx.build(b, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
        if check_state:
            m = torch.empty(T, wl.n_q_heads, device="cuda"); l = torch.empty_like(m)
            o = torch.empty(T, wl.n_q_heads, wl.head_dim, device="cuda")
            ctx.export_state(m, l, o)
            state0 = (m.clone(), l.clone(), o.clone())
        steps = sorted({1, wl.steps_per_block})
        for s in steps:
            qb, kb, vb = sch.draw_step(b, s)
            out.fill_(float("nan")); lse.fill_(float("nan"))
            ctx.step(to_dev(qb, wl), to_dev(kb, wl), to_dev(vb, wl), out, lse)
            torch.cuda.synchronize()
            st, msg = ctx.poll_status()
            assert st == 0, msg
            rows = rows_fn(wl, sch, b) if rows_fn else None
            emax, _ = check_against_oracle(wl, sch, out, lse, rows, "%s blk %d step %d" % (wl.name, b, s))
            worst = max(worst, emax)
            if check_full:
                ctx.full_recompute(to_dev(sch.q, wl), to_dev(sch.k, wl), to_dev(sch.v, wl), fout, flse)
                torch.cuda.synchronize()
                check_against_oracle(wl, sch, fout, flse, rows, "%s full blk %d step %d" % (wl.name, b, s))
                diff = (out - fout).abs().max().item()
                assert diff <= TOL_CACHED_VS_FULL[wl.dtype], "cached vs full recompute: %.4g" % diff
                assert (lse - flse).abs().max().item() <= 1e-3
        if check_state:
            # the cache is immutable between builds (reuse pass writes only O and L)
            ctx.export_state(m, l, o)
            torch.cuda.synchronize()
            fixed = torch.from_numpy(sch.is_block(b) == 0).cuda()
            for a0, a1 in zip(state0, (m, l, o)):
                assert torch.equal(a0[fixed], a1[fixed])
    ctx.destroy()
    return worst


@pytest.mark.parametrize("case", sorted(SMALL))
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_small_cases(case, dtype):
    kw = dict(SMALL[case])
    if dtype == "fp32":
        # the 1e-5 bar is stated for the fp32 config's value distribution
        # (N(0,1)/sqrt(d), scores of order 1e-2); fp32 rounding of scores of
        # order 50 alone exceeds it, so fp32 cases keep that distribution
        kw["scale_mode"] = "inv_sqrt_d"
    for d in ((128, 64) if dtype == "fp32" else (128,)):
        wl = small_workload(name=case, dtype=dtype, d=d, **kw)
        for engine in _engines_for(dtype, d):
            _run_points(wl, engine, seed=5)


@pytest.mark.parametrize("block_len", [16, 48])
def test_block_lengths_that_split_a_warp(block_len):
    """Blocks of 16 and 48 rows on the tcgen05 engine with the block queries' keys cut into several
    chunks: the rows of the block end in the middle of a warp of row threads, which must still take
    part in the warp-wide TMEM loads of the partial-state epilogue."""
    wl = small_workload(name="blk%d" % block_len, prompt_lens=(700, 333), gen_len=96, block_len=block_len,
                        steps=2, hq=4, hkv=2)
    _run_points(wl, "tc", seed=8, blocks=[0, wl.n_blocks - 1], sc_tiles_per_chunk=2)


@pytest.mark.parametrize("block_len", [48, 64])
@pytest.mark.parametrize("tiles_per_chunk", [0, 2])
def test_mha_blocks_of_48_and_64_rows(block_len, tiles_per_chunk):
    """A model without grouped heads (one KV head per query head) with blocks of 33..64 rows: the step
    runs unpacked block queries together with the merge variant that takes up to 64 block keys.  Per-head
    scales up to 2 (the harsh value distribution), a ragged batch, prompts long enough for the block
    queries' keys to be cut into several chunks."""
    wl = small_workload(name="mha%d" % block_len, prompt_lens=(700, 333, 61), gen_len=192, block_len=block_len,
                        steps=2, hq=4, hkv=4, scale_mode="per_head_u(0.5,2)")
    _run_points(wl, "tc", seed=14, blocks=[0, 1, wl.n_blocks - 1], sc_tiles_per_chunk=tiles_per_chunk)


@pytest.mark.parametrize("hq,hkv,block_len", [(6, 2, 64), (10, 2, 32), (7, 1, 64), (14, 2, 16)])
def test_packed_block_queries_odd_groups(hq, hkv, block_len):
    """GQA steps put the block rows of two (blocks of 33..64 rows) or four (up to 32 rows) heads of a KV
    group into one tile.  Groups that do not divide evenly leave a last, partly filled tile; with the
    keys cut into chunks every head of a tile has its own arrival counter and is merged on its own."""
    wl = small_workload(name="pack%d_%d_%d" % (hq, hkv, block_len), prompt_lens=(420, 150), gen_len=64,
                        block_len=block_len, steps=2, hq=hq, hkv=hkv, scale_mode="inv_sqrt_d")
    for tiles_per_chunk in (0, 2):
        _run_points(wl, "tc", seed=12, blocks=[0, wl.n_blocks - 1], sc_tiles_per_chunk=tiles_per_chunk)


@pytest.mark.parametrize("engine", ["simt", "tc"])
def test_cached_state_matches_oracle_state(engine):
    wl = small_workload(prompt_lens=(150, 40), gen_len=96, block_len=32, steps=1, hq=4, hkv=2, d=128)
    sch = SyntheticSchedule(wl, seed=2)
    ctx = make_ctx(wl, engine=ENGINES[engine])
    T = wl.total_tokens
    b = 1
    q, k, v = advance_to_block(sch, b)
    ctx.build(b, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
    m = torch.empty(T, wl.n_q_heads, device="cuda"); l = torch.empty_like(m)
    o = torch.empty(T, wl.n_q_heads, wl.head_dim, device="cuda")
    ctx.export_state(m, l, o)
    torch.cuda.synchronize()
    isb = sch.is_block(b)
    rm, rl, ro = oracle.build_state(q, k, v, wl.cu_seqlens, isb, wl.rope_theta, wl.head_dim ** -0.5)
    fixed = isb == 0
    m, l, o = (x.cpu().numpy().astype(np.float64) for x in (m, l, o))
    # the triple is not unique: compare O~/l and m + log l (fixed rows only;
    # rows of the current block carry no state)
    m, l, o, rm, rl, ro = m[fixed], l[fixed], o[fixed], rm[fixed], rl[fixed], ro[fixed]
    assert np.abs(o / l[..., None] - ro / rl[..., None]).max() <= 2e-2
    assert np.abs((m + np.log(l)) - (rm + np.log(rl))).max() <= 2e-2
    ctx.destroy()


@pytest.mark.parametrize("engine,dtype", [("simt", "fp32"), ("simt", "bf16"), ("tc", "bf16")])
def test_rope_cache_and_index_meta(engine, dtype):
    wl = small_workload(dtype=dtype, prompt_lens=(150, 40, 7), gen_len=64, block_len=32, steps=1, hq=4, hkv=2, d=128)
    sch = SyntheticSchedule(wl, seed=4)
    ctx = make_ctx(wl, engine=ENGINES[engine])
    T = wl.total_tokens
    b = 1
    q, k, v = advance_to_block(sch, b)
    ctx.build(b, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
    qb, kb, vb = sch.draw_step(b, 1)
    out, lse = new_outputs(wl)
    ctx.step(to_dev(qb, wl), to_dev(kb, wl), to_dev(vb, wl), out, lse)
    # integer metadata: bit exact against an independent derivation
    seq, pos, isb, kvh = ctx.export_index_meta()
    cu = wl.cu_seqlens
    assert np.array_equal(seq, np.repeat(np.arange(wl.batch), wl.seq_lens).astype(np.int32))
    assert np.array_equal(pos, sch.positions())
    assert np.array_equal(isb, sch.is_block(b).astype(np.int32))
    assert np.array_equal(kvh, np.arange(wl.n_q_heads) // (wl.n_q_heads // wl.n_kv_heads))
    assert cu[-1] == ctx.total_tokens
    # rotated cache after the step holds the block's fresh rows too
    qr = torch.empty(T, wl.n_q_heads, wl.head_dim, device="cuda")
    kr = torch.empty(T, wl.n_kv_heads, wl.head_dim, device="cuda"); vv = torch.empty_like(kr)
    ctx.export_rope_cache(qr, kr, vv)
    torch.cuda.synchronize()
    rq = oracle.rope(sch.q, sch.positions(), wl.rope_theta)
    rk = oracle.rope(sch.k, sch.positions(), wl.rope_theta)
    for got, ref in ((qr, rq), (kr, rk)):
        g = got.cpu().numpy().astype(np.float64)
        nrm = np.abs(ref).max(-1, keepdims=True) + 1e-30
        rel = np.abs(g - ref) / nrm
        # fp32: a few ulp of fp32; split bf16 planes: 2^-16 of the vector's scale
        assert rel.max() <= (2.0 ** -15 if engine == "tc" else 1e-6), rel.max()
    assert np.array_equal(vv.cpu().numpy().astype(np.float64), sch.v.astype(np.float64))
    ctx.destroy()


def test_runs_are_bit_reproducible():
    wl = small_workload(prompt_lens=(200, 77), gen_len=64, block_len=32, steps=1, hq=4, hkv=2, d=128)
    for engine in ("simt", "tc"):
        outs = []
        for rep in range(2):
            sch = SyntheticSchedule(wl, seed=9)
            ctx = make_ctx(wl, engine=ENGINES[engine])
            q, k, v = sch.begin_block(0)
            ctx.build(0, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
            qb, kb, vb = sch.draw_step(0, 1)
            out, lse = new_outputs(wl)
            ctx.step(to_dev(qb, wl), to_dev(kb, wl), to_dev(vb, wl), out, lse)
            torch.cuda.synchronize()
            outs.append((out.clone(), lse.clone()))
            ctx.destroy()
        assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


_MHA64 = small_workload(name="mha64", prompt_lens=(700, 333, 61), gen_len=192, block_len=64, steps=6, hq=4, hkv=4,
                        scale_mode="per_head_u(0.5,2)")


@pytest.mark.parametrize("cfg", [2, 4, 5, "mha64", "2-fp16", "4-fp16"])
@pytest.mark.parametrize("overlap", [True, False])
def test_back_to_back_steps_match_synchronised_steps(cfg, overlap):
    """With the overlap of consecutive steps switched on (precomputed inputs), the next step's kernels
    are scheduled while the previous attention kernel drains.  A stream of steps and builds issued
    without any host synchronisation must give, bit for bit, what the same calls give when the host
    waits after each one -- with a separate output buffer per step and with one reused; likewise with
    the default, plain stream order."""
    # ("-fp16": one fp16 plane per operand; at config 2 the step then runs its two key chunks as pairs of CTAs)
    mode = binding.PRECISION_SPLIT
    if isinstance(cfg, str) and cfg.endswith("-fp16"):
        cfg, mode = int(cfg[0]), binding.PRECISION_FP16
    wl = _MHA64 if cfg == "mha64" else WORKLOADS[cfg]
    S = min(wl.steps_per_block, 6)
    calls = []   # ("build", blk, q, k, v) / ("step", qb, kb, vb)
    sch = SyntheticSchedule(wl, seed=21)
    for blk in (0, 1):
        q, k, v = sch.begin_block(blk)
        calls.append(("build", blk, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl)))
        for s in range(1, S + 1):
            qb, kb, vb = sch.draw_step(blk, s)
            calls.append(("step", to_dev(qb, wl), to_dev(kb, wl), to_dev(vb, wl)))
    n_steps = sum(1 for c in calls if c[0] == "step")

    def run(sync, one_buffer):
        ctx = make_ctx(wl, engine=ENGINES["tc"], precision_mode=mode)
        ctx.set_step_overlap(overlap)
        bufs = [new_outputs(wl) for _ in range(1 if one_buffer else n_steps)]
        res, i = [], 0
        for c in calls:
            if c[0] == "build":
                ctx.build(c[1], c[2], c[3], c[4])
            else:
                out, lse = bufs[0 if one_buffer else i]
                ctx.step(c[1], c[2], c[3], out, lse)
                i += 1
                if sync:
                    torch.cuda.synchronize()
                    res.append((out.clone(), lse.clone()))
            if sync:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        st, msg = ctx.poll_status()
        assert st == 0, msg
        if not sync:
            res = [(o.clone(), l.clone()) for o, l in bufs]
        ctx.destroy()
        return res

    ref = run(sync=True, one_buffer=False)
    for rep in range(3):
        got = run(sync=False, one_buffer=False)
        for i, ((o0, l0), (o1, l1)) in enumerate(zip(ref, got)):
            assert torch.equal(o0, o1) and torch.equal(l0, l1), "step %d differs when issued back to back" % i
        last = run(sync=False, one_buffer=True)
        assert torch.equal(ref[-1][0], last[0][0]) and torch.equal(ref[-1][1], last[0][1])


@pytest.mark.parametrize("cfg", [2, 5])
def test_steps_fed_by_same_stream_writes(cfg):
    """Block inputs that are written on the stream between two steps (here: copied into one reused
    trio of buffers right before each step) with the default setting (no cross-step overlap): every
    kernel of a step is ordered after the copy.  Bit for bit what synchronised steps give."""
    wl = WORKLOADS[cfg]
    S = min(wl.steps_per_block, 5)
    sch = SyntheticSchedule(wl, seed=33)
    q, k, v = (to_dev(a, wl) for a in sch.begin_block(0))
    steps = [tuple(to_dev(a, wl) for a in sch.draw_step(0, s)) for s in range(1, S + 1)]
    ctx = make_ctx(wl, engine=ENGINES["tc"])
    ctx.build(0, q, k, v)
    ref = []
    for qb, kb, vb in steps:
        out, lse = new_outputs(wl)
        ctx.step(qb, kb, vb, out, lse)
        torch.cuda.synchronize()
        ref.append((out, lse))
    qs, ks, vs = (torch.empty_like(t) for t in steps[0])
    for rep in range(3):
        got = [new_outputs(wl) for _ in steps]
        for (qb, kb, vb), (out, lse) in zip(steps, got):
            qs.copy_(qb); ks.copy_(kb); vs.copy_(vb)      # same stream, no host wait
            ctx.step(qs, ks, vs, out, lse)
        torch.cuda.synchronize()
        for i, ((o0, l0), (o1, l1)) in enumerate(zip(ref, got)):
            assert torch.equal(o0, o1) and torch.equal(l0, l1), "step %d" % i
    assert ctx.poll_status()[0] == 0
    ctx.destroy()


@pytest.mark.parametrize("hq,hkv,block_len", [(4, 2, 32), (6, 2, 16), (8, 2, 32), (6, 2, 64), (4, 2, 64)])
def test_packed_block_rows_several_units_per_cta(hq, hkv, block_len, monkeypatch):
    """Block rows of a GQA model share a tile (heads of a KV group side by side).  A CTA's first unit
    rotates its queries itself; every later unit's tile comes through the packed tensor map, whose box
    must fill the tile whatever the group size (2 and 3 heads of 32 rows leave lanes over).  Forced here
    with two stream CTAs for all units, and once with the first unit loaded the same way."""
    wl = small_workload(name="packed-%d-%d-%d" % (hq, hkv, block_len), prompt_lens=(150, 61, 230), gen_len=2 * block_len,
                        block_len=block_len, steps=2, hq=hq, hkv=hkv)
    monkeypatch.setenv("LACACHE_STREAM_CTAS", "2")       # (experiment knobs are read when a context is created)
    _run_points(wl, "tc", seed=8)
    monkeypatch.setenv("LACACHE_NO_QCOMP", "1")
    _run_points(wl, "tc", seed=9, check_state=False)
    monkeypatch.delenv("LACACHE_NO_QCOMP")
    monkeypatch.delenv("LACACHE_STREAM_CTAS")


@pytest.mark.parametrize("mode", ["fp16", "plain"])
@pytest.mark.parametrize("block_len", [16, 32])
def test_two_key_chunks_as_a_pair_of_ctas(mode, block_len, monkeypatch):
    """With one-plane operands, unpacked heads, one round of block-row units and exactly two key chunks per
    (sequence, head), the two chunks run as a thread-block cluster of two CTAs: the second hands its partial
    state to the first through distributed shared memory, and the first writes the merged rows.  Forced here
    by the chunk size and the role split; the same cases with the pairing switched off must agree within the
    tolerance between two orders of the same merge, and both with the oracle."""
    kw = dict(prompt_lens=(150, 180, 130), gen_len=2 * block_len, block_len=block_len, steps=2, hq=4, hkv=4)
    if mode == "plain":
        kw["scale_mode"] = "inv_sqrt_d"
    wl = small_workload(name="pair-%s-%d" % (mode, block_len), dtype="bf16", d=128, **kw)
    units = wl.batch * 2 * wl.n_q_heads
    monkeypatch.setenv("LACACHE_STREAM_CTAS", str(units))      # (experiment knobs are read when a context is created)
    outs = {}
    for pair in (True, False):
        if not pair:
            monkeypatch.setenv("LACACHE_NO_PAIR", "1")
        _run_points(wl, "tc", seed=12, precision_mode=_MODES[mode], sc_tiles_per_chunk=1)
        sch = SyntheticSchedule(wl, seed=12)
        ctx = make_ctx(wl, engine=ENGINES["tc"], precision_mode=_MODES[mode], sc_tiles_per_chunk=1)
        q, k, v = (to_dev(a, wl) for a in advance_to_block(sch, 1))
        ctx.build(1, q, k, v)
        out, lse = new_outputs(wl)
        ctx.step(*(to_dev(a, wl) for a in sch.draw_step(1, 1)), out, lse)
        torch.cuda.synchronize()
        assert ctx.poll_status()[0] == 0
        outs[pair] = (out.clone(), lse.clone())
        ctx.destroy()
    monkeypatch.delenv("LACACHE_NO_PAIR")
    monkeypatch.delenv("LACACHE_STREAM_CTAS")
    assert (outs[True][0] - outs[False][0]).abs().max().item() <= 1e-5
    assert (outs[True][1] - outs[False][1]).abs().max().item() <= 1e-5


@pytest.mark.parametrize("cfg", [3, 4])
def test_step_split_over_several_launches(cfg, monkeypatch):
    """A step with more fixed-row tiles per CTA than the pipelined merge variant tabulates goes out in
    several launches (block queries and the first row tiles, then row tiles only on all SMs).  Forced
    here with a tiny table: the result must be, bit for bit, that of the single launch."""
    wl = WORKLOADS[cfg]
    sch = SyntheticSchedule(wl, seed=5)
    b = 1
    q, k, v = (to_dev(a, wl) for a in advance_to_block(sch, b))
    steps = [tuple(to_dev(a, wl) for a in sch.draw_step(b, s)) for s in (1, 2, 3)]
    ctx = make_ctx(wl, engine=ENGINES["tc"])
    ctx.build(b, q, k, v)
    ref = []
    for qb, kb, vb in steps:
        out, lse = new_outputs(wl)
        ctx.step(qb, kb, vb, out, lse)
        ref.append((out, lse))
    torch.cuda.synchronize()
    assert ctx.last_launch_count == 2
    for cap in ("3", "1"):
        monkeypatch.setenv("LACACHE_DEEP_UNITS", cap)     # (experiment knobs are read when a context is created)
        ctx.destroy()
        ctx = make_ctx(wl, engine=ENGINES["tc"])
        ctx.set_step_overlap(True)
        ctx.build(b, q, k, v)
        got = []
        for qb, kb, vb in steps:              # back to back: the launches of consecutive steps overlap
            out, lse = new_outputs(wl)
            ctx.step(qb, kb, vb, out, lse)
            got.append((out, lse))
        torch.cuda.synchronize()
        assert ctx.last_launch_count >= 3, ctx.last_launch_count
        for (o0, l0), (o1, l1) in zip(ref, got):
            assert torch.equal(o0, o1) and torch.equal(l0, l1)
    monkeypatch.delenv("LACACHE_DEEP_UNITS")
    assert ctx.poll_status()[0] == 0
    check_against_oracle(wl, sch, got[-1][0], got[-1][1], rows=sample_rows(wl, sch, b), what="split step")
    ctx.destroy()


@pytest.mark.parametrize("mode", ["split", "plain", "fp16"])
def test_large_batch_extension_full_size(mode):
    """The large-batch extension (256 sequences, 28/4 heads, ~287k tokens) at full size, in the
    launch configuration the bench times: the step's fixed rows exceed one launch of the pipelined
    merge variant and go out in several.  Cached path vs full recompute on every row; vs the oracle
    on all rows of three sequences (first, longest, last)."""
    from paper_2607_16339_b200.workloads import DeviceSchedule
    wl = WORKLOADS[6]
    S = 3
    sched = DeviceSchedule(wl, 17, torch.device("cuda"), S)
    ctx = make_ctx(wl, engine=ENGINES["tc"],
                   precision_mode={"plain": binding.PRECISION_PLAIN, "split": binding.PRECISION_SPLIT,
                                   "fp16": binding.PRECISION_FP16}[mode])
    q, k, v = sched.full[0]
    ctx.build(0, q, k, v)
    out, lse = new_outputs(wl)
    for s in range(S):
        qb, kb, vb = sched.steps[s]
        ctx.step(qb, kb, vb, out, lse)
    torch.cuda.synchronize()
    assert ctx.last_launch_count >= 3            # RoPE + more than one attention launch
    assert ctx.poll_status()[0] == 0
    cu = wl.cu_seqlens
    rows = torch.cat([torch.arange(cu[b] + P, cu[b] + P + wl.block_len) for b, P in enumerate(wl.prompt_lens)]).cuda()
    qf, kf, vf = q.clone(), k.clone(), v.clone()
    qf[rows], kf[rows], vf[rows] = qb, kb, vb
    out2, lse2 = new_outputs(wl)
    ctx.full_recompute(qf, kf, vf, out2, lse2)
    torch.cuda.synchronize()
    assert float((out - out2).abs().max()) <= TOL_CACHED_VS_FULL["bf16"]
    assert float((lse - lse2).abs().max()) <= TOL_CACHED_VS_FULL["bf16"]
    seqs = sorted({0, int(np.argmax(wl.prompt_lens)), wl.batch - 1})
    idx = np.concatenate([np.arange(cu[b], cu[b + 1]) for b in seqs])
    sub_cu = np.concatenate([[0], np.cumsum([cu[b + 1] - cu[b] for b in seqs])]).astype(np.int32)
    t_idx = torch.from_numpy(idx).cuda()
    host = lambda t: t[t_idx].float().cpu().numpy().astype(np.float64)
    ref, rlse = oracle.attention(host(qf), host(kf), host(vf), sub_cu, wl.rope_theta, wl.head_dim ** -0.5)
    err = np.abs(out[t_idx].cpu().numpy().astype(np.float64) - ref)
    assert err.max() <= TOL["bf16"][0] and err.mean() <= TOL["bf16"][1], (err.max(), err.mean())
    # the outputs here are small (values ~ N(0,1)/sqrt(d), near-uniform attention): also relative to their scale
    assert err.max() <= 2e-2 * np.abs(ref).max(), (err.max(), np.abs(ref).max())
    assert np.abs(lse[t_idx].cpu().numpy() - rlse).max() <= TOL["bf16"][0]
    ctx.destroy()


@pytest.mark.parametrize("case", sorted(SMALL) + ["mha64", "long48"])
def test_plain_operands_small_cases(case):
    """precision_mode = plain (one bf16 plane of the rotated Q', K', one score product, 128-key tiles) on
    the value distribution it is meant for, N(0,1)/sqrt(d): same tolerances against the oracle and
    against the GPU full recompute as the split mode."""
    extra = {"mha64": dict(prompt_lens=(700, 333, 61), gen_len=192, block_len=64, steps=2, hq=4, hkv=4),
             "long48": dict(prompt_lens=(900, 333), gen_len=96, block_len=48, steps=2, hq=8, hkv=2)}
    kw = dict(extra[case] if case in extra else SMALL[case])
    kw["scale_mode"] = "inv_sqrt_d"
    wl = small_workload(name=case, dtype="bf16", d=128, **kw)
    for tiles_per_chunk in (0, 2):
        _run_points(wl, "tc", seed=6, precision_mode=binding.PRECISION_PLAIN, sc_tiles_per_chunk=tiles_per_chunk)


@pytest.mark.parametrize("case", sorted(SMALL) + ["mha64", "long48"])
def test_fp16_operands_small_cases(case):
    """precision_mode = fp16 (one fp16 plane of the rotated Q', K', one score product, 128-key tiles) at
    the harsh value scale (per-head scales up to 2): the same tolerances against the oracle and against
    the GPU full recompute as the split mode."""
    extra = {"mha64": dict(prompt_lens=(700, 333, 61), gen_len=192, block_len=64, steps=2, hq=4, hkv=4),
             "long48": dict(prompt_lens=(900, 333), gen_len=96, block_len=48, steps=2, hq=8, hkv=2)}
    kw = dict(extra[case] if case in extra else SMALL[case])
    wl = small_workload(name=case, dtype="bf16", d=128, **kw)
    for tiles_per_chunk in (0, 2):
        _run_points(wl, "tc", seed=6, precision_mode=binding.PRECISION_FP16, sc_tiles_per_chunk=tiles_per_chunk)


@pytest.mark.parametrize("case", ["ragged3", "gqa", "gqa32", "blk16", "mha64"])
@pytest.mark.parametrize("engine", ["tc", "simt"])
def test_bf16_output(case, engine):
    """out_dtype = bf16: every epilogue (fixed rows through both merge variants, block rows, merged key
    chunks, the full recompute) rounds the very fp32 value the fp32 context writes, once, to nearest even:
    the two outputs agree bit for bit after that rounding.  Against the oracle the error is the fp32
    path's plus at most half a bf16 unit of the value (at most 2^-8 |o|); the figures are printed."""
    kw = dict(prompt_lens=(700, 333, 61), gen_len=192, block_len=64, steps=2, hq=4, hkv=4) if case == "mha64" else dict(SMALL[case])
    wl = small_workload(name=case, dtype="bf16", d=128, **kw)
    sch = SyntheticSchedule(wl, seed=31)
    b = wl.n_blocks - 1
    q, k, v = (to_dev(a, wl) for a in advance_to_block(sch, b))
    qb, kb, vb = (to_dev(a, wl) for a in sch.draw_step(b, 1))
    T = wl.total_tokens
    res = {}
    for od in (binding.OUT_FP32, binding.OUT_BF16):
        ctx = make_ctx(wl, engine=ENGINES[engine], out_dtype=od, sc_tiles_per_chunk=2)
        tdt = torch.float32 if od == binding.OUT_FP32 else torch.bfloat16
        out = torch.full((T, wl.n_q_heads, wl.head_dim), float("nan"), device="cuda", dtype=tdt)
        fout = torch.full_like(out, float("nan"))
        lse = torch.full((T, wl.n_q_heads), float("nan"), device="cuda")
        ctx.build(b, q, k, v)
        ctx.step(qb, kb, vb, out, lse)
        ctx.full_recompute(to_dev(sch.q, wl), to_dev(sch.k, wl), to_dev(sch.v, wl), fout, None)
        torch.cuda.synchronize()
        assert ctx.poll_status()[0] == 0
        res[od] = (out, fout, lse)
        ctx.destroy()
    o32, f32, l32 = res[binding.OUT_FP32]
    o16, f16, l16 = res[binding.OUT_BF16]
    assert torch.equal(o32.to(torch.bfloat16), o16)
    assert torch.equal(f32.to(torch.bfloat16), f16)
    assert torch.equal(l32, l16)
    ref, _ = oracle.attention(sch.q, sch.k, sch.v, wl.cu_seqlens, wl.rope_theta, wl.head_dim ** -0.5)
    e32 = np.abs(o32.cpu().numpy().astype(np.float64) - ref)
    e16 = np.abs(o16.float().cpu().numpy().astype(np.float64) - ref)
    assert (e16 <= e32 + 2.0 ** -8 * (np.abs(ref) + e32) + 1e-12).all()
    print("bf16 out, %s/%s: max abs err %.4g (fp32 out %.4g), mean %.4g (%.4g), max |o| %.3g"
          % (case, engine, e16.max(), e32.max(), e16.mean(), e32.mean(), np.abs(ref).max()))


def test_error_paths():
    wl = small_workload(prompt_lens=(40,), gen_len=64, block_len=32, steps=1, hq=2, hkv=2, d=128)
    sch = SyntheticSchedule(wl, seed=1)
    ctx = make_ctx(wl)
    q, k, v = (to_dev(a, wl) for a in sch.begin_block(0))
    out, lse = new_outputs(wl)
    qb, kb, vb = (to_dev(a, wl) for a in sch.draw_step(0, 1))
    with pytest.raises(binding.LacacheError) as e:
        ctx.step(qb, kb, vb, out, lse)
    assert e.value.status == binding.ERR_STATE
    for bad in (-1, wl.n_blocks):
        with pytest.raises(binding.LacacheError) as e:
            ctx.build(bad, q, k, v)
        assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.LacacheError) as e:
        ctx.build(0, q, None, v)
    assert e.value.status == binding.ERR_INVALID_ARG
    mis = torch.empty(q.numel() + 8, dtype=q.dtype, device="cuda")[1:]
    with pytest.raises(binding.LacacheError) as e:
        ctx.build(0, mis, k, v)
    assert e.value.status == binding.ERR_INVALID_ARG
    ctx.build(0, q, k, v)
    ctx.step(qb, kb, vb, out, None)       # lse is optional
    torch.cuda.synchronize()
    assert ctx.poll_status()[0] == 0 and torch.isfinite(out).all()
    assert ctx.last_launch_count >= 1
    ctx.destroy()


def test_host_entry_points_match_device_ones():
    wl = small_workload(prompt_lens=(100, 30), gen_len=64, block_len=32, steps=1, hq=4, hkv=2, d=128)
    sch = SyntheticSchedule(wl, seed=6)
    ctx = make_ctx(wl)
    tdt = torch.bfloat16
    q, k, v = sch.begin_block(0)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(tdt).pin_memory()
    ctx.build_host(0, pin(q), pin(k), pin(v))
    qb, kb, vb = sch.draw_step(0, 1)
    T = wl.total_tokens
    out_h = torch.empty(T, wl.n_q_heads, wl.head_dim).pin_memory()
    lse_h = torch.empty(T, wl.n_q_heads).pin_memory()
    ctx.step_host(pin(qb), pin(kb), pin(vb), out_h, lse_h)
    torch.cuda.synchronize()
    out, lse = new_outputs(wl)
    ctx.step(to_dev(qb, wl), to_dev(kb, wl), to_dev(vb, wl), out, lse)
    torch.cuda.synchronize()
    assert torch.equal(out.cpu(), out_h) and torch.equal(lse.cpu(), lse_h)
    check_against_oracle(wl, sch, out, lse, None, "host entry")
    ctx.destroy()


def test_cfg1_every_step():
    wl = WORKLOADS[1]
    sch = SyntheticSchedule(wl, seed=0)
    ctx = make_ctx(wl)
    out, lse = new_outputs(wl)
    fout, flse = new_outputs(wl)
    for b in range(wl.n_blocks):
        q, k, v = sch.begin_block(b)
        ctx.build(b, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))   # the cache is rebuilt per block
        for s in range(1, wl.steps_per_block + 1):
            qb, kb, vb = sch.draw_step(b, s)
            ctx.step(to_dev(qb, wl), to_dev(kb, wl), to_dev(vb, wl), out, lse)
            ctx.full_recompute(to_dev(sch.q, wl), to_dev(sch.k, wl), to_dev(sch.v, wl), fout, flse)
            torch.cuda.synchronize()
            check_against_oracle(wl, sch, out, lse, None, "cfg1 blk %d step %d" % (b, s))
            assert (out - fout).abs().max().item() <= 1e-5
    ctx.destroy()


_MODES = {"plain": binding.PRECISION_PLAIN, "split": binding.PRECISION_SPLIT, "fp16": binding.PRECISION_FP16}


@pytest.mark.parametrize("cfg,mode", [(2, "split"), (3, "split"), (4, "split"), (5, "split"), (5, "plain"),
                                      (2, "fp16"), (4, "fp16"), (5, "fp16")])
def test_full_size_configs_at_parity_points(cfg, mode):
    """Full-size workloads in the launch configuration the benchmark times;
    the oracle is evaluated on all block rows, edge rows and a seeded sample.  The GQA long-context
    configuration (values ~ N(0,1)/sqrt(d)) also with plain operands; with one fp16 plane per operand the
    configurations it holds on (not the one whose keys carry 4x outliers: 0.024 there, outside the bar)."""
    wl = WORKLOADS[cfg]
    blocks = sorted({b for b, _ in parity_points(wl)})
    worst = _run_points(wl, "tc", seed=0, blocks=blocks, rows_fn=sample_rows, check_full=True, check_state=(cfg == 2),
                        precision_mode=_MODES[mode])
    print("config %d, %s operands: max abs err against the oracle %.3g" % (cfg, mode, worst))
