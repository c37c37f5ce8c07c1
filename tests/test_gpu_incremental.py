"""GPU parity tests of the incremental rebuild across blocks: a context that is built once and then
advanced block by block must serve every step like one that is rebuilt from scratch for every block --
against the fp64 oracle within the path's tolerance, against the from-scratch context within the
tolerance between two GPU orders of the same reduction, and its cached state must describe the same
softmax (O~/l and m + log l agree)."""
import numpy as np
import pytest
import torch

from paper_2607_16339_b200 import binding
from paper_2607_16339_b200.workloads import SyntheticSchedule, small_workload

from lacache_testlib import TOL_CACHED_VS_FULL, check_against_oracle, make_ctx, new_outputs, to_dev

pytestmark = pytest.mark.gpu

CASES = {
    # several row tiles, ragged batch, four blocks
    "ragged3": dict(prompt_lens=(200, 77, 130), gen_len=128, block_len=32, steps=2, hq=4, hkv=4),
    # empty prefix at block 0 (no keys before the block), tiny second sequence
    "noprompt": dict(prompt_lens=(0, 5), gen_len=96, block_len=32, steps=1, hq=2, hkv=1),
    # a single block: nothing to advance to, and no keys after the block
    "oneblock": dict(prompt_lens=(131,), gen_len=32, block_len=32, steps=2, hq=2, hkv=2),
    # GQA, block of 64 rows
    "gqa64": dict(prompt_lens=(190,), gen_len=192, block_len=64, steps=2, hq=8, hkv=2, scale_mode="inv_sqrt_d"),
    # block of 16 rows (the rows of a finished block end inside a warp of row threads)
    "blk16": dict(prompt_lens=(50, 64), gen_len=48, block_len=16, steps=1, hq=2, hkv=2),
    # long prompts: the prefix spans many key tiles, the suffix windows one to three
    "long": dict(prompt_lens=(700, 333), gen_len=256, block_len=32, steps=1, hq=4, hkv=2),
    # key outliers as in the long-generation configuration
    "outliers": dict(prompt_lens=(300,), gen_len=96, block_len=32, steps=1, hq=4, hkv=4, outlier_frac=0.02),
}


def _state(ctx, wl):
    T = wl.total_tokens
    m = torch.empty(T, wl.n_q_heads, device="cuda")
    l = torch.empty_like(m)
    o = torch.empty(T, wl.n_q_heads, wl.head_dim, device="cuda")
    ctx.export_state(m, l, o)
    torch.cuda.synchronize()
    return m.double(), l.double(), o.double()


def _run(wl, seed, **ctx_kw):
    sch = SyntheticSchedule(wl, seed=seed)
    inc = make_ctx(wl, engine=binding.ENGINE_TCGEN05, **ctx_kw)
    ref = make_ctx(wl, engine=binding.ENGINE_TCGEN05, **ctx_kw)
    out, lse = new_outputs(wl)
    rout, rlse = new_outputs(wl)
    fin = None
    for b in range(wl.n_blocks):
        q, k, v = sch.begin_block(b)
        if b == 0:
            inc.build_incremental(0, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
        else:
            inc.build_advance(*(to_dev(x, wl) for x in fin))
        ref.build(b, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
        torch.cuda.synchronize()
        for c in (inc, ref):
            st, msg = c.poll_status()
            assert st == 0, msg
        # same softmax in both caches (the triple itself is not unique)
        fixed = torch.from_numpy(sch.is_block(b) == 0).cuda()
        (m1, l1, o1), (m2, l2, o2) = _state(inc, wl), _state(ref, wl)
        has_keys = (l2[fixed] > 0)
        assert torch.equal(l1[fixed] > 0, has_keys)
        n1 = (o1[fixed] / l1[fixed][..., None])[has_keys]
        n2 = (o2[fixed] / l2[fixed][..., None])[has_keys]
        assert (n1 - n2).abs().max().item() <= TOL_CACHED_VS_FULL[wl.dtype], "block %d" % b
        e1 = (m1[fixed] + torch.log(l1[fixed]))[has_keys]
        e2 = (m2[fixed] + torch.log(l2[fixed]))[has_keys]
        assert (e1 - e2).abs().max().item() <= 1e-3, "block %d" % b
        for s in sorted({1, wl.steps_per_block}):
            qb, kb, vb = sch.draw_step(b, s)
            out.fill_(float("nan")); lse.fill_(float("nan"))
            inc.step(to_dev(qb, wl), to_dev(kb, wl), to_dev(vb, wl), out, lse)
            ref.step(to_dev(qb, wl), to_dev(kb, wl), to_dev(vb, wl), rout, rlse)
            torch.cuda.synchronize()
            st, msg = inc.poll_status()
            assert st == 0, msg
            check_against_oracle(wl, sch, out, lse, None, "%s incremental blk %d step %d" % (wl.name, b, s))
            assert (out - rout).abs().max().item() <= TOL_CACHED_VS_FULL[wl.dtype]
            assert (lse - rlse).abs().max().item() <= 1e-3
        fin = (qb, kb, vb)   # the block's rows as its last step saw them are its final rows
    inc.destroy()
    ref.destroy()


@pytest.mark.parametrize("case", sorted(CASES))
def test_advanced_context_serves_steps_like_a_rebuilt_one(case):
    _run(small_workload(name=case, **CASES[case]), seed=21)


def test_advance_with_the_finished_rows_as_window_units(monkeypatch):
    """The finished block's rows over the keys before the next block: by default block-row units of the
    step kernel over key chunks plus a merge launch; behind a knob, key-window units of the build kernel."""
    monkeypatch.setenv("LACACHE_NO_CHUNKED_ADVANCE", "1")      # (read when a context is created)
    _run(small_workload(name="long-window", **CASES["long"]), seed=22)
    monkeypatch.delenv("LACACHE_NO_CHUNKED_ADVANCE")


@pytest.mark.parametrize("case", ["gqa64", "long", "noprompt", "mha64"])
def test_advanced_context_with_plain_operands(case):
    """The same walk with precision_mode = plain (128-key tiles in the key-window units) on the value
    distribution that mode is meant for."""
    kw = dict(CASES[case]) if case in CASES else dict(prompt_lens=(700, 333, 61), gen_len=192, block_len=64, steps=1,
                                                       hq=4, hkv=4)
    kw["scale_mode"] = "inv_sqrt_d"
    _run(small_workload(name=case, **kw), seed=22, precision_mode=binding.PRECISION_PLAIN)


@pytest.mark.parametrize("case", ["gqa64", "long", "ragged3", "mha64"])
def test_advanced_context_with_fp16_operands(case):
    """The same walk with precision_mode = fp16 (one fp16 plane per operand) at the harsh value scale."""
    kw = dict(CASES[case]) if case in CASES else dict(prompt_lens=(700, 333, 61), gen_len=192, block_len=64, steps=1,
                                                       hq=4, hkv=4)
    _run(small_workload(name=case, **kw), seed=23, precision_mode=binding.PRECISION_FP16)


@pytest.mark.parametrize("block_len", [48, 64])
def test_advanced_context_mha_blocks_of_48_and_64_rows(block_len):
    """No grouped heads, blocks of 33..64 rows, per-head scales up to 2, ragged, long prompts."""
    _run(small_workload(name="mha%d" % block_len, prompt_lens=(700, 333, 61), gen_len=192, block_len=block_len, steps=2,
                        hq=4, hkv=4, scale_mode="per_head_u(0.5,2)"), seed=23)


def test_incremental_build_at_a_later_block_then_advance():
    """The incremental build may start at any block (a resumed generation), not only at block 0."""
    wl = small_workload(name="resume", prompt_lens=(150, 61), gen_len=128, block_len=32, steps=1, hq=4, hkv=2)
    sch = SyntheticSchedule(wl, seed=3)
    ctx = make_ctx(wl, engine=binding.ENGINE_TCGEN05)
    out, lse = new_outputs(wl)
    for b in range(2):
        sch.begin_block(b)
        sch.draw_step(b, wl.steps_per_block)
    q, k, v = sch.begin_block(2)
    ctx.build_incremental(2, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
    fin = sch.draw_step(2, 1)
    ctx.step(*(to_dev(x, wl) for x in fin), out, lse)
    torch.cuda.synchronize()
    check_against_oracle(wl, sch, out, lse, None, "resume blk 2")
    sch.begin_block(3)
    ctx.build_advance(*(to_dev(x, wl) for x in fin))
    blk = sch.draw_step(3, 1)
    ctx.step(*(to_dev(x, wl) for x in blk), out, lse)
    torch.cuda.synchronize()
    st, msg = ctx.poll_status()
    assert st == 0, msg
    check_against_oracle(wl, sch, out, lse, None, "resume blk 3")
    ctx.destroy()


def test_advance_needs_an_incremental_state():
    wl = small_workload(name="state", prompt_lens=(40,), gen_len=64, block_len=32, steps=1, hq=2, hkv=2)
    sch = SyntheticSchedule(wl, seed=1)
    q, k, v = sch.begin_block(0)
    blk = tuple(to_dev(x, wl) for x in sch.draw_step(0, 1))
    ctx = make_ctx(wl, engine=binding.ENGINE_TCGEN05)
    with pytest.raises(binding.LacacheError) as e:
        ctx.build_advance(*blk)                       # nothing built
    assert e.value.status == binding.ERR_STATE
    ctx.build(0, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
    with pytest.raises(binding.LacacheError) as e:
        ctx.build_advance(*blk)                       # a plain build leaves no prefix state
    assert e.value.status == binding.ERR_STATE
    ctx.build_incremental(0, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
    ctx.build_advance(*blk)
    with pytest.raises(binding.LacacheError) as e:
        ctx.build_advance(*blk)                       # block 1 is the last one
    assert e.value.status == binding.ERR_STATE
    ctx.destroy()
    simt = make_ctx(wl, engine=binding.ENGINE_SIMT)
    with pytest.raises(binding.LacacheError) as e:
        simt.build_incremental(0, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
    assert e.value.status == binding.ERR_UNSUPPORTED
    simt.destroy()


def test_token_fed_generation_advances():
    """The incremental rebuild fed by token ids: all T tokens projected once at block 0, afterwards only
    the finished block's final tokens (projection -> RoPE-on-write -> advance); every block's last step
    against the oracle chain (token-wise oracle at model precision -> attention oracle)."""
    import oracle
    from paper_2607_16339_b200.workloads import TokenModel
    from test_gpu_tokenwise import make_producer, oracle_qkv
    wl = small_workload(name="tokgen", prompt_lens=(150, 61), gen_len=96, block_len=32, steps=2, hq=4, hkv=2)
    tm = TokenModel(wl, 512, 3000)
    prod = make_producer(tm, wl.total_tokens)
    ctx = make_ctx(wl, engine=binding.ENGINE_TCGEN05)
    sch = SyntheticSchedule(wl)   # index sets only
    out, lse = new_outputs(wl)
    ids = tm.full_ids(0).copy()
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    ctx.build_tokens_incremental(prod, 0, token_ids=dev(ids))
    fin = None
    for b in range(wl.n_blocks):
        if b > 0:
            ctx.build_advance_tokens(prod, fin_token_ids=dev(fin))
        fin = tm.block_ids(b, wl.steps_per_block)      # the block's last step sees its final tokens
        assert not (fin == tm.mask_id).any()
        ctx.step_tokens(prod, out, lse, blk_token_ids=dev(fin))
        torch.cuda.synchronize()
        for o in (ctx, prod):
            st, msg = o.poll_status()
            assert st == binding.OK, msg
        ids[sch.block_rows(b)] = fin
        _, qf, kf, vf = oracle_qkv(tm, ids=ids)
        ref, rlse = oracle.attention(qf, kf, vf, wl.cu_seqlens, wl.rope_theta, wl.head_dim ** -0.5)
        err = np.abs(out.cpu().numpy().astype(np.float64) - ref)
        assert err.max() <= 2e-2 and err.mean() <= 2e-3, (b, err.max(), err.mean())
        assert np.abs(lse.cpu().numpy() - rlse).max() <= 2e-2
    ctx.destroy()
    prod.destroy()


@pytest.mark.parametrize("cfg,n_adv", [(3, 3), (5, 2), (6, 2)])
def test_full_size_advance(cfg, n_adv):
    """Full-size workloads (the long-generation and the GQA long-prompt configurations, and the
    large-batch extension) advanced n_adv blocks from an incremental build: the step after the last
    advance against a full recompute of the same inputs on every row, and against the oracle on all
    rows of up to three whole sequences (first, longest, last)."""
    import oracle
    from paper_2607_16339_b200.workloads import WORKLOADS, DeviceSchedule
    from lacache_testlib import TOL
    wl = WORKLOADS[cfg]
    S = wl.steps_per_block
    sched = DeviceSchedule(wl, 23, torch.device("cuda"), n_adv * S + 1)
    ctx = make_ctx(wl, engine=binding.ENGINE_TCGEN05)
    ctx.build_incremental(0, *sched.full[0])
    for b in range(1, n_adv + 1):
        ctx.build_advance(*sched.steps[b * S - 1])     # the finished block's rows as its last step saw them
    out, lse = new_outputs(wl)
    qb, kb, vb = sched.steps[n_adv * S]
    ctx.step(qb, kb, vb, out, lse)
    torch.cuda.synchronize()
    st, msg = ctx.poll_status()
    assert st == 0, msg
    cu = wl.cu_seqlens
    rows = torch.cat([torch.arange(cu[b] + P + n_adv * wl.block_len, cu[b] + P + (n_adv + 1) * wl.block_len)
                      for b, P in enumerate(wl.prompt_lens)]).cuda()
    qf, kf, vf = (x.clone() for x in sched.full[n_adv])
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
    assert np.abs(lse[t_idx].cpu().numpy() - rlse).max() <= TOL["bf16"][0]
    ctx.destroy()
