"""GPU parity of the token-wise producer (embedding gather, RMS norm, Q/K/V
projection on tcgen05; Sec. 3.3.2) against the fp64 oracle, through the C ABI.

Tolerance.  The oracle rounds the norm output and the projections once each to
bf16 ("model precision").  The kernels evaluate the norm in fp32 and accumulate
the projection in fp32 before the same two roundings, so the two can differ in
two ways only.  (1) The fp32 projection falls on the other side of a bf16
rounding boundary: one bf16 unit in the last place of the result, at most
2^-7 relative.  (2) The same happens to an element i of the normalised row
(about one element in 10^4): that operand moves by at most 2^-7 |h^_i|, and
every projection of that token by at most 2^-7 |h^_i w_fi|; two such elements
per token are allowed for, each bounded by max_i |h^_i| max_i |w_fi|.  Both
are rare, so besides the bound at most 3 % of the elements may differ at all.
"""
import numpy as np
import pytest
import torch

from oracle import tokenwise as tw
import oracle
from paper_2607_16339_b200 import binding, workloads as W
from paper_2607_16339_b200.workloads import SyntheticSchedule, TokenModel

from lacache_testlib import TOL, make_ctx, new_outputs

pytestmark = pytest.mark.gpu


def dev_bf16(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda().to(torch.bfloat16).contiguous()


def make_producer(tm, max_tokens, with_table=True):
    wl = tm.wl
    return binding.QkvProducer(dev_bf16(tm.embed) if with_table else None, dev_bf16(tm.norm_weight),
                               dev_bf16(tm.w_qkv), wl.n_q_heads, wl.n_kv_heads, wl.head_dim, tm.rms_eps,
                               max_tokens)


def project(prod, tm, n, ids=None, hidden=None, want_h=False):
    wl = tm.wl
    q = torch.full((n, wl.n_q_heads, wl.head_dim), float("nan"), device="cuda", dtype=torch.bfloat16)
    k = torch.full((n, wl.n_kv_heads, wl.head_dim), float("nan"), device="cuda", dtype=torch.bfloat16)
    v = torch.full_like(k, float("nan"))
    h = torch.full((n, tm.d_model), float("nan"), device="cuda", dtype=torch.bfloat16) if want_h else None
    prod.project(n, q, k, v, token_ids=None if ids is None else torch.from_numpy(ids).cuda(),
                 hidden=None if hidden is None else dev_bf16(hidden), h_out=h)
    torch.cuda.synchronize()
    st, msg = prod.poll_status()
    return st, msg, q, k, v, h


def check_rows(got, ref, flip_bound, what):
    """got: bf16 tensor from the GPU; ref: the oracle's bf16-rounded fp64 array [n, H, d];
    flip_bound [n, H, d]: what one moved element of the normalised row can change."""
    g = got.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(g).all(), what
    diff = np.abs(g - ref)
    bound = np.abs(ref) * 2.0 ** -7 + 2.0 * flip_bound + 1e-30
    assert np.all(diff <= bound), "%s: max excess %.3g" % (what, (diff - bound).max())
    frac = np.mean(diff != 0)
    assert frac <= 0.03, "%s: %.2f%% of the elements differ" % (what, 100 * frac)
    return frac


def check_qkv(tm, q, k, v, ids=None, hidden=None, what=""):
    wl = tm.wl
    h, qr, kr, vr = oracle_qkv(tm, ids=ids, hidden=hidden)
    hmax = np.abs(tw.round_bf16(tw.rms_norm(h, tm.norm_weight, tm.rms_eps))).max(axis=1)   # [n]
    wmax = np.abs(tm.w_qkv.astype(np.float64)).max(axis=1).reshape(-1, wl.head_dim)     # [Hq + 2 Hkv, d]
    nq, nk = wl.n_q_heads, wl.n_kv_heads
    for got, ref, wm, name in ((q, qr, wmax[:nq], "q"), (k, kr, wmax[nq:nq + nk], "k"),
                               (v, vr, wmax[nq + nk:], "v")):
        check_rows(got, ref, 2.0 ** -7 * hmax[:, None, None] * wm[None], "%s %s" % (name, what))
    return h


def oracle_qkv(tm, ids=None, hidden=None):
    wl = tm.wl
    return tw.tokenwise_qkv(tm.embed, tm.norm_weight, tm.w_qkv, tm.rms_eps, wl.n_q_heads, wl.n_kv_heads,
                            wl.head_dim, token_ids=ids, hidden=hidden)


@pytest.fixture(scope="module")
def small_model():
    return TokenModel(W.small_workload(hq=4, hkv=2), 256, 1000)


@pytest.mark.parametrize("n", [1, 17, 32, 40, 100, 256, 300])
def test_projection_small_model(small_model, n):
    """Reduced width: 8 feature tiles x 4 k chunks, fewer chunks than SMs at small n (every tile is
    split over several CTAs), two ragged token tiles at n = 300."""
    tm = small_model
    prod = make_producer(tm, 300)
    ids = np.random.default_rng(n).integers(0, tm.vocab, n).astype(np.int32)
    st, msg, q, k, v, h = project(prod, tm, n, ids=ids, want_h=True)
    assert st == binding.OK, msg
    assert prod.last_launch_count == 2
    hr = check_qkv(tm, q, k, v, ids=ids, what="n=%d" % n)
    assert np.array_equal(h.float().cpu().numpy(), hr.astype(np.float32))   # the gather is exact
    prod.destroy()


@pytest.mark.parametrize("n", [32, 300])
def test_a_bounded_wait_that_runs_out_is_reported_and_the_handle_stays_usable(small_model, n):
    """Every device-side wait is bounded.  Here one is made to run out without any fault: the projection
    kernel is launched without the norm kernel that publishes its operand rows, with the bound set to
    about a millisecond.  Its thread blocks give up, unwind and return; the status word says time-out and
    where; the outputs are untouched; and the next ordinary projection on the same handle is correct."""
    import time
    tm = small_model
    prod = make_producer(tm, 300)
    ids = np.random.default_rng(3 * n).integers(0, tm.vocab, n).astype(np.int32)
    st, msg, q, k, v, _ = project(prod, tm, n, ids=ids)          # an ordinary call first
    assert st == binding.OK, msg
    prod.set_wait_limit(1000.0)
    wl = tm.wl
    qx = torch.full((n, wl.n_q_heads, wl.head_dim), 7.0, device="cuda", dtype=torch.bfloat16)
    kx = torch.full((n, wl.n_kv_heads, wl.head_dim), 7.0, device="cuda", dtype=torch.bfloat16)
    vx = torch.full_like(kx, 7.0)
    hidden = torch.zeros(n, tm.d_model, device="cuda", dtype=torch.bfloat16)
    t0 = time.perf_counter()
    prod.project_without_norm(n, qx, kx, vx, hidden)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 1.0                         # gave up after about a millisecond, not two seconds
    st, msg = prod.poll_status()
    assert st == binding.ERR_TIMEOUT, (st, msg)
    assert "location" in msg
    assert (qx == 7.0).all() and (kx == 7.0).all() and (vx == 7.0).all()    # nothing was written
    assert prod.poll_status()[0] == binding.OK                    # the status word is cleared by the read
    prod.set_wait_limit(0.0)
    st, msg, q2, k2, v2, _ = project(prod, tm, n, ids=ids)        # and the handle works as before
    assert st == binding.OK, msg
    assert torch.equal(q, q2) and torch.equal(k, k2) and torch.equal(v, v2)
    check_qkv(tm, q2, k2, v2, ids=ids, what="after a time-out, n=%d" % n)
    prod.destroy()


@pytest.fixture(scope="module")
def llada_model():
    return TokenModel(W.WORKLOADS[2], 4096, 4096)


@pytest.mark.parametrize("n", [32, 256])
def test_projection_llada_width(llada_model, n):
    """LLaDA-8B first-layer width (4096 -> 3 x 4096), the token counts of one step of the
    single-sequence and the 8-sequence configurations: 96 feature tiles x 64 k chunks dealt
    stream-K over all SMs."""
    tm = llada_model
    prod = make_producer(tm, 256)
    ids = tm.block_ids(1, 5)[:n] if n <= 32 else np.random.default_rng(7).integers(0, tm.vocab, n).astype(np.int32)
    st, msg, q, k, v, _ = project(prod, tm, n, ids=ids)
    assert st == binding.OK, msg
    check_qkv(tm, q, k, v, ids=ids, what="n=%d" % n)
    # equal inputs give equal bits, whatever the arrival order of the partial tiles
    st, msg, q2, k2, v2, _ = project(prod, tm, n, ids=ids)
    assert torch.equal(q, q2) and torch.equal(k, k2) and torch.equal(v, v2)
    prod.destroy()


def test_projection_gqa_width_many_tokens():
    """Dream-7B-like width (3584 -> (28 + 2 x 4) x 128) over 768 tokens: three full token tiles per
    feature tile, most tiles whole inside one CTA."""
    wl = W.small_workload(name="dream-width", hq=28, hkv=4, scale_mode="inv_sqrt_d", theta=1.0e6)
    tm = TokenModel(wl, 3584, 2048)
    n = 768
    prod = make_producer(tm, n)
    ids = np.random.default_rng(11).integers(0, tm.vocab, n).astype(np.int32)
    st, msg, q, k, v, _ = project(prod, tm, n, ids=ids)
    assert st == binding.OK, msg
    check_qkv(tm, q, k, v, ids=ids)
    prod.destroy()


def test_hidden_state_entry_and_bad_token_id(small_model):
    tm = small_model
    n = 48
    prod = make_producer(tm, 64)
    ids = np.random.default_rng(5).integers(0, tm.vocab, n).astype(np.int32)
    st, msg, q, k, v, _ = project(prod, tm, n, ids=ids)
    assert st == binding.OK, msg
    st, msg, q2, k2, v2, _ = project(prod, tm, n, hidden=tm.embed[ids])
    assert st == binding.OK, msg
    assert torch.equal(q, q2) and torch.equal(k, k2) and torch.equal(v, v2)
    # a producer without a table takes hidden states only
    prod2 = make_producer(tm, 64, with_table=False)
    st, msg, q3, _, _, _ = project(prod2, tm, n, hidden=tm.embed[ids])
    assert st == binding.OK and torch.equal(q, q3)
    with pytest.raises(binding.LacacheError) as e:
        project(prod2, tm, n, ids=ids)
    assert e.value.status == binding.ERR_STATE
    prod2.destroy()
    # an id outside the table: reported, its rows zero, the others right, the handle still usable
    bad = ids.copy()
    bad[7] = tm.vocab
    st, msg, qb, kb, vb, _ = project(prod, tm, n, ids=bad)
    assert st == binding.ERR_INVALID_ARG and "row 7" in msg, (st, msg)
    assert float(qb[7].float().abs().max()) == 0.0 and float(vb[7].float().abs().max()) == 0.0
    keep = np.arange(n) != 7
    assert torch.equal(qb[torch.from_numpy(keep).cuda()], q[torch.from_numpy(keep).cuda()])
    st, msg, q4, _, _, _ = project(prod, tm, n, ids=ids)
    assert st == binding.OK and torch.equal(q, q4)
    # argument checks
    for kw in (dict(), dict(ids=ids, hidden=tm.embed[ids])):
        with pytest.raises(binding.LacacheError) as e:
            project(prod, tm, n, **kw)
        assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.LacacheError) as e:
        project(prod, tm, 65, ids=np.zeros(65, np.int32))
    assert e.value.status == binding.ERR_SHAPE
    prod.destroy()


@pytest.mark.parametrize("shape", ["mha", "gqa-ragged", "mha-fp16"])
def test_build_and_step_from_token_ids(shape):
    """Algorithm 1 fed by token ids: build_tokens over all T tokens, then step_tokens over the block's
    tokens; checked against the oracle chain (token-wise oracle at model precision -> attention
    oracle) and, bit for bit, against lacache_build / lacache_step fed with the projected rows."""
    ctx_kw = dict(precision_mode=binding.PRECISION_FP16) if shape == "mha-fp16" else {}
    if shape in ("mha", "mha-fp16"):
        wl = W.small_workload(prompt_lens=(200,), gen_len=96, block_len=32, steps=3, hq=4, hkv=4)
    else:
        wl = W.small_workload(prompt_lens=(150, 61), gen_len=128, block_len=64, steps=2, hq=8, hkv=2,
                              scale_mode="inv_sqrt_d")
    tm = TokenModel(wl, 512, 3000)
    T, nb = wl.total_tokens, wl.batch * wl.block_len
    prod = make_producer(tm, T)
    ctx = make_ctx(wl, **ctx_kw)
    ctx2 = make_ctx(wl, **ctx_kw)
    sch = SyntheticSchedule(wl)   # index sets only
    b = 1
    ids_full = tm.full_ids(b)
    ctx.build_tokens(prod, b, token_ids=torch.from_numpy(ids_full).cuda())
    _, qf, kf, vf = oracle_qkv(tm, ids=ids_full)
    rows = sch.block_rows(b)
    scale = wl.head_dim ** -0.5
    # the same build through the plain entry point, from the producer's own rows
    st, msg, qg, kg, vg, _ = project(prod, tm, T, ids=ids_full)
    assert st == binding.OK, msg
    ctx2.build(b, qg, kg, vg)
    for s in (1, wl.steps_per_block):
        ids_blk = tm.block_ids(b, s)
        out, lse = new_outputs(wl)
        ctx.step_tokens(prod, out, lse, blk_token_ids=torch.from_numpy(ids_blk).cuda())
        torch.cuda.synchronize()
        assert ctx.poll_status()[0] == binding.OK and prod.poll_status()[0] == binding.OK
        assert ctx.last_launch_count == 4
        _, qb, kb, vb = oracle_qkv(tm, ids=ids_blk)
        qf[rows], kf[rows], vf[rows] = qb, kb, vb
        ref, rlse = oracle.attention(qf, kf, vf, wl.cu_seqlens, wl.rope_theta, scale)
        err = np.abs(out.cpu().numpy().astype(np.float64) - ref)
        assert err.max() <= TOL["bf16"][0] and err.mean() <= TOL["bf16"][1], (err.max(), err.mean())
        assert np.abs(lse.cpu().numpy() - rlse).max() <= TOL["bf16"][0]
        st, msg, qgb, kgb, vgb, _ = project(prod, tm, nb, ids=ids_blk)
        out2, lse2 = new_outputs(wl)
        ctx2.step(qgb, kgb, vgb, out2, lse2)
        torch.cuda.synchronize()
        assert torch.equal(out, out2) and torch.equal(lse, lse2)
    # a producer whose heads do not fit the context is refused
    other = TokenModel(W.small_workload(hq=4, hkv=1), 512, 100)
    prod_bad = make_producer(other, 64)
    out, lse = new_outputs(wl)
    with pytest.raises(binding.LacacheError) as e:
        ctx.step_tokens(prod_bad, out, lse, blk_token_ids=torch.zeros(nb, dtype=torch.int32, device="cuda"))
    assert e.value.status == binding.ERR_SHAPE
    for o in (prod_bad, prod, ctx, ctx2):
        o.destroy()


def test_build_update_reprojects_only_changed_rows():
    """From one block to the next only the finished block's tokens change: an update that re-projects
    those rows alone must leave the context in the state a build from all T token ids leaves it in.
    Untouched rows are bit-identical.  Re-projected rows may differ in the last bf16 place in a few
    elements (the reduction over d_model is split over the SMs differently for 64 tokens than for T,
    so the fp32 sums round differently); a step taken from either state meets the oracle tolerance."""
    wl = W.small_workload(prompt_lens=(130, 75), gen_len=96, block_len=32, steps=2, hq=8, hkv=4)
    tm = TokenModel(wl, 384, 2000)
    T, nb = wl.total_tokens, wl.batch * wl.block_len
    sch = SyntheticSchedule(wl)   # index sets only
    prod_a, prod_b = make_producer(tm, T), make_producer(tm, T)
    ctx_a, ctx_b = make_ctx(wl), make_ctx(wl)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    ids0, ids1 = tm.full_ids(0).copy(), tm.full_ids(1).copy()
    rows = sch.block_rows(0).astype(np.int32)
    ids0[rows] = tm.mask_id                       # block 0 still masked at its build
    assert np.array_equal(np.flatnonzero(ids0 != ids1), np.sort(rows))
    # an update needs the all-token rows of a preceding build of the same pair
    with pytest.raises(binding.LacacheError) as e:
        ctx_a.build_tokens_update(prod_a, 1, dev(rows), token_ids=dev(ids1[rows]))
    assert e.value.status == binding.ERR_STATE
    ctx_a.build_tokens(prod_a, 0, token_ids=dev(ids0))
    out, lse = new_outputs(wl)
    ctx_a.step_tokens(prod_a, out, lse, blk_token_ids=dev(tm.block_ids(0, 1)))   # block scratch must not disturb it
    perm = np.random.default_rng(3).permutation(len(rows))                        # any order of the changed rows
    ctx_a.build_tokens_update(prod_a, 1, dev(rows[perm]), token_ids=dev(ids1[rows[perm]]))
    assert ctx_a.last_launch_count == 4
    ctx_b.build_tokens(prod_b, 1, token_ids=dev(ids1))
    caches = []
    for ctx in (ctx_a, ctx_b):
        qr = torch.empty(T, wl.n_q_heads, wl.head_dim, device="cuda")
        kr = torch.empty(T, wl.n_kv_heads, wl.head_dim, device="cuda")
        vr = torch.empty_like(kr)
        ctx.export_rope_cache(qr, kr, vr)
        caches.append((qr, kr, vr))
    keep = torch.ones(T, dtype=torch.bool, device="cuda")
    keep[torch.from_numpy(rows.astype(np.int64)).cuda()] = False
    for x, y in zip(*caches):
        assert torch.equal(x[keep], y[keep])
        d = (x[~keep] - y[~keep]).abs()
        assert float(d.max()) <= 2.0 ** -7 * float(y[~keep].abs().max())
        assert float((d != 0).float().mean()) <= 0.03
    ids_blk = dev(tm.block_ids(1, 2))
    res = []
    for ctx, prod in ((ctx_a, prod_a), (ctx_b, prod_b)):
        out, lse = new_outputs(wl)
        ctx.step_tokens(prod, out, lse, blk_token_ids=ids_blk)
        torch.cuda.synchronize()
        res.append((out, lse))
    _, qf, kf, vf = oracle_qkv(tm, ids=ids1)
    _, qb, kb, vb = oracle_qkv(tm, ids=tm.block_ids(1, 2))
    brows = sch.block_rows(1)
    qf[brows], kf[brows], vf[brows] = qb, kb, vb
    ref, rlse = oracle.attention(qf, kf, vf, wl.cu_seqlens, wl.rope_theta, wl.head_dim ** -0.5)
    for out, lse in res:
        err = np.abs(out.cpu().numpy().astype(np.float64) - ref)
        assert err.max() <= TOL["bf16"][0] and err.mean() <= TOL["bf16"][1], (err.max(), err.mean())
        assert np.abs(lse.cpu().numpy() - rlse).max() <= TOL["bf16"][0]
    assert float((res[0][0] - res[1][0]).abs().max()) <= TOL["bf16"][0]
    # hidden-state entry of the update, and n_changed = 0
    ctx_a.build_tokens_update(prod_a, 1, dev(rows), hidden=dev_bf16(tm.embed[ids1[rows]]))
    ctx_a.build_tokens_update(prod_a, 1, dev(rows[:0]), token_ids=dev(ids1[:0]))
    out, lse = new_outputs(wl)
    ctx_a.step_tokens(prod_a, out, lse, blk_token_ids=ids_blk)
    torch.cuda.synchronize()
    assert torch.equal(out, res[0][0])      # the same update again: the same bits
    # a row outside [0, T): reported, dropped, the other rows still written
    bad = rows.copy()
    bad[3] = T
    ctx_a.build_tokens_update(prod_a, 1, dev(bad), token_ids=dev(ids1[rows]))
    torch.cuda.synchronize()
    st, msg = prod_a.poll_status()
    assert st == binding.ERR_INVALID_ARG and "destination row" in msg, (st, msg)
    # another context's build with the same producer invalidates the kept rows
    ctx_b.build_tokens(prod_a, 1, token_ids=dev(ids1))
    with pytest.raises(binding.LacacheError) as e:
        ctx_a.build_tokens_update(prod_a, 1, dev(rows), token_ids=dev(ids1[rows]))
    assert e.value.status == binding.ERR_STATE
    assert ctx_a.poll_status()[0] == binding.OK and ctx_b.poll_status()[0] == binding.OK
    for o in (prod_a, prod_b, ctx_a, ctx_b):
        o.destroy()


@pytest.mark.parametrize("d_model,hq,hkv,n", [(64, 1, 1, 1), (64, 2, 1, 33), (192, 3, 1, 257), (1024, 6, 2, 130),
                                              (8192, 2, 2, 20)])
def test_projection_odd_shapes(d_model, hq, hkv, n):
    """Corners of the work split: a single k chunk per tile (every segment covers its tile alone),
    fewer chunks than SMs, one token, token counts just past a tile, the widest row the norm
    kernel takes."""
    wl = W.small_workload(name="odd", hq=hq, hkv=hkv, scale_mode="inv_sqrt_d")
    tm = TokenModel(wl, d_model, 300, seed=d_model + n)
    prod = make_producer(tm, n)
    ids = np.random.default_rng(n).integers(0, tm.vocab, n).astype(np.int32)
    st, msg, q, k, v, h = project(prod, tm, n, ids=ids, want_h=True)
    assert st == binding.OK, msg
    hr = check_qkv(tm, q, k, v, ids=ids, what="d_model=%d n=%d" % (d_model, n))
    assert np.array_equal(h.float().cpu().numpy(), hr.astype(np.float32))
    st, msg, q2, k2, v2, _ = project(prod, tm, n, ids=ids)
    assert torch.equal(q, q2) and torch.equal(k, k2) and torch.equal(v, v2)
    prod.destroy()


@pytest.mark.parametrize("overlap", [True, False])
def test_back_to_back_token_steps_match_synchronised_ones(overlap):
    """Token-fed steps issued without any host synchronisation (with the overlap of consecutive steps
    switched on, the norm kernel of a step runs alongside the previous step's attention kernel) give,
    bit for bit, what the same calls give when the host waits after each."""
    wl = W.small_workload(prompt_lens=(300, 170), gen_len=64, block_len=32, steps=6, hq=8, hkv=4)
    tm = TokenModel(wl, 512, 1500)
    T = wl.total_tokens
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    ids_full = dev(tm.full_ids(0))
    ids_steps = [dev(tm.block_ids(0, s)) for s in range(1, wl.steps_per_block + 1)]

    def run(sync):
        prod = make_producer(tm, T)
        ctx = make_ctx(wl)
        ctx.set_step_overlap(overlap)
        ctx.build_tokens(prod, 0, token_ids=ids_full)
        res = []
        for ids in ids_steps:
            out, lse = new_outputs(wl)
            ctx.step_tokens(prod, out, lse, blk_token_ids=ids)
            if sync:
                torch.cuda.synchronize()
            res.append((out, lse))
        torch.cuda.synchronize()
        assert ctx.poll_status()[0] == binding.OK and prod.poll_status()[0] == binding.OK
        ctx.destroy()
        prod.destroy()
        return res

    ref = run(True)
    for rep in range(3):
        got = run(False)
        for i, ((o0, l0), (o1, l1)) in enumerate(zip(ref, got)):
            assert torch.equal(o0, o1) and torch.equal(l0, l1), "step %d differs when issued back to back" % i
