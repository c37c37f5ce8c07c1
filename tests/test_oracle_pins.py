"""Pins for the fp64 oracle: every check here is against something other than
the oracle itself (hand-derived closed forms, brute force written a different
way, a library routine, algebraic invariants of Eq. 1-6)."""
import numpy as np
import pytest
import torch

import oracle


def _complex_rope(x, pos, theta):
    """Independent restatement of Eq. 1: pair (c, c+d/2) as a complex number
    and multiply by e^{i p theta^(-2c/d)}."""
    T, H, d = x.shape
    half = d // 2
    z = x[..., :half] + 1j * x[..., half:]
    f = theta ** (-2.0 * np.arange(half) / d)
    ang = np.asarray(pos, dtype=np.float64)[:, None, None] * f[None, None, :]
    z = z * np.exp(1j * ang)
    return np.concatenate([z.real, z.imag], axis=-1)


def _brute(q, k, v, theta, scale):
    """Single sequence, no max subtraction (scores are small), explicit matrices."""
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    pos = np.arange(T)
    qr = _complex_rope(q, pos, theta)
    kr = _complex_rope(k, pos, theta)
    out = np.zeros_like(q)
    lse = np.zeros((T, Hq))
    for h in range(Hq):
        kh = h // (Hq // Hkv)
        e = np.exp(scale * qr[:, h, :] @ kr[:, kh, :].T)
        out[:, h, :] = (e / e.sum(1, keepdims=True)) @ v[:, kh, :]
        lse[:, h] = np.log(e.sum(1))
    return out, lse


def test_hand_worked_two_token_case():
    # d = 2 => single frequency f_0 = 1; tokens at positions 0 and 1.
    # q0 = (1,0) at p=0.  k0 = (1,0) at p=0, k1 = (0,1) at p=1:
    #   R(1) k1 = (-sin 1, cos 1)  =>  s0 = scale, s1 = -scale sin 1.
    # v0 = (1,0), v1 = (0,1) => out(row 0) = (w0, w1), w1 = 1/(1+exp(s0-s1)).
    scale = 0.7
    q = np.array([[[1.0, 0.0]], [[1.0, 0.0]]])
    k = np.array([[[1.0, 0.0]], [[0.0, 1.0]]])
    v = np.array([[[1.0, 0.0]], [[0.0, 1.0]]])
    out, lse = oracle.attention(q, k, v, [0, 2], 10000.0, scale)
    s0, s1 = scale, -scale * np.sin(1.0)
    w1 = 1.0 / (1.0 + np.exp(s0 - s1))
    assert np.allclose(out[0, 0], [1 - w1, w1], atol=1e-14)
    assert np.isclose(lse[0, 0], np.log(np.exp(s0) + np.exp(s1)), atol=1e-14)
    # row 1: q1 = (1,0) at p=1 => R(1) q1 = (cos 1, sin 1);
    #   <R(1)q1, k0> = cos 1 ; <R(1)q1, R(1)k1> = <q1,k1> = 0.
    t0, t1 = scale * np.cos(1.0), 0.0
    u1 = 1.0 / (1.0 + np.exp(t0 - t1))
    assert np.allclose(out[1, 0], [1 - u1, u1], atol=1e-14)


def test_rope_basics():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((9, 3, 16))
    pos = np.array([0, 1, 2, 5, 7, 100, 1000, 4095, 5119], dtype=np.int32)
    y = oracle.rope(x, pos, 5.0e5)
    assert np.array_equal(y[0], x[0])                      # R(0) = I
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)
    assert np.allclose(y, _complex_rope(x, pos, 5.0e5), atol=1e-12)
    # V-style check: the two halves are paired (c, c+d/2), not (2c, 2c+1)
    e = np.zeros((1, 1, 16)); e[0, 0, 3] = 1.0
    r = oracle.rope(e, np.array([1], dtype=np.int32), 100.0)
    f3 = 100.0 ** (-2.0 * 3 / 16)
    expect = np.zeros(16); expect[3] = np.cos(f3); expect[3 + 8] = np.sin(f3)
    assert np.allclose(r[0, 0], expect, atol=1e-15)


def test_rope_relative_and_toeplitz():
    rng = np.random.default_rng(1)
    d = 32
    q = rng.standard_normal((1, 1, d))
    k = rng.standard_normal((1, 1, d))
    n = 12
    pos = np.arange(n, dtype=np.int32)
    Q = oracle.rope(np.repeat(q, n, 0), pos, 1.0e4)[:, 0]
    K = oracle.rope(np.repeat(k, n, 0), pos, 1.0e4)[:, 0]
    S = Q @ K.T
    # identical pre-RoPE vectors => scores depend only on j - i (Toeplitz)
    for off in range(-n + 1, n):
        diag = np.diagonal(S, off)
        assert np.allclose(diag, diag[0], atol=1e-12)
    # shifting every position by a constant leaves all scores unchanged
    Q2 = oracle.rope(np.repeat(q, n, 0), pos + 977, 1.0e4)[:, 0]
    K2 = oracle.rope(np.repeat(k, n, 0), pos + 977, 1.0e4)[:, 0]
    assert np.allclose(Q2 @ K2.T, S, atol=1e-10)


@pytest.mark.parametrize("hq,hkv", [(2, 2), (4, 2), (6, 1)])
def test_brute_force_tiny(hq, hkv):
    rng = np.random.default_rng(2)
    T, d = 7, 4
    q = rng.standard_normal((T, hq, d)) * 0.5
    k = rng.standard_normal((T, hkv, d)) * 0.5
    v = rng.standard_normal((T, hkv, d))
    out, lse = oracle.attention(q, k, v, [0, T], 50.0, 0.5)
    bo, bl = _brute(q, k, v, 50.0, 0.5)
    assert np.allclose(out, bo, atol=1e-13)
    assert np.allclose(lse, bl, atol=1e-13)
    # convex combination of the values
    for h in range(hq):
        vv = v[:, h // (hq // hkv), :]
        assert np.all(out[:, h, :] <= vv.max(0) + 1e-13)
        assert np.all(out[:, h, :] >= vv.min(0) - 1e-13)


def test_closed_forms():
    rng = np.random.default_rng(3)
    T, H, d = 11, 2, 8
    k = rng.standard_normal((T, H, d))
    v = rng.standard_normal((T, H, d))
    # q = 0 -> uniform weights
    out, lse = oracle.attention(np.zeros((T, H, d)), k, v, [0, T], 1.0e4, 0.3)
    assert np.allclose(out, np.broadcast_to(v.mean(0), out.shape), atol=1e-14)
    assert np.allclose(lse, np.log(T), atol=1e-14)
    # all values equal -> that value
    q = rng.standard_normal((T, H, d))
    vc = np.broadcast_to(rng.standard_normal((1, H, d)), (T, H, d))
    out, _ = oracle.attention(q, k, vc, [0, T], 1.0e4, 0.3)
    assert np.allclose(out, vc, atol=1e-14)
    # one dominant key (score 60 above the rest at p = 0 where R = I)
    q1 = np.zeros((1, 1, d)); q1[0, 0, 0] = 1.0
    kk = np.zeros((1, 1, d)); kk[0, 0, 0] = 60.0
    out, lse = oracle.attention(q1, kk, v[:1, :1], [0, 1], 1.0e4, 1.0)
    assert np.allclose(out[0, 0], v[0, 0], atol=1e-14) and np.isclose(lse[0, 0], 60.0)


def test_matches_torch_sdpa_on_rotated_inputs():
    rng = np.random.default_rng(4)
    T, Hq, Hkv, d = 37, 4, 2, 16
    q = rng.standard_normal((T, Hq, d))
    k = rng.standard_normal((T, Hkv, d))
    v = rng.standard_normal((T, Hkv, d))
    theta, scale = 5.0e5, d ** -0.5
    out, _ = oracle.attention(q, k, v, [0, T], theta, scale)
    pos = np.arange(T)
    qr = torch.from_numpy(_complex_rope(q, pos, theta)).permute(1, 0, 2)[None]
    kr = torch.from_numpy(_complex_rope(k, pos, theta)).permute(1, 0, 2)[None]
    vv = torch.from_numpy(v).permute(1, 0, 2)[None]
    kr = kr.repeat_interleave(Hq // Hkv, 1)
    vv = vv.repeat_interleave(Hq // Hkv, 1)
    ref = torch.nn.functional.scaled_dot_product_attention(qr, kr, vv, scale=scale)
    assert np.allclose(out, ref[0].permute(1, 0, 2).numpy(), atol=1e-12)


def test_gqa_equals_repeated_mha_and_packed_equals_alone():
    rng = np.random.default_rng(5)
    lens = [5, 9, 3]
    cu = np.concatenate([[0], np.cumsum(lens)])
    T, Hq, Hkv, d = cu[-1], 6, 2, 8
    q = rng.standard_normal((T, Hq, d))
    k = rng.standard_normal((T, Hkv, d))
    v = rng.standard_normal((T, Hkv, d))
    out, lse = oracle.attention(q, k, v, cu, 1.0e4, 0.4)
    out2, lse2 = oracle.attention(q, np.repeat(k, 3, 1), np.repeat(v, 3, 1), cu, 1.0e4, 0.4)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)
    for b in range(3):
        sl = slice(cu[b], cu[b + 1])
        o1, l1 = oracle.attention(q[sl], k[sl], v[sl], [0, lens[b]], 1.0e4, 0.4)
        assert np.allclose(out[sl], o1, atol=1e-15) and np.allclose(lse[sl], l1, atol=1e-15)
    # row subset selection is consistent
    rows = np.array([16, 0, 7])
    o3, l3 = oracle.attention(q, k, v, cu, 1.0e4, 0.4, rows=rows)
    assert np.array_equal(o3, out[rows]) and np.array_equal(l3, lse[rows])


def test_key_permutation_invariance():
    rng = np.random.default_rng(6)
    n, d = 23, 8
    qr = rng.standard_normal(d)
    kr = rng.standard_normal((n, d))
    v = rng.standard_normal((n, d))
    keep = np.ones(n, dtype=np.uint8)
    m, l, O = oracle.state_stream(qr, kr, v, keep, 0.5, 4)
    p = rng.permutation(n)
    m2, l2, O2 = oracle.state_stream(qr, kr[p], v[p], keep, 0.5, 7)
    assert np.allclose(O / l, O2 / l2, atol=1e-14)
    assert np.isclose(m + np.log(l), m2 + np.log(l2), atol=1e-14)


def test_split_merge_identity_random_partitions():
    rng = np.random.default_rng(7)
    n, d = 41, 8
    for trial in range(20):
        qr = rng.standard_normal(d) * 3
        kr = rng.standard_normal((n, d)) * 3
        v = rng.standard_normal((n, d))
        s = 0.5 * kr @ qr
        w = np.exp(s - s.max()); w /= w.sum()
        ref_out = w @ v
        ref_lse = s.max() + np.log(np.exp(s - s.max()).sum())
        full = oracle.state_stream(qr, kr, v, np.ones(n, np.uint8), 0.5, 5)
        assert np.allclose(full[2] / full[1], ref_out, atol=1e-13)
        assert np.isclose(full[0] + np.log(full[1]), ref_lse, atol=1e-13)
        # random 3-way partition, merged in two different association orders
        lab = rng.integers(0, 3, n)
        parts = [oracle.state_stream(qr, kr, v, (lab == i).astype(np.uint8), 0.5, 1 + trial % 6)
                 for i in range(3)]
        a = oracle.state_merge(oracle.state_merge(parts[0], parts[1]), parts[2])
        b = oracle.state_merge(parts[2], oracle.state_merge(parts[1], parts[0]))
        for st in (a, b):
            assert np.allclose(st[2] / st[1], ref_out, atol=1e-12)
            assert np.isclose(st[0] + np.log(st[1]), ref_lse, atol=1e-12)
        # merging with the empty state is the identity
        e = oracle.state_merge(parts[0], (-np.inf, 0.0, np.zeros(d)))
        assert e[0] == parts[0][0] and e[1] == parts[0][1] and np.array_equal(e[2], parts[0][2])
        e = oracle.state_merge((-np.inf, 0.0, np.zeros(d)), parts[1])
        assert np.allclose(e[2] / e[1], parts[1][2] / parts[1][1], atol=1e-15)
        # continuing the stream from a state == merging
        c = oracle.state_stream(qr, kr, v, (lab != 0).astype(np.uint8), 0.5, 4, state=parts[0])
        assert np.allclose(c[2] / c[1], ref_out, atol=1e-12)


def test_cached_reuse_pass_equals_definition():
    """The paper's exactness claim (Sec. 3.1, 3.3): Algorithm 1's reuse pass on
    the cached state equals the plain definition."""
    from paper_2607_16339_b200.workloads import SyntheticSchedule, small_workload
    wl = small_workload(prompt_lens=(13, 6), gen_len=12, block_len=4, steps=2, hq=4, hkv=2, d=8,
                        theta=1.0e4, dtype="fp32")
    sch = SyntheticSchedule(wl, seed=3)
    cu = wl.cu_seqlens
    scale = wl.head_dim ** -0.5
    for b in range(wl.n_blocks):
        q, k, v = sch.begin_block(b)
        isb = sch.is_block(b)
        state = oracle.build_state(q, k, v, cu, isb, wl.rope_theta, scale, Bc=5)
        # the cached triple is the softmax over fixed keys only
        keep_rows = np.flatnonzero(isb == 0)
        for s in range(1, wl.steps_per_block + 1):
            sch.draw_step(b, s)
            out, lse = oracle.reuse_step(sch.q, sch.k, sch.v, cu, isb, wl.rope_theta, scale, state, Bc=3)
            ref, rl = oracle.attention(sch.q, sch.k, sch.v, cu, wl.rope_theta, scale)
            assert np.allclose(out, ref, atol=1e-13)
            assert np.allclose(lse, rl, atol=1e-13)
        assert keep_rows.size == wl.total_tokens - wl.batch * wl.block_len


def test_empty_fixed_set_state_is_empty():
    # U empty (no prompt, a single block): cached state is (-inf, 0, 0) and the
    # reuse pass still gives the block-only result with no NaN.
    rng = np.random.default_rng(8)
    T, H, d = 4, 1, 4
    q = rng.standard_normal((T, H, d)); k = rng.standard_normal((T, H, d)); v = rng.standard_normal((T, H, d))
    isb = np.ones(T, np.uint8)
    m, l, O = oracle.build_state(q, k, v, [0, T], isb, 1.0e4, 0.5)
    assert np.all(np.isneginf(m)) and np.all(l == 0) and np.all(O == 0)
    out, lse = oracle.reuse_step(q, k, v, [0, T], isb, 1.0e4, 0.5, (m, l, O))
    ref, rl = oracle.attention(q, k, v, [0, T], 1.0e4, 0.5)
    assert np.allclose(out, ref, atol=1e-14) and not np.isnan(out).any()
