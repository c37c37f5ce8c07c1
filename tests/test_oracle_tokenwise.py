"""Pins of the token-wise oracle (embedding, RMS norm, Q/K/V projections;
Sec. 3.3.2) against things it does not compute itself: hand-worked values,
closed forms, invariants, brute-force loops, and a library conversion."""
import math

import numpy as np
import torch

from oracle import tokenwise as tw


def test_round_bf16_hand_values_and_ties():
    # bf16 keeps 8 significant bits: the spacing in [1, 2) is 2^-7
    u = 2.0 ** -7
    cases = [
        (1.0, 1.0), (1.0 + u, 1.0 + u),
        (1.0 + 0.5 * u, 1.0),            # tie -> even significand (1.0)
        (1.0 + 1.5 * u, 1.0 + 2 * u),    # tie -> even significand
        (1.0 + 0.5 * u + 1e-9, 1.0 + u),
        (1.0 + 0.49 * u, 1.0),
        (-3.0 - 0.5 * 2 * u, -3.0),      # spacing in [2, 4) is 2^-6; tie to the even neighbour
        (0.0, 0.0), (2.0 ** -20 * (1 + 3 * u), 2.0 ** -20 * (1 + 3 * u)),
        (255.5, 256.0), (256.0 + 1.0, 256.0), (256.0 + 3.0, 260.0),
    ]
    for x, want in cases:
        assert tw.round_bf16(x) == want, (x, float(tw.round_bf16(x)), want)


def test_round_bf16_matches_library_conversion():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    got = tw.round_bf16(x.astype(np.float64))
    assert np.array_equal(got, want)
    # idempotent, and the error is at most half a unit in the last place
    assert np.array_equal(tw.round_bf16(got), got)
    assert np.all(np.abs(got - x) <= np.abs(x) * 2.0 ** -8)


def test_embed_is_a_row_gather():
    table = np.arange(7 * 3, dtype=np.float64).reshape(7, 3)
    h = tw.embed(table, [6, 0, 0, 3])
    assert np.array_equal(h, np.array([[18, 19, 20], [0, 1, 2], [0, 1, 2], [9, 10, 11]], dtype=np.float64))
    for bad in ([7], [-1]):
        try:
            tw.embed(table, bad)
        except IndexError:
            continue
        raise AssertionError("out-of-range id accepted")


def test_rms_norm_hand_example_and_invariants():
    # h = (3, 4): mean square 12.5, rms = sqrt(12.5)
    out = tw.rms_norm(np.array([[3.0, 4.0]]), np.array([1.0, 2.0]), 0.0)
    assert np.allclose(out, [[3 / math.sqrt(12.5), 8 / math.sqrt(12.5)]], rtol=1e-15)
    rng = np.random.default_rng(1)
    h = rng.standard_normal((5, 64)) * rng.uniform(0.1, 30, (5, 1))
    w = rng.uniform(0.5, 1.5, 64)
    one = tw.rms_norm(h, np.ones(64), 0.0)
    assert np.allclose(np.mean(one * one, axis=-1), 1.0, rtol=1e-13)          # unit mean square
    assert np.allclose(tw.rms_norm(7.5 * h, w, 0.0), tw.rms_norm(h, w, 0.0), rtol=1e-13)  # scale-free
    assert np.allclose(tw.rms_norm(h, w, 0.0), one * w, rtol=1e-15)            # weight is a plain scale
    # eps enters under the root, added to the mean square
    c = np.full((1, 16), 2.0)
    assert np.allclose(tw.rms_norm(c, np.ones(16), 5.0), 2.0 / 3.0, rtol=1e-15)
    # per token: permuting tokens permutes rows
    perm = np.array([3, 0, 4, 1, 2])
    assert np.array_equal(tw.rms_norm(h[perm], w, 1e-5), tw.rms_norm(h, w, 1e-5)[perm])


def test_projection_orientation_and_head_split_by_hand():
    # d_model 3, one q head, one kv head, head_dim 2: rows of w are output features
    w = np.array([[1, 0, 0], [0, 2, 0],        # q features 0, 1
                  [0, 0, 3], [1, 1, 1],        # k features 0, 1
                  [1, -1, 0], [0, 1, -1]], dtype=np.float64)   # v features 0, 1
    x = np.array([[1.0, 10.0, 100.0], [2.0, 3.0, 5.0]])
    q, k, v = tw.qkv_project(x, w, 1, 1, 2)
    assert q.shape == (2, 1, 2) and k.shape == (2, 1, 2) and v.shape == (2, 1, 2)
    assert np.array_equal(q[:, 0], [[1, 20], [2, 6]])
    assert np.array_equal(k[:, 0], [[300, 111], [15, 10]])
    assert np.array_equal(v[:, 0], [[-9, -90], [-1, -2]])


def test_projection_matches_brute_force_loops_with_gqa_split():
    rng = np.random.default_rng(2)
    n, dm, hq, hkv, d = 3, 10, 4, 2, 4
    x = rng.standard_normal((n, dm))
    w = rng.standard_normal(((hq + 2 * hkv) * d, dm))
    q, k, v = tw.qkv_project(x, w, hq, hkv, d)
    for t in range(n):
        for h in range(hq):
            for c in range(d):
                s = sum(x[t, i] * w[h * d + c, i] for i in range(dm))
                assert abs(q[t, h, c] - s) < 1e-12
        for h in range(hkv):
            for c in range(d):
                sk = sum(x[t, i] * w[(hq + h) * d + c, i] for i in range(dm))
                sv = sum(x[t, i] * w[(hq + hkv + h) * d + c, i] for i in range(dm))
                assert abs(k[t, h, c] - sk) < 1e-12 and abs(v[t, h, c] - sv) < 1e-12


def test_chain_special_cases():
    rng = np.random.default_rng(3)
    vocab, dm, hq, hkv, d = 11, 8, 1, 1, 2
    table = rng.standard_normal((vocab, dm))
    # selector weights: every output feature copies one normalised channel
    sel = [0, 5, 2, 2, 7, 1]
    w = np.zeros((6, dm))
    w[np.arange(6), sel] = 1.0
    ids = np.array([4, 4, 10, 0])
    h, q, k, v = tw.tokenwise_qkv(table, np.ones(dm), w, 0.0, hq, hkv, d, token_ids=ids, model_precision=False)
    assert np.array_equal(h, table[ids])
    hn = table[ids] / np.sqrt(np.mean(table[ids] ** 2, axis=-1, keepdims=True))
    assert np.allclose(np.concatenate([q[:, 0], k[:, 0], v[:, 0]], axis=1), hn[:, sel], rtol=1e-14)
    # the same token gives the same rows; hidden-state entry equals the id entry
    assert np.array_equal(q[0], q[1])
    h2, q2, k2, v2 = tw.tokenwise_qkv(table, np.ones(dm), w, 0.0, hq, hkv, d, hidden=table[ids], model_precision=False)
    assert np.array_equal(q2, q) and np.array_equal(k2, k) and np.array_equal(v2, v)
    # model precision: outputs lie on the bf16 grid and stay within the two roundings of the exact
    # result (each at most 2^-9 relative; selector weights add no accumulation error)
    _, qb, kb, vb = tw.tokenwise_qkv(table, np.ones(dm), w, 0.0, hq, hkv, d, token_ids=ids)
    for a, b in ((qb, q), (kb, k), (vb, v)):
        assert np.array_equal(tw.round_bf16(a), a)
        assert np.all(np.abs(a - b) <= np.abs(b) * (2.0 ** -8 + 2.0 ** -16))
    # linear in the norm weight: doubling it doubles the unrounded projections
    _, q3, _, _ = tw.tokenwise_qkv(table, 2 * np.ones(dm), w, 0.0, hq, hkv, d, token_ids=ids, model_precision=False)
    assert np.allclose(q3, 2 * q, rtol=1e-15)
