"""Pins of the sampling-stage oracle (oracle/sampler.py) to things other than itself: hand-computed
values, closed forms, invariants, a library routine, and the truncation property."""
import numpy as np
import scipy.special

from oracle import sampler


def test_hand_values():
    # two tokens with logits 0 and ln 3: probabilities 1/4 and 3/4
    x = np.array([[0.0, np.log(3.0)]])
    tok, conf, lse = sampler.block_confidence(x, [0])
    assert tok[0] == 1 and abs(conf[0] - 0.75) < 1e-15 and abs(lse[0] - np.log(4.0)) < 1e-15
    # three tokens, logits ln 1, ln 2, ln 5 in another order: p = 2/8, 5/8, 1/8
    x = np.log(np.array([[2.0, 5.0, 1.0]]))
    tok, conf, lse = sampler.block_confidence(x, [0])
    assert tok[0] == 1 and abs(conf[0] - 0.625) < 1e-15 and abs(lse[0] - np.log(8.0)) < 1e-15


def test_uniform_logits_and_ties():
    V = 1000
    x = np.full((2, V), -3.25)
    tok, conf, lse = sampler.block_confidence(x, [1])
    assert tok[0] == 0                      # all equal: the lowest id
    assert abs(conf[0] - 1.0 / V) < 1e-18
    assert abs(lse[0] - (np.log(V) - 3.25)) < 1e-12
    x[1, [17, 400, 999]] = 2.0              # three equal maxima: the first of them
    tok, conf, _ = sampler.block_confidence(x, [1])
    assert tok[0] == 17
    e = np.exp(2.0 + 3.25)
    assert abs(conf[0] - e / (3 * e + V - 3)) < 1e-15


def test_shift_invariance_and_large_logits():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(3, 257)) * 4
    t0, c0, l0 = sampler.block_confidence(x, [0, 1, 2])
    t1, c1, l1 = sampler.block_confidence(x + 700.0, [0, 1, 2])     # exp(700 + x) alone would overflow
    assert np.array_equal(t0, t1) and np.abs(c0 - c1).max() < 1e-13 and np.abs(l1 - l0 - 700.0).max() < 1e-10
    assert np.all(np.isfinite(c1)) and np.all(c1 > 0) and np.all(c1 <= 1)


def test_against_library_softmax():
    rng = np.random.default_rng(1)
    x = rng.normal(size=(5, 4099)) * 6
    rows = [4, 0, 2]
    tok, conf, lse = sampler.block_confidence(x, rows)
    p = scipy.special.softmax(x[rows], axis=-1)
    assert np.array_equal(tok, p.argmax(-1))
    assert np.abs(conf - p.max(-1)).max() < 1e-14
    assert np.abs(lse - scipy.special.logsumexp(x[rows], axis=-1)).max() < 1e-12
    # the confidence is exp(x_max - lse)
    assert np.abs(conf - np.exp(x[rows].max(-1) - lse)).max() < 1e-14


def test_truncation_reads_only_the_listed_rows():
    rng = np.random.default_rng(2)
    x = rng.normal(size=(6, 64))
    rows = [1, 4]
    a = sampler.block_confidence(x, rows)
    y = x.copy()
    y[[0, 2, 3, 5]] = np.nan                 # rows outside the block may hold anything
    b = sampler.block_confidence(y, rows)
    for u, v in zip(a, b):
        assert np.array_equal(u, v)
    assert a[0].shape == (2,)
    tok, conf, lse = sampler.block_confidence(x, [])
    assert tok.shape == (0,) and conf.shape == (0,) and lse.shape == (0,)
