"""CPU emulation of the device's rounding points (test-side only): it decided
the precision design, and keeps deciding it.  One head, LLaDA-8B shape, harsh
value scale; reference = the fp64 definition."""
import numpy as np
import torch


def _rope(x, pos, theta):
    d = x.shape[-1]; h = d // 2
    f = theta ** (-2.0 * torch.arange(h, dtype=torch.float64) / d)
    a = pos[:, None].double() * f[None]
    c, s = a.cos(), a.sin()
    return torch.cat([x[:, :h] * c - x[:, h:] * s, x[:, h:] * c + x[:, :h] * s], 1)


_bf = lambda x: x.float().to(torch.bfloat16).double()
_f16 = lambda x: x.float().to(torch.float16).double()


def _emulate(seed, qk_mode, p_round, N=768, P=512, Lb=32, scale_h=2.0, tile=128):
    g = torch.Generator().manual_seed(seed); d = 128
    q, k, v = [_bf(torch.randn(N, d, generator=g, dtype=torch.float64) * scale_h) for _ in range(3)]
    mq, mk, mv = [_bf(torch.randn(d, generator=g, dtype=torch.float64) * scale_h) for _ in range(3)]
    blk0 = P + 2 * Lb
    q[blk0 + Lb:] = mq; k[blk0 + Lb:] = mk; v[blk0 + Lb:] = mv
    pos = torch.arange(N)
    qr, kr = _rope(q, pos, 5e5), _rope(k, pos, 5e5)
    sc = d ** -0.5
    ref = torch.softmax(qr @ kr.T * sc, 1) @ v
    qf, kf = qr.float().double(), kr.float().double()
    if qk_mode == "bf16":
        S = _bf(qf) @ _bf(kf).T
    elif qk_mode == "fp16":
        S = _f16(qf) @ _f16(kf).T
    else:
        qh, kh = _bf(qf), _bf(kf)
        ql, kl = _bf(qf - qh), _bf(kf - kh)
        S = qh @ kh.T + qh @ kl.T + ql @ kh.T
    S = (S.float() * np.float32(sc * 1.4426950408889634)).float()

    def stream(rows, cols_list, state=None):
        n = len(rows)
        if state is None:
            m = torch.full((n,), -float("inf")); l = torch.zeros(n); O = torch.zeros(n, d)
        else:
            m, l, O = [x.clone() for x in state]
        for cols in cols_list:
            s = S[rows][:, cols]
            mn = torch.maximum(m, torch.ceil(s.max(1).values))       # integer reference exponent
            al = torch.exp2(m - mn); al[torch.isinf(m)] = 0
            pq = p_round(torch.exp2(s - mn[:, None]).float())
            l = (al * l + pq.sum(1).float()).float()
            O = (al[:, None] * O + (pq @ v[cols]).float()).float()
            m = mn
        return m, l, O

    allrows = torch.arange(N)
    U = torch.cat([torch.arange(0, blk0), torch.arange(blk0 + Lb, N)])
    C = torch.arange(blk0, blk0 + Lb)
    tiles = lambda idx: [idx[i:i + tile] for i in range(0, len(idx), tile)]
    m, l, O = stream(allrows, tiles(allrows))
    full = (O / l[:, None]).double()
    m2, l2, O2 = stream(U, [C], state=stream(U, tiles(U)))
    m3, l3, O3 = stream(C, tiles(allrows))
    cached = torch.zeros(N, d, dtype=torch.float64)
    cached[U] = (O2 / l2[:, None]).double(); cached[C] = (O3 / l3[:, None]).double()
    err = (cached - ref).abs()
    return err.max().item(), err.mean().item(), (cached - full).abs().max().item()


def test_plain_bf16_operands_miss_the_bar_and_the_split_meets_it():
    emax, emean, _ = _emulate(0, "bf16", _f16)
    assert emax > 2e-2                                  # why rotated Q', K' are stored as hi + lo planes
    for seed in range(2):
        emax, emean, diff = _emulate(seed, "split", _f16)
        assert emax < 1e-2 and emean < 1e-3             # well inside 2e-2 / 2e-3
        assert diff < 1e-3                              # cached path vs full recompute


def test_bf16_probabilities_without_integer_reference_would_break_cached_vs_recompute():
    # with the integer reference exponent the rounding of P is identical on both paths
    _, _, diff = _emulate(0, "split", _bf)
    assert diff < 1e-4


def test_plain_operands_hold_where_the_scores_are_small():
    """Which inputs the plain mode (one bf16 plane of the rotated Q', K', one score product) suits: the
    rounding of an operand to bf16 moves a score by about 2^-9 |s|, so the error against the fp64
    definition grows with the magnitude of the scores.  With q, k ~ N(0,1)/sqrt(d) (the GQA long-context
    configuration; |s| << 1) it is orders of magnitude inside the bar, at per-head scale 1 (|s| ~ 10) still
    a factor of five inside, at scale 2 (|s| ~ 50; the LLaDA-shaped configurations) outside."""
    d = 128
    emax, emean, diff = _emulate(0, "bf16", _f16, scale_h=d ** -0.5)
    assert emax < 1e-3 and emean < 1e-4 and diff < 1e-3
    rows = {}
    for sh in (0.5, 1.0, 2.0):
        rows[sh] = _emulate(0, "bf16", _f16, scale_h=sh)
    assert rows[0.5][0] < 2e-2 and rows[0.5][1] < 2e-3     # scores of order 3: still inside
    assert rows[2.0][0] > 2e-2                             # scores of order 50: outside
    assert rows[0.5][0] < rows[1.0][0] < rows[2.0][0]


def test_one_fp16_plane_holds_at_the_harsh_scale_with_a_smaller_margin_than_the_split():
    """fp16 keeps three more significant bits than bf16, so one fp16 plane per operand moves a score by
    about 2^-12 |s|: at per-head scale 2 (scores of order 50), where one bf16 plane is outside the bar by
    a factor of three, it is inside by a factor of about two on the maximum and four on the mean; the
    split planes are inside by a factor of twenty.  Both paths round alike, so cached and recomputed
    outputs still agree."""
    for seed in range(3):
        emax, emean, diff = _emulate(seed, "fp16", _f16)
        assert emax < 1.2e-2 and emean < 7e-4
        assert diff < 1e-3
        smax, smean, _ = _emulate(seed, "split", _f16)
        assert smax < emax and smean < emean
