"""GPU parity of the sampling-stage truncation (softmax over the vocabulary on the current block's rows
only) against the fp64 oracle, through the C ABI.

Tolerance.  The token is an argmax over the stored logits themselves (no arithmetic): bit-exact, ties to
the lowest id on both sides.  The probability is 1 / sum_v exp(x_v - x_max) in fp32 with the hardware
exp2: each term carries a relative error of about |x_v - x_max| * 2^-23 from the scaled exponent plus
2^-22 from exp2, weighted by the term's share of the sum, and the fp32 sum over threads, warps and slices
adds a few 2^-24: 2e-5 relative (and absolute on the log normaliser) covers vocabularies of 1e5 entries.
"""
import numpy as np
import pytest
import torch

from oracle import sampler
from paper_2607_16339_b200 import binding
from paper_2607_16339_b200.workloads import WORKLOADS, SyntheticSchedule, small_workload

from lacache_testlib import make_ctx, to_dev

pytestmark = pytest.mark.gpu


def _built_ctx(wl, b):
    sch = SyntheticSchedule(wl, seed=4)
    for bb in range(b):
        sch.begin_block(bb)
        sch.draw_step(bb, wl.steps_per_block)
    q, k, v = sch.begin_block(b)
    ctx = make_ctx(wl)
    ctx.build(b, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
    return ctx, sch


def _check(ctx, rows, logits_t, want_lse=True):
    n = rows.shape[0]
    conf = torch.full((n,), float("nan"), device="cuda")
    tok = torch.full((n,), -7, device="cuda", dtype=torch.int32)
    lse = torch.full((n,), float("nan"), device="cuda") if want_lse else None
    ctx.sample_block(logits_t, conf, tok, lse)
    torch.cuda.synchronize()
    st, msg = ctx.poll_status()
    assert st == 0, msg
    ref_tok, ref_conf, ref_lse = sampler.block_confidence(logits_t.float().cpu().numpy().astype(np.float64), rows)
    assert np.array_equal(tok.cpu().numpy().astype(np.int64), ref_tok)
    c = conf.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(c - ref_conf) <= 2e-5 * ref_conf + 1e-30), np.abs(c / ref_conf - 1).max()
    if want_lse:
        assert np.abs(lse.cpu().numpy().astype(np.float64) - ref_lse).max() <= 2e-5 * np.maximum(1.0, np.abs(ref_lse)).max()
    return c


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("vocab", [1, 7, 1000, 4099, 32768, 126464])
def test_block_rows_against_oracle(dtype, vocab):
    wl = small_workload(name="samp", prompt_lens=(70, 33), gen_len=64, block_len=32, steps=1, hq=2, hkv=2)
    ctx, sch = _built_ctx(wl, 1)
    g = torch.Generator(device="cuda").manual_seed(vocab)
    T = wl.total_tokens
    logits = (torch.randn(T, vocab, generator=g, device="cuda") * 4).to(dtype)
    rows = sch.block_rows(1)
    # a peaked row, a row with exact ties at the maximum, a row with masked (-inf) entries
    if vocab >= 7:
        logits[rows[0], vocab // 2] = 30.0
        logits[rows[1], [5, 3, vocab - 1]] = 25.0
        logits[rows[2], ::2] = float("-inf")
    # rows outside the block must not be read: poison them
    outside = torch.ones(T, dtype=torch.bool, device="cuda")
    outside[torch.from_numpy(rows).cuda()] = False
    logits[outside] = float("nan")
    _check(ctx, rows, logits)
    _check(ctx, rows, logits, want_lse=False)      # lse is optional; repeated calls reuse the counters
    ctx.destroy()


def test_full_size_block_and_vocabulary():
    """The headline configuration's block (32 rows) and the large-batch extension's (8192 rows) at a
    vocabulary of 126464 entries (bf16 logits of every token would not fit for the latter: its logits
    array holds the block's rows of a smaller context with the same number of block rows)."""
    wl = WORKLOADS[2]
    ctx, sch = _built_ctx(wl, 3)
    g = torch.Generator(device="cuda").manual_seed(9)
    logits = (torch.randn(wl.total_tokens, 126464, generator=g, device="cuda") * 3).to(torch.bfloat16)
    _check(ctx, sch.block_rows(3), logits)
    ctx.destroy()
    wl = small_workload(name="samp-batch", prompt_lens=(3,) * 256, gen_len=64, block_len=32, steps=1, hq=2, hkv=2)
    ctx, sch = _built_ctx(wl, 0)
    rows = sch.block_rows(0)
    assert rows.shape[0] == 8192
    logits = (torch.randn(wl.total_tokens, 16384, generator=g, device="cuda") * 3).to(torch.bfloat16)
    _check(ctx, rows, logits)
    ctx.destroy()


def test_sample_needs_a_build_and_valid_arguments():
    wl = small_workload(name="samp-err", prompt_lens=(40,), gen_len=64, block_len=32, steps=1, hq=2, hkv=2)
    ctx = make_ctx(wl)
    logits = torch.zeros(wl.total_tokens, 64, device="cuda", dtype=torch.bfloat16)
    conf = torch.empty(32, device="cuda"); tok = torch.empty(32, device="cuda", dtype=torch.int32)
    with pytest.raises(binding.LacacheError) as e:
        ctx.sample_block(logits, conf, tok)
    assert e.value.status == binding.ERR_STATE
    sch = SyntheticSchedule(wl, seed=1)
    q, k, v = sch.begin_block(0)
    ctx.build(0, to_dev(q, wl), to_dev(k, wl), to_dev(v, wl))
    with pytest.raises(binding.LacacheError) as e:
        ctx.sample_block(logits, None, tok)
    assert e.value.status == binding.ERR_INVALID_ARG
    ctx.sample_block(logits, conf, tok)
    torch.cuda.synchronize()
    assert torch.equal(tok, torch.zeros_like(tok))          # all logits equal: the lowest id
    assert torch.allclose(conf, torch.full_like(conf, 1.0 / 64))
    ctx.destroy()
