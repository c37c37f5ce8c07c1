"""Host-side checks of the synthetic workload generators (data only)."""
import numpy as np
import torch

from paper_2607_16339_b200.workloads import (WORKLOADS, SyntheticSchedule, parity_points,
                                             round_to_bf16, small_workload)


def test_config_table_matches_named_shapes():
    w = WORKLOADS
    assert [w[i].total_tokens for i in (1, 2, 3, 5)] == [112, 768, 1536, 5120]
    assert w[4].total_tokens == 6411 and w[4].batch == 8
    assert list(w[4].prompt_lens) == list(
        np.random.Generator(np.random.Philox(key=4)).integers(256, 1025, 8))
    assert [w[i].n_steps for i in (1, 2, 3, 4, 5)] == [16, 256, 256, 256, 1024]
    assert (w[5].n_q_heads, w[5].n_kv_heads, w[5].block_len) == (28, 4, 64)
    assert w[4].cu_seqlens[0] == 0 and w[4].cu_seqlens[-1] == 6411


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(100000) * np.exp(rng.uniform(-20, 20, 100000))).astype(np.float32)
    x[:4] = [0.0, -0.0, 1.00390625, 1.01171875]          # ties
    ref = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    assert np.array_equal(round_to_bf16(x).view(np.uint32), ref.view(np.uint32))


def test_schedule_structure():
    wl = small_workload(prompt_lens=(20, 9), gen_len=16, block_len=4, steps=3, hq=4, hkv=2, d=8,
                        outlier_frac=0.2)
    sch = SyntheticSchedule(wl, seed=1)
    cu = wl.cu_seqlens
    # masked suffix rows are identical per head
    for b, P in enumerate(wl.prompt_lens):
        assert np.all(sch.q[cu[b] + P:cu[b + 1]] == sch.mask_q)
        assert np.all(sch.k[cu[b] + P:cu[b + 1]] == sch.mask_k)
    assert len(sch.outlier_rows) == 4 + 1
    # values are exactly representable in the storage dtype
    assert np.array_equal(round_to_bf16(sch.k), sch.k)
    q0 = sch.q.copy()
    sch.begin_block(0)
    qb, kb, vb = sch.draw_step(0, 1)
    rows = sch.block_rows(0)
    assert rows.tolist() == [20, 21, 22, 23, 36 + 9, 36 + 10, 36 + 11, 36 + 12]
    assert np.array_equal(sch.q[rows], qb) and qb.shape == (8, 4, 8)
    fixed = np.flatnonzero(sch.is_block(0) == 0)
    assert np.array_equal(sch.q[fixed], q0[fixed])
    # seeded: same seed, same bits; other seed differs
    s2 = SyntheticSchedule(wl, seed=1); s2.begin_block(0)
    assert np.array_equal(s2.draw_step(0, 1)[0], qb)
    assert not np.array_equal(SyntheticSchedule(wl, seed=2).q, q0)
    # moving to block 1 keeps block 0's last draw and masks block 1
    sch.begin_block(1)
    assert np.array_equal(sch.q[rows], qb)
    assert np.all(sch.q[sch.block_rows(1)] == sch.mask_q)


def test_parity_points():
    assert len(parity_points(WORKLOADS[1])) == 16
    assert parity_points(WORKLOADS[2]) == [(0, 1), (0, 32), (4, 1), (4, 32), (7, 1), (7, 32)]
