"""The seeded input recipes: shapes, ranges, page-table structure, reproducibility."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2512_22560_b200 import workloads as W


@pytest.mark.parametrize("i", range(5))
def test_layout_properties(i):
    spec = W.CONFIGS[i]
    b = W.make_layout(spec)
    T, P = spec.num_traj, spec.page_size
    assert b.seq_lens_before.shape == (T,) and b.seq_lens_before.dtype == np.int32
    assert b.seq_lens_before.min() >= 1
    need = (b.seq_lens_before.astype(np.int64) + b.n_new + P - 1) // P
    owned = b.page_table >= 0
    assert np.array_equal(owned.sum(1), need)
    ids = b.page_table[owned]
    assert len(np.unique(ids)) == len(ids) and ids.max() < b.num_pages
    assert b.num_pages >= int(need.sum() * 1.12)
    # consecutive logical pages of a trajectory are not physically consecutive as a rule
    adj = (np.diff(b.page_table, axis=1) == 1) & owned[:, 1:]
    assert adj.mean() < 0.01
    b2 = W.make_layout(spec)
    assert np.array_equal(b.page_table, b2.page_table) and np.array_equal(b.seq_lens_before, b2.seq_lens_before)
    b3 = W.make_layout(spec, seed=7)
    assert not np.array_equal(b.seq_lens_before, b3.seq_lens_before)


def test_recipe_ranges():
    l0 = W.make_layout(W.CONFIGS[0]).seq_lens_before
    assert 64 <= l0.min() and l0.max() <= 512
    b1 = W.make_layout(W.CONFIGS[1])
    assert 2 * 300 <= b1.seq_lens_before.min() and b1.seq_lens_before.max() <= 15000
    assert all(len(t) % 2 == 0 and 4 <= len(t) <= 20 for t in b1.turns)
    l2 = W.make_layout(W.CONFIGS[2]).seq_lens_before
    assert l2.max() <= 32768 and 6000 < np.median(l2) < 11000
    l3 = W.make_layout(W.CONFIGS[3]).seq_lens_before
    assert 32768 <= l3.min() and l3.max() <= 131072
    b4 = W.make_layout(W.CONFIGS[4])
    assert b4.is_chunk.sum() == 64 and np.all(b4.n_new[~b4.is_chunk] == 1)
    assert 64 <= b4.n_new[b4.is_chunk].min() and b4.n_new[b4.is_chunk].max() <= 2048
    assert 1024 <= b4.seq_lens_before.min() and b4.seq_lens_before.max() <= 24576


def test_tensors_reproducible_and_extract():
    spec = W.shrink(W.CONFIGS[4], 6, 64, 16)
    a = W.make_batch(spec)
    b = W.make_batch(spec)
    assert torch.equal(a.k_pool.view(torch.int16), b.k_pool.view(torch.int16))
    assert a.k_pool.shape == (a.num_pages, 8, 16, 128) and a.q_new.shape[0] == a.new_indptr[-1]
    sub = W.extract_trajs(a, [4, 1])
    for i, t in enumerate([4, 1]):
        n = (a.seq_lens_before[t] + a.n_new[t] + 15) // 16
        for lp in range(n):
            assert torch.equal(sub.k_pool[sub.page_table[i, lp]].view(torch.int16),
                               a.k_pool[a.page_table[t, lp]].view(torch.int16))
    assert sub.q_new.shape[0] == a.n_new[[4, 1]].sum()


def test_poison_and_needles_change_only_what_they_say():
    spec = W.shrink(W.CONFIGS[0], 3, 4)
    b = W.make_batch(spec)
    k0 = b.k_pool.clone()
    W.poison_dead_slots(b, b.seq_lens_before)
    live = W.slot_owner_mask(b, b.seq_lens_before)
    same = (b.k_pool.view(torch.int16) == k0.view(torch.int16)).all(dim=3).all(dim=1)   # [pages][P]
    assert same[live].all() and not same[~live].any()
    assert live.sum().item() == int(b.seq_lens_before.sum())
    # oracle run over a poisoned pool stays finite, and a needle makes an O(1) output
    W.plant_needles(b, {0: [0, int(b.seq_lens_before[0]) - 1]})
    kp, vp = W.bf16_to_u16(b.k_pool), W.bf16_to_u16(b.v_pool)
    after = oracle.kv_append(kp, vp, b.page_table, b.seq_lens_before, b.new_indptr,
                             W.bf16_to_u16(b.k_new), W.bf16_to_u16(b.v_new))
    out, _ = oracle.decode_attn(kp, vp, b.page_table, after, W.bf16_to_u16(b.q_new), spec.sm_scale)
    assert np.all(np.isfinite(out))
    assert np.abs(out[0]).max() > 0.5


def test_share_group_prefix_aliases_whole_pages_only():
    spec = dataclasses.replace(W.shrink(W.CONFIGS[1], 19, 16), name="groups")
    b = W.make_layout(spec, seed=3)
    before = b.page_table.copy()
    indptr, shared = W.share_group_prefix(b, 8, 0.7)
    assert indptr.tolist() == [0, 8, 16, 19] and shared.dtype == np.int32
    P = spec.page_size
    for gi in range(3):
        a, e = int(indptr[gi]), int(indptr[gi + 1])
        s = int(shared[gi])
        assert s % P == 0 and s <= int(b.seq_lens_before[a:e].min())
        assert s == int(int(b.seq_lens_before[a:e].min()) * 0.7) // P * P
        assert (b.page_table[a:e, :s // P] == before[a, :s // P]).all()          # the first member's pages
        assert (b.page_table[a:e, s // P:] == before[a:e, s // P:]).all()        # the rest untouched
    # distinct pages are still distinct outside the shared region: no page is listed by two different groups
    owned = [set(b.page_table[t, :(int(b.seq_lens_before[t]) + 1 + P - 1) // P].tolist()) for t in range(19)]
    for t in range(19):
        for u in range(t + 1, 19):
            if np.searchsorted(indptr, t, side="right") != np.searchsorted(indptr, u, side="right"):
                assert not (owned[t] & owned[u])
