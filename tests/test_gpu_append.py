"""KV append on the GPU vs the oracle: every byte of both pools, and the new lengths."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from harness import DeviceBatch, dev_i32, make_ctx, oracle_append
from paper_2512_22560_b200 import rollart
from paper_2512_22560_b200 import workloads as W

pytestmark = pytest.mark.gpu


def check_append(batch, device):
    ctx = make_ctx(batch.spec, batch.spec.num_traj, 0)
    db = DeviceBatch(batch, device)
    db.append(ctx)
    ctx.check()
    kp, vp, after = oracle_append(batch)
    assert np.array_equal(W.bf16_to_u16(db.k_pool), kp)
    assert np.array_equal(W.bf16_to_u16(db.v_pool), vp)
    assert np.array_equal(db.lens_after.cpu().numpy(), after)
    ctx.close()


@pytest.mark.parametrize("i,T,div,cdiv", [(0, 4, 1, 1), (1, 9, 8, 1), (2, 7, 32, 1), (3, 3, 64, 1), (4, 12, 16, 4)])
def test_append_matches_oracle_bit_exact(cuda_device, i, T, div, cdiv):
    batch = W.make_batch(W.shrink(W.CONFIGS[i], T, div, cdiv), seed=100 + i)
    W.poison_dead_slots(batch, batch.seq_lens_before)
    check_append(batch, cuda_device)


@pytest.mark.parametrize("P", [16, 32, 64])
def test_append_page_boundaries_and_empty_items(cuda_device, P):
    spec = dataclasses.replace(W.CONFIGS[0], page_size=P, num_traj=7, num_kv_heads=3, num_q_heads=3, name=f"edge{P}")
    batch = W.make_layout(spec, seed=5)
    # lengths and chunk sizes that start/end on, before and after page boundaries; one empty item
    batch.seq_lens_before = np.array([0, 1, P - 1, P, P + 1, 3 * P - 2, 5], np.int32)
    batch.n_new = np.array([1, P, 2, 1, 2 * P + 3, 5, 0], np.int32)
    batch.new_indptr = np.concatenate([[0], np.cumsum(batch.n_new)]).astype(np.int32)
    pages = (batch.seq_lens_before + batch.n_new + P - 1) // P
    batch.page_table, batch.num_pages = W.build_page_table(pages.astype(np.int64), 0.5, np.random.default_rng(3))
    W.fill_tensors(batch)
    check_append(batch, cuda_device)


def test_append_with_traj_ids_subset(cuda_device):
    batch = W.make_batch(W.shrink(W.CONFIGS[4], 10, 32, 8), seed=9)
    ids = np.array([7, 2, 9, 0], np.int32)
    n = batch.n_new[ids]
    indptr = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
    rows = np.concatenate([np.arange(batch.new_indptr[t], batch.new_indptr[t + 1]) for t in ids])
    k_new, v_new = batch.k_new[rows].contiguous(), batch.v_new[rows].contiguous()
    kp, vp = W.bf16_to_u16(batch.k_pool), W.bf16_to_u16(batch.v_pool)
    after = oracle.kv_append(kp, vp, batch.page_table, batch.seq_lens_before, indptr, W.bf16_to_u16(k_new),
                             W.bf16_to_u16(v_new), traj_ids=ids)
    ctx = rollart.Context(0, 0)
    dk, dv = batch.k_pool.to(cuda_device), batch.v_pool.to(cuda_device)
    lens = dev_i32(batch.seq_lens_before, cuda_device)
    out = lens.clone()
    ctx.kv_append(dk, dv, dev_i32(batch.page_table, cuda_device), lens, dev_i32(indptr, cuda_device),
                  k_new.to(cuda_device), v_new.to(cuda_device), traj_ids=dev_i32(ids, cuda_device), seq_lens_out=out)
    ctx.check()
    assert np.array_equal(W.bf16_to_u16(dk), kp) and np.array_equal(W.bf16_to_u16(dv), vp)
    assert np.array_equal(out.cpu().numpy(), after)


def test_append_device_side_errors_are_reported_not_fatal(cuda_device):
    batch = W.make_batch(W.shrink(W.CONFIGS[0], 4, 4), seed=11)
    db = DeviceBatch(batch, cuda_device)
    ctx = rollart.Context(0, 0)
    k_before = db.k_pool.clone()
    bad_table = db.page_table.clone()
    t = 2
    lp = int(batch.seq_lens_before[t]) // batch.spec.page_size
    bad_table[t, lp] = batch.num_pages + 5            # page id outside the pool
    ctx.kv_append(db.k_pool, db.v_pool, bad_table, db.lens_before, db.new_indptr, db.k_new, db.v_new)
    assert ctx.status() == rollart.ERR_BOUNDS
    assert "kv_append" in ctx.last_error()
    # rows of the other trajectories were written, the offending one skipped; the context still works
    assert ctx.status() == rollart.OK
    db.k_pool.copy_(k_before)
    db.append(ctx)
    ctx.check()
    kp, _, _ = oracle_append(batch)
    assert np.array_equal(W.bf16_to_u16(db.k_pool), kp)


def test_malformed_indptr_is_a_device_side_error_and_touches_nothing(cuda_device):
    # new_indptr[0] = 3: the first rows belong to no item.  Before the check such a row computed a negative position
    # and stored in front of its page; now it is reported and skipped.
    batch = W.make_batch(W.shrink(W.CONFIGS[0], 4, 4), seed=13)
    db = DeviceBatch(batch, cuda_device)
    ctx = rollart.Context(0, 0)
    k_before, v_before = db.k_pool.clone(), db.v_pool.clone()
    indptr = db.new_indptr.clone()
    indptr[:] = int(db.new_indptr[-1])        # every item empty, and rows 0 .. total-1 lie before indptr[0]
    ctx.kv_append(db.k_pool, db.v_pool, db.page_table, db.lens_before, indptr, db.k_new, db.v_new)
    assert ctx.status() == rollart.ERR_BOUNDS
    assert torch.equal(db.k_pool.view(torch.int16), k_before.view(torch.int16))
    assert torch.equal(db.v_pool.view(torch.int16), v_before.view(torch.int16))
    # the gather has the same check: rows before out_indptr[0] are left unwritten
    lens = batch.seq_lens_before
    good = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    total = int(good[-1])
    k_out = torch.full((total, batch.spec.num_kv_heads, 128), 7.0, dtype=torch.bfloat16, device=cuda_device)
    v_out = k_out.clone()
    bad = good.copy()
    bad[0] = 3
    ctx.kv_gather(db.k_pool, db.v_pool, db.page_table, db.lens_before, dev_i32(bad, cuda_device), k_out, v_out)
    assert ctx.status() == rollart.ERR_BOUNDS
    assert bool(torch.all(k_out[:3] == 7.0)) and bool(torch.all(v_out[:3] == 7.0))
    ctx.close()


def test_append_host_side_validation(cuda_device):
    batch = W.make_batch(W.shrink(W.CONFIGS[0], 2, 4), seed=12)
    db = DeviceBatch(batch, cuda_device)
    ctx = rollart.Context(0, 0)
    with pytest.raises(rollart.RollartError) as e:
        ctx.kv_append(db.k_pool, db.v_pool, db.page_table, db.lens_before, db.new_indptr, db.k_new, db.v_new,
                      seq_lens_out=db.lens_before)
    assert e.value.status == rollart.ERR_INVALID_ARG
    bad = torch.zeros(4, 2, 24, 128, dtype=torch.bfloat16, device=cuda_device)
    with pytest.raises(rollart.RollartError) as e:
        ctx.kv_append(bad, bad, db.page_table, db.lens_before, db.new_indptr, db.k_new, db.v_new)
    assert e.value.status == rollart.ERR_UNSUPPORTED


@pytest.mark.parametrize("i,T,div", [(0, 4, 1), (3, 3, 32), (4, 9, 16)])
def test_gather_matches_oracle_and_round_trips_through_append(cuda_device, i, T, div):
    """Hand-off of whole trajectories: gather from one pool, append into another (different page table)."""
    batch = W.make_batch(W.shrink(W.CONFIGS[i], T, div, 8), seed=300 + i)
    spec = batch.spec
    db = DeviceBatch(batch, cuda_device)
    ctx = rollart.Context(0, 0)
    ids = np.array(sorted(range(T), key=lambda t: -t)[: max(2, T - 1)], np.int32)      # a subset in reverse order
    lens = batch.seq_lens_before[ids]
    indptr = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    total = int(indptr[-1])
    k_out = torch.full((total, spec.num_kv_heads, 128), float("nan"), dtype=torch.bfloat16, device=cuda_device)
    v_out = torch.full_like(k_out, float("nan"))
    ctx.kv_gather(db.k_pool, db.v_pool, db.page_table, db.lens_before, dev_i32(indptr, cuda_device), k_out, v_out,
                  traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    ko, vo = oracle.kv_gather(W.bf16_to_u16(batch.k_pool), W.bf16_to_u16(batch.v_pool), batch.page_table,
                              batch.seq_lens_before, indptr, traj_ids=ids)
    assert np.array_equal(W.bf16_to_u16(k_out), ko) and np.array_equal(W.bf16_to_u16(v_out), vo)
    # receiving side: empty trajectories with their own pages
    pages = (lens.astype(np.int64) + spec.page_size - 1) // spec.page_size
    table2, num_pages2 = W.build_page_table(pages, 0.25, np.random.default_rng(9))
    k2 = torch.zeros(num_pages2, spec.num_kv_heads, spec.page_size, 128, dtype=torch.bfloat16, device=cuda_device)
    v2 = torch.zeros_like(k2)
    zero = dev_i32(np.zeros(len(ids)), cuda_device)
    after = torch.empty_like(zero)
    ctx.kv_append(k2, v2, dev_i32(table2, cuda_device), zero, dev_i32(indptr, cuda_device), k_out, v_out, seq_lens_out=after)
    k_back = torch.empty_like(k_out)
    v_back = torch.empty_like(v_out)
    ctx.kv_gather(k2, v2, dev_i32(table2, cuda_device), after, dev_i32(indptr, cuda_device), k_back, v_back)
    ctx.check()
    assert np.array_equal(after.cpu().numpy(), lens)
    assert torch.equal(k_back.view(torch.int16), k_out.view(torch.int16)) and torch.equal(v_back.view(torch.int16), v_out.view(torch.int16))
    # asking for more rows than a trajectory holds is reported, not read
    bad = indptr.copy()
    bad[-1] += 1
    big = torch.zeros(total + 1, spec.num_kv_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    ctx.kv_gather(db.k_pool, db.v_pool, db.page_table, db.lens_before, dev_i32(bad, cuda_device), big, big.clone(),
                  traj_ids=dev_i32(ids, cuda_device))
    assert ctx.status() == rollart.ERR_BOUNDS and "kv_gather" in ctx.last_error()
