"""Page bookkeeping on the GPU (reserve / release) against the oracle, bit for bit, through a
trajectory lifecycle: add, grow over several steps, abort some, add again, then use the pages."""
import numpy as np
import pytest
import torch

import oracle
from harness import assert_attn_close, dev_i32
from paper_2512_22560_b200 import rollart
from paper_2512_22560_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_lifecycle_matches_oracle_and_pages_serve_attention(cuda_device):
    rng = np.random.default_rng(5)
    P, T, max_pages, num_pages, Hkv, Hq = 16, 40, 24, 512, 2, 8
    free = rng.permutation(num_pages).astype(np.int32)
    cnt = num_pages
    table = np.full((T, max_pages), -1, np.int32)
    lens = np.zeros(T, np.int32)
    d_free, d_cnt = dev_i32(free, cuda_device), dev_i32([cnt], cuda_device)
    d_table, d_lens = dev_i32(table, cuda_device), dev_i32(lens, cuda_device)
    d_lens_next = torch.empty_like(d_lens)
    k_pool = torch.zeros(num_pages, Hkv, P, 128, dtype=torch.bfloat16, device=cuda_device)
    v_pool = torch.zeros_like(k_pool)
    kp, vp = W.bf16_to_u16(k_pool), W.bf16_to_u16(v_pool)
    ctx = rollart.Context(0, rollart.workspace_size(T, Hq, Hkv, max_pages * P))
    gen = torch.Generator().manual_seed(3)

    for step in range(12):
        if step % 5 == 4:
            ids = rng.permutation(T)[:7].astype(np.int32)                   # ABORT / evict
            cnt = oracle.pages_release(free, cnt, P, table, lens, ids)
            ctx.pages_release(d_free, d_cnt, P, d_table, d_lens, dev_i32(ids, cuda_device))
        else:
            ids = rng.permutation(T)[: rng.integers(1, T + 1)].astype(np.int32)   # ADD new ones / grow running ones
            new = rng.integers(0, 60, size=len(ids)).astype(np.int32)
            new = np.minimum(new, max_pages * P - lens[ids])
            cnt = oracle.pages_reserve(free, cnt, P, table, lens, new, traj_ids=ids)
            ctx.pages_reserve(d_free, d_cnt, P, d_table, d_lens, dev_i32(new, cuda_device), traj_ids=dev_i32(ids, cuda_device))
            # the tokens themselves: append on both sides onto the pages just reserved
            indptr = np.concatenate([[0], np.cumsum(new)]).astype(np.int32)
            k_new = torch.randn(int(indptr[-1]), Hkv, 128, generator=gen).to(torch.bfloat16)
            v_new = torch.randn(int(indptr[-1]), Hkv, 128, generator=gen).to(torch.bfloat16)
            lens = oracle.kv_append(kp, vp, table, lens, indptr, W.bf16_to_u16(k_new), W.bf16_to_u16(v_new), traj_ids=ids)
            d_lens_next.copy_(d_lens)
            ctx.kv_append(k_pool, v_pool, d_table, d_lens, dev_i32(indptr, cuda_device), k_new.to(cuda_device),
                          v_new.to(cuda_device), traj_ids=dev_i32(ids, cuda_device), seq_lens_out=d_lens_next)
            d_lens, d_lens_next = d_lens_next, d_lens
        ctx.check()
        assert int(d_cnt.item()) == cnt
        assert np.array_equal(d_free.cpu().numpy()[:cnt], free[:cnt])
        assert np.array_equal(d_table.cpu().numpy(), table)
        assert np.array_equal(d_lens.cpu().numpy(), lens)
    assert np.array_equal(W.bf16_to_u16(k_pool), kp) and np.array_equal(W.bf16_to_u16(v_pool), vp)

    # the tables built on the device serve a decode call
    q = torch.randn(T, Hq, 128, generator=gen).to(torch.bfloat16)
    out = torch.empty(T, Hq, 128, dtype=torch.bfloat16, device=cuda_device)
    ctx.decode_attn(k_pool, v_pool, d_table, d_lens, q.to(cuda_device), 0.09, max_pages * P, out)
    ctx.check()
    ref, _ = oracle.decode_attn(kp, vp, np.where(table < 0, 0, table).astype(np.int32), lens, W.bf16_to_u16(q), 0.09)
    assert_attn_close(out, ref, "decode over reserved pages")


def test_refusals_change_nothing(cuda_device):
    P = 16
    ctx = rollart.Context(0, 0)
    d_free, d_cnt = dev_i32(np.arange(4), cuda_device), dev_i32([4], cuda_device)
    d_table, d_lens = dev_i32(np.full((2, 3), -1), cuda_device), dev_i32([0, 0], cuda_device)
    ctx.pages_reserve(d_free, d_cnt, P, d_table, d_lens, dev_i32([40, 33], cuda_device))      # 5 pages wanted, 4 free
    assert ctx.status() == rollart.ERR_BOUNDS and "pages" in ctx.last_error()
    ctx.pages_reserve(d_free, d_cnt, P, d_table, d_lens, dev_i32([49, 0], cuda_device))       # row of 3 entries, 4 wanted
    assert ctx.status() == rollart.ERR_BOUNDS
    assert int(d_cnt.item()) == 4 and bool((d_table == -1).all())
    ctx.pages_reserve(d_free, d_cnt, P, d_table, d_lens, dev_i32([17, 16], cuda_device))      # 2 + 1 pages: fine
    ctx.check()
    assert int(d_cnt.item()) == 1 and d_table.cpu().tolist() == [[3, 2, -1], [1, -1, -1]]


def test_many_items_use_several_scan_chunks(cuda_device):
    rng = np.random.default_rng(6)
    P, T, max_pages = 16, 3000, 4
    num_pages = T * max_pages
    free = rng.permutation(num_pages).astype(np.int32)
    table = np.full((T, max_pages), -1, np.int32)
    lens = np.zeros(T, np.int32)
    new = rng.integers(0, max_pages * P + 1, size=T).astype(np.int32)
    ctx = rollart.Context(0, 0)
    d_free, d_cnt = dev_i32(free, cuda_device), dev_i32([num_pages], cuda_device)
    d_table, d_lens = dev_i32(table, cuda_device), dev_i32(lens, cuda_device)
    cnt = oracle.pages_reserve(free, num_pages, P, table, lens, new)
    ctx.pages_reserve(d_free, d_cnt, P, d_table, d_lens, dev_i32(new, cuda_device))
    ctx.check()
    assert int(d_cnt.item()) == cnt and np.array_equal(d_table.cpu().numpy(), table)
    lens = new.copy()
    d_lens.copy_(dev_i32(new, cuda_device))
    ids = rng.permutation(T)[:2500].astype(np.int32)
    cnt = oracle.pages_release(free, cnt, P, table, lens, ids)
    ctx.pages_release(d_free, d_cnt, P, d_table, d_lens, dev_i32(ids, cuda_device))
    ctx.check()
    assert int(d_cnt.item()) == cnt and np.array_equal(d_free.cpu().numpy()[:cnt], free[:cnt])
    assert np.array_equal(d_table.cpu().numpy(), table) and np.array_equal(d_lens.cpu().numpy(), lens)


def test_stale_eviction_matches_oracle_over_several_versions(cuda_device):
    # Sec. 6.2: the model version advances, trajectories started before the window are evicted, new ones start under
    # the current version; every array is compared with the oracle after each step.  2500 trajectories: the kernel
    # walks them in several chunks.
    rng = np.random.default_rng(8)
    P, T, max_pages, num_pages = 16, 2500, 6, 9000
    free = rng.permutation(num_pages).astype(np.int32)
    cnt = num_pages
    table = np.full((T, max_pages), -1, np.int32)
    lens = np.zeros(T, np.int32)
    sv = np.zeros(T, np.int32)
    d_free, d_cnt = dev_i32(free, cuda_device), dev_i32([cnt], cuda_device)
    d_table, d_lens = dev_i32(table, cuda_device), dev_i32(lens, cuda_device)
    d_ids, d_n = torch.full((T,), -9, dtype=torch.int32, device=cuda_device), dev_i32([-9], cuda_device)
    ctx = rollart.Context(0, 0)
    alpha = 1
    for version in range(1, 7):
        # trajectories without pages start under this version and take some
        starters = np.flatnonzero(lens == 0)
        starters = starters[rng.random(len(starters)) < 0.6].astype(np.int32)
        new = rng.integers(1, max_pages * P + 1, size=len(starters)).astype(np.int32)
        cnt = oracle.pages_reserve(free, cnt, P, table, lens, new, traj_ids=starters)
        ctx.pages_reserve(d_free, d_cnt, P, d_table, d_lens, dev_i32(new, cuda_device), traj_ids=dev_i32(starters, cuda_device))
        lens[starters] += new
        sv[starters] = version
        d_lens.copy_(dev_i32(lens, cuda_device))
        cnt, ids = oracle.pages_evict_stale(free, cnt, P, table, lens, sv, version, alpha)
        ctx.pages_evict_stale(d_free, d_cnt, P, d_table, d_lens, dev_i32(sv, cuda_device), version, alpha, d_ids, d_n)
        ctx.check()
        assert int(d_n.item()) == len(ids) and np.array_equal(d_ids.cpu().numpy()[: len(ids)], ids)
        assert int(d_cnt.item()) == cnt and np.array_equal(d_free.cpu().numpy()[:cnt], free[:cnt])
        assert np.array_equal(d_table.cpu().numpy(), table) and np.array_equal(d_lens.cpu().numpy(), lens)
        if version >= 3:
            assert len(ids) > 0
    # a stack too small for the returned pages: refused, nothing changes, the count reads 0
    small = d_free[: cnt + 1].clone()
    t0, l0 = d_table.clone(), d_lens.clone()
    ctx.pages_evict_stale(small, d_cnt, P, d_table, d_lens, dev_i32(sv, cuda_device), 50, 0, d_ids, d_n)
    assert ctx.status() == rollart.ERR_BOUNDS
    assert int(d_n.item()) == 0 and int(d_cnt.item()) == cnt and torch.equal(d_table, t0) and torch.equal(d_lens, l0)
    ctx.close()
