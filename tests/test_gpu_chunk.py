"""Observation-chunk attention on the GPU vs the oracle, and its cross-call invariants."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from harness import DeviceBatch, assert_attn_close, assert_lse_close, dev_i32, make_ctx, oracle_append
from paper_2512_22560_b200 import rollart
from paper_2512_22560_b200 import workloads as W

pytestmark = pytest.mark.gpu


def run_chunk_case(batch, device, poison=True):
    spec = batch.spec
    if poison:
        W.poison_dead_slots(batch, batch.seq_lens_before)
    ids = batch.chunk_ids
    rows, q_indptr = batch.chunk_rows()
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, len(ids), msl)
    db = DeviceBatch(batch, device)
    db.append(ctx)
    q = db.q_new[torch.from_numpy(rows).to(device)].contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], spec.num_q_heads), float("nan"), device=device)
    ctx.obs_chunk_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32(q_indptr, device), q, spec.sm_scale,
                       msl, out, lse=lse, traj_ids=dev_i32(ids, device))
    ctx.check()
    kp, vp, after = oracle_append(batch)
    ref_o, ref_l = oracle.obs_chunk_attn(kp, vp, batch.page_table, after, q_indptr, W.bf16_to_u16(batch.q_new[rows]),
                                         spec.sm_scale, traj_ids=ids)
    assert_attn_close(out, ref_o, spec.name)
    assert_lse_close(lse, ref_l, spec.name)
    return db, ctx, out, (kp, vp, after)


def test_shrunk_mixed_batch_chunk_half(cuda_device):
    run_chunk_case(W.make_batch(W.shrink(W.CONFIGS[4], 8, 16, 8), seed=41), cuda_device)


def test_recompute_from_empty_cache(cuda_device):
    # KV recomputation: whole contexts as one causal chunk onto empty pages (prior = 0)
    batch = W.make_batch(W.shrink(W.RECOMPUTE, 5, 16), seed=46)
    assert batch.seq_lens_before.max() == 0 and batch.is_chunk.all()
    run_chunk_case(batch, cuda_device)


@pytest.mark.parametrize("P,hq,hkv", [(16, 8, 2), (32, 7, 1), (64, 16, 1), (16, 3, 3)])
def test_chunk_edges(cuda_device, P, hq, hkv):
    prior = [0, 0, 1, P - 1, P, 5, 130, 64]
    n_new = [1, P + 3, P, 2, 1, 130, 31, 128]
    spec = dataclasses.replace(W.CONFIGS[4], page_size=P, num_traj=len(prior), num_q_heads=hq, num_kv_heads=hkv,
                               name=f"chunk_edge_{P}_{hq}_{hkv}")
    batch = W.make_layout(spec, seed=3)
    batch.seq_lens_before = np.array(prior, np.int32)
    batch.n_new = np.array(n_new, np.int32)
    batch.is_chunk[:] = True
    batch.new_indptr = np.concatenate([[0], np.cumsum(batch.n_new)]).astype(np.int32)
    pages = (batch.seq_lens_before + batch.n_new + P - 1) // P
    batch.page_table, batch.num_pages = W.build_page_table(pages.astype(np.int64), 0.3, np.random.default_rng(2))
    W.fill_tensors(batch)
    run_chunk_case(batch, cuda_device)


@pytest.mark.parametrize("shape", ["rising", "falling", "spike"])
def test_chunk_scores_that_jump_between_key_tiles(cuda_device, shape):
    # Keys whose magnitude changes by steps of 64 positions: scores of later key tiles tower over (or vanish
    # under) those of the first tile, so the running reference max has to move, the accumulator has to be
    # rescaled, and the result is close to one-hot (O(1) outputs: a wrong key would show).
    P = 16
    prior = [700, 333, 64, 129]
    n_new = [100, 40, 70, 3]
    spec = dataclasses.replace(W.CONFIGS[4], page_size=P, num_traj=len(prior), num_q_heads=8, num_kv_heads=2,
                               name=f"chunk_jump_{shape}")
    batch = W.make_layout(spec, seed=11)
    batch.seq_lens_before = np.array(prior, np.int32)
    batch.n_new = np.array(n_new, np.int32)
    batch.is_chunk[:] = True
    batch.new_indptr = np.concatenate([[0], np.cumsum(batch.n_new)]).astype(np.int32)
    pages = (batch.seq_lens_before + batch.n_new + P - 1) // P
    batch.page_table, batch.num_pages = W.build_page_table(pages.astype(np.int64), 0.3, np.random.default_rng(5))
    W.fill_tensors(batch)
    for t, L in enumerate(prior):
        steps = (L + 63) // 64
        for pos in range(L):
            s = pos // 64
            if shape == "rising":
                gain = 1.0 + 6.0 * s
            elif shape == "falling":
                gain = 1.0 + 6.0 * (steps - 1 - s)
            else:
                gain = 60.0 if s == steps // 2 else 1.0
            pg = int(batch.page_table[t, pos // P])
            batch.k_pool[pg, :, pos % P, :] = (batch.k_pool[pg, :, pos % P, :].float() * gain).to(torch.bfloat16)
    run_chunk_case(batch, cuda_device)


def test_chunk_equals_sequential_append_and_decode_on_gpu(cuda_device):
    spec = dataclasses.replace(W.shrink(W.CONFIGS[4], 3, 64, 32), name="seq")
    batch = W.make_batch(spec, seed=43)
    batch.is_chunk[:] = True
    db, ctx, out_chunk, _ = run_chunk_case(batch, cuda_device, poison=False)
    # replay token by token from the state before the append
    db2 = DeviceBatch(W.make_batch(spec, seed=43), cuda_device)
    msl = int(batch.seq_lens_after.max())
    lens = db2.lens_before.clone()
    nxt = torch.empty_like(lens)
    one = dev_i32([0, 1], cuda_device)
    for t in range(spec.num_traj):
        tid = dev_i32([t], cuda_device)
        for j in range(int(batch.n_new[t])):
            r = int(batch.new_indptr[t]) + j
            nxt.copy_(lens)
            ctx.kv_append(db2.k_pool, db2.v_pool, db2.page_table, lens, one, db2.k_new[r:r + 1], db2.v_new[r:r + 1],
                          traj_ids=tid, seq_lens_out=nxt)
            lens, nxt = nxt, lens
            o = torch.empty(1, spec.num_q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
            ctx.decode_attn(db2.k_pool, db2.v_pool, db2.page_table, lens, db2.q_new[r:r + 1], spec.sm_scale, msl, o,
                            traj_ids=tid)
            # same math through a different schedule: a few bf16 ulps at most
            assert torch.allclose(o[0].float(), out_chunk[r].float(), atol=2e-3, rtol=2e-2), (t, j)
    ctx.check()
    assert torch.equal(db2.k_pool.view(torch.int16), db.k_pool.view(torch.int16))


def test_chunk_longer_than_trajectory_is_a_device_error(cuda_device):
    batch = W.make_batch(W.shrink(W.CONFIGS[0], 2, 4), seed=44)
    db = DeviceBatch(batch, cuda_device)
    ctx = make_ctx(batch.spec, 2, 100)
    q = torch.zeros(40, batch.spec.num_q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    out = torch.zeros_like(q)
    lens = dev_i32([10, 50], cuda_device)
    ctx.obs_chunk_attn(db.k_pool, db.v_pool, db.page_table, lens, dev_i32([0, 20, 40], cuda_device), q, 0.1, 100, out)
    assert ctx.status() == rollart.ERR_BOUNDS and "obs_chunk_attn" in ctx.last_error()


def test_many_small_chunks_span_several_launches(cuda_device):
    # 1100 chunk items of 1..5 tokens: more items than one launch's tile table holds, ragged single-tile units
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=1100, len_lo=1, len_hi=40, chunk_fraction=1.0, chunk_lo=1, chunk_hi=5,
                               name="many_chunks")
    run_chunk_case(W.make_batch(spec, seed=72), cuda_device)


def test_empty_items_and_empty_calls(cuda_device):
    # an item with no chunk rows among live ones, and calls with nothing to do at all
    spec = dataclasses.replace(W.CONFIGS[4], num_traj=4, name="empties")
    batch = W.make_layout(W.shrink(spec, 4, 64, 16), seed=47)
    batch.is_chunk[:] = True
    batch.n_new = np.array([5, 0, 40, 1], np.int32)
    batch.new_indptr = np.concatenate([[0], np.cumsum(batch.n_new)]).astype(np.int32)
    P = batch.spec.page_size
    pages = (batch.seq_lens_before.astype(np.int64) + batch.n_new + P - 1) // P
    batch.page_table, batch.num_pages = W.build_page_table(pages, 0.3, np.random.default_rng(1))
    W.fill_tensors(batch)
    db, ctx, out, _ = run_chunk_case(batch, cuda_device)
    empty_q = torch.zeros(0, batch.spec.num_q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    n0 = ctx.launch_count
    ctx.obs_chunk_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32([0], cuda_device), empty_q, 0.1, 100,
                       empty_q.clone())
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, empty_q, 0.1, 100, empty_q.clone(),
                    traj_ids=dev_i32([], cuda_device))
    ctx.kv_append(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32([0], cuda_device),
                  torch.zeros(0, batch.spec.num_kv_heads, 128, dtype=torch.bfloat16, device=cuda_device),
                  torch.zeros(0, batch.spec.num_kv_heads, 128, dtype=torch.bfloat16, device=cuda_device))
    ctx.check()
    assert ctx.launch_count == n0          # nothing was enqueued


def test_append_and_chunk_attention_replayed_from_a_cuda_graph(cuda_device):
    """kv_append + obs_chunk_attn captured once into a CUDA graph (Sec. 7.1: rollout runs with CUDA graphs) and replayed:
    the same bits as the eager calls."""
    batch = W.make_batch(W.shrink(W.CONFIGS[4], 6, 32, 16), seed=91)
    db, ctx, out_eager, _ = run_chunk_case(batch, cuda_device)
    spec = batch.spec
    ids = batch.chunk_ids
    rows, q_indptr = batch.chunk_rows()
    msl = int(batch.seq_lens_after.max())
    db2 = DeviceBatch(batch, cuda_device)                          # the pools as they were before the append
    q = db2.q_new[torch.from_numpy(rows).to(cuda_device)].contiguous()
    out = torch.full_like(q, float("nan"))
    qi, tid = dev_i32(q_indptr, cuda_device), dev_i32(ids, cuda_device)
    lens_after = torch.empty_like(db2.lens_before)
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize(cuda_device)
    with torch.cuda.graph(graph, stream=torch.cuda.Stream(device=cuda_device)):
        ctx.kv_append(db2.k_pool, db2.v_pool, db2.page_table, db2.lens_before, db2.new_indptr, db2.k_new, db2.v_new,
                      seq_lens_out=lens_after)
        ctx.obs_chunk_attn(db2.k_pool, db2.v_pool, db2.page_table, lens_after, qi, q, spec.sm_scale, msl, out, traj_ids=tid)
    for _ in range(2):                                             # the append is idempotent: same rows to the same slots
        out.fill_(float("nan"))
        graph.replay()
    torch.cuda.synchronize(cuda_device)
    ctx.check()
    assert torch.equal(out.view(torch.int16), out_eager.view(torch.int16))
    assert torch.equal(db2.k_pool.view(torch.int16), db.k_pool.view(torch.int16))
    assert torch.equal(lens_after, db.lens_after)
    ctx.close()


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(cuda_device):
    # The bounded wait of the tensor-core kernels on a barrier nothing arrives at: it gives up after about a second, the
    # status word carries ERR_TIMEOUT, and afterwards the same context computes a chunk call correctly.
    batch = W.make_batch(W.shrink(W.CONFIGS[4], 4, 32, 16), seed=48)
    spec = batch.spec
    ids = batch.chunk_ids
    rows, q_indptr = batch.chunk_rows()
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, len(ids), msl)
    ctx.selftest_bounded_wait()
    assert ctx.status() == rollart.ERR_TIMEOUT
    assert "wait" in ctx.last_error()
    assert ctx.status() == rollart.OK
    db = DeviceBatch(batch, cuda_device)
    db.append(ctx)
    q = db.q_new[torch.from_numpy(rows).to(cuda_device)].contiguous()
    out = torch.full_like(q, float("nan"))
    ctx.obs_chunk_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32(q_indptr, cuda_device), q, spec.sm_scale,
                       msl, out, traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    kp, vp, after = oracle_append(batch)
    ref_o, _ = oracle.obs_chunk_attn(kp, vp, batch.page_table, after, q_indptr, W.bf16_to_u16(batch.q_new[rows]), spec.sm_scale,
                                     traj_ids=ids)
    assert_attn_close(out, ref_o, "chunk call after a reported timeout")
    ctx.close()


def _custom_chunk_batch(P, hq, hkv, prior, n_new, seed, name):
    spec = dataclasses.replace(W.CONFIGS[4], page_size=P, num_traj=len(prior), num_q_heads=hq, num_kv_heads=hkv, name=name)
    batch = W.make_layout(spec, seed=seed)
    batch.seq_lens_before = np.array(prior, np.int32)
    batch.n_new = np.array(n_new, np.int32)
    batch.is_chunk[:] = True
    batch.new_indptr = np.concatenate([[0], np.cumsum(batch.n_new)]).astype(np.int32)
    pages = (batch.seq_lens_before + batch.n_new + P - 1) // P
    batch.page_table, batch.num_pages = W.build_page_table(pages.astype(np.int64), 0.3, np.random.default_rng(seed + 1))
    W.fill_tensors(batch)
    return batch


@pytest.mark.parametrize("P,hq,hkv", [(16, 4, 4), (16, 8, 4), (32, 10, 2), (16, 12, 2), (64, 8, 1), (32, 24, 2), (16, 32, 2)])
def test_chunk_lengths_around_the_tiles_of_the_pair_kernel(cuda_device, P, hq, hkv):
    # Group sizes 1, 2, 5, 6, 8, 12, 16 (128 / g tokens per M-tile, with and without padding rows).  Contexts that end
    # just before, on and just after the 128-key tiles and their 64-key halves (the two key streams of a tile), chunks of
    # one M-tile or less (the second CTA of the pair has no row), exactly one and exactly two M-tiles, and one token more.
    g = hq // hkv
    tpt = 128 // g
    prior = [0, 0, 63, 64, 65, 127, 128, 129, 191, 192, 200, 255, 256 + 64, 0, 1]
    n_new = [1, tpt, 1, tpt - 1 if tpt > 1 else 1, tpt + 1, 2 * tpt, 2 * tpt + 1, 3, 1, 2 * tpt - 1 if tpt > 1 else 1, 5 * tpt + 2, 1,
             tpt, 128 + 3, 127]
    batch = _custom_chunk_batch(P, hq, hkv, prior, n_new, 21, f"pair_edges_{P}_{hq}_{hkv}")
    run_chunk_case(batch, cuda_device)


def test_chunk_rerun_is_bit_identical(cuda_device):
    # units are independent and every unit adds its tiles and merges its two key streams in a fixed order
    batch = W.make_batch(W.shrink(W.CONFIGS[4], 8, 16, 8), seed=49)
    db, ctx, out, _ = run_chunk_case(batch, cuda_device)
    spec = batch.spec
    ids = batch.chunk_ids
    rows, q_indptr = batch.chunk_rows()
    msl = int(batch.seq_lens_after.max())
    q = db.q_new[torch.from_numpy(rows).to(cuda_device)].contiguous()
    for _ in range(3):
        again = torch.full_like(q, float("nan"))
        lse = torch.full((q.shape[0], spec.num_q_heads), float("nan"), device=cuda_device)
        ctx.obs_chunk_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32(q_indptr, cuda_device), q, spec.sm_scale,
                           msl, again, lse=lse, traj_ids=dev_i32(ids, cuda_device))
        ctx.check()
        assert torch.equal(again.view(torch.int16), out.view(torch.int16))
    ctx.close()


def test_chunk_with_one_stream_towering_over_the_other(cuda_device):
    # The two halves of every 128-key tile are separate softmax streams merged at the end.  Here the keys of one half are
    # scaled up (scores far above the other half's, by tile parity and by half), so the streams' reference maxima sit
    # far apart and the final merge has to weigh one stream down to nothing, or both equally, row by row.
    P = 16
    prior = [640, 500, 128]
    n_new = [70, 33, 130]
    batch = _custom_chunk_batch(P, 8, 2, prior, n_new, 31, "pair_streams")
    for t, L in enumerate(prior):
        for pos in range(L):
            half, tile = (pos // 64) & 1, pos // 128
            gain = 40.0 if (half == (tile & 1) and t != 1) or (t == 1 and half == 1) else 1.0
            pg = int(batch.page_table[t, pos // P])
            batch.k_pool[pg, :, pos % P, :] = (batch.k_pool[pg, :, pos % P, :].float() * gain).to(torch.bfloat16)
    run_chunk_case(batch, cuda_device)


def _lone_key_batch(seed, name):
    P = 16
    prior = [700, 400, 420, 1000]
    n_new = [100, 40, 70, 129]
    batch = _custom_chunk_batch(P, 8, 2, prior, n_new, seed, name)
    return batch.spec, batch, prior, P


# positions inside a 128-key tile: both halves of the tile, first and second half of a thread's columns, odd and even
_LONE_OFFSETS = (4, 5, 10, 29, 36, 37, 47, 68, 69, 100, 101, 125, 0, 63, 64, 127)


def test_chunk_lone_key_towering_over_its_tile(cuda_device):
    # One key per key tile whose score lies hundreds of log2 units above everything the row has seen, every other
    # key of the tile far below, and the same for every row (so no neighbouring row raises the alarm for it):
    # whichever unit takes that column's exponential (the special-function unit or the FMA pipe, whose range ends at
    # 2^127) has to notice by itself.  The rows become one-hot on the last such key.
    spec, batch, prior, P = _lone_key_batch(17, "chunk_lone_key")
    batch.q_new[:, :, 0] = 4.0                                 # every query row has the same component along dim 0 ...
    for t, L in enumerate(prior):
        for tile in range(1, (L + 127) // 128):
            pos = tile * 128 + _LONE_OFFSETS[(tile + 3 * t) % len(_LONE_OFFSETS)]
            if pos >= L:
                continue
            x_log2 = (150.0, 200.0, 400.0, 700.0)[(t + tile) % 4] + 40.0 * tile      # rising: each one towers over the last
            key = torch.zeros(128)
            key[0] = x_log2 / (4.0 * spec.sm_scale * 1.4426950408889634)   # ... so this key scores x_log2 log2 units for all of them
            pg = int(batch.page_table[t, pos // P])
            batch.k_pool[pg, :, pos % P, :] = key.to(torch.bfloat16)
    run_chunk_case(batch, cuda_device)


def test_chunk_nan_key_reaches_every_row_that_sees_it(cuda_device):
    # A NaN in one cached key: the rows that see the key are NaN (as the definition gives), wherever the key's
    # column falls, and no other row is touched.
    spec, batch, prior, P = _lone_key_batch(19, "chunk_nan_key")
    ids = batch.chunk_ids
    rows, q_indptr = batch.chunk_rows()
    msl = int(batch.seq_lens_after.max())
    W.poison_dead_slots(batch, batch.seq_lens_before)
    kp, vp, after = oracle_append(batch)
    ref_o, _ = oracle.obs_chunk_attn(kp, vp, batch.page_table, after, q_indptr, W.bf16_to_u16(batch.q_new[rows]),
                                     spec.sm_scale, traj_ids=ids)
    for trial, off in enumerate((4, 37, 68, 101, 0, 127)):
        db = DeviceBatch(batch, cuda_device)
        ctx = make_ctx(spec, len(ids), msl)
        db.append(ctx)
        nan_pos = {}
        for t, L in enumerate(prior):
            pos = 128 * (1 + (t + trial) % 2) + off
            nan_pos[t] = pos
            pg = int(batch.page_table[t, pos // P])
            db.k_pool[pg, t % 2, pos % P, 7] = float("nan")
        q = db.q_new[torch.from_numpy(rows).to(cuda_device)].contiguous()
        out = torch.zeros_like(q)
        ctx.obs_chunk_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32(q_indptr, cuda_device), q,
                           spec.sm_scale, msl, out, traj_ids=dev_i32(ids, cuda_device))
        ctx.check()
        got = out.float().cpu().numpy()
        g = spec.num_q_heads // spec.num_kv_heads
        for i, t in enumerate(ids):
            a, b = int(q_indptr[i]), int(q_indptr[i + 1])
            hit = slice((t % 2) * g, (t % 2) * g + g)          # the query heads of the kv head that holds the NaN
            assert np.isnan(got[a:b, hit]).all(), (off, t)      # every chunk row sees the prior cache
            other = slice((1 - t % 2) * g, (1 - t % 2) * g + g)
            assert np.isfinite(got[a:b, other]).all(), (off, t)
            assert np.allclose(got[a:b, other], ref_o[a:b, other], atol=1e-2, rtol=2e-2), (off, t)


def test_chunk_second_pass_among_thousands_of_units(cuda_device):
    # More (item, kv head, M-tile pair) units than the bitmap of units to compute again has bits, a few of them with a
    # key that towers over the rows' reference: those go through the second kernel, their aliases in the bitmap with
    # them, and every row of every unit has to come out right whichever kernel wrote it last.
    P, hq, hkv = 16, 8, 8
    rng = np.random.default_rng(77)
    T = 700
    prior = rng.integers(129, 300, T).tolist()
    n_new = rng.integers(1, 4, T).tolist()
    batch = _custom_chunk_batch(P, hq, hkv, prior, n_new, 23, "chunk_many_units")
    assert T * hkv > 4096
    batch.q_new[:, :, 0] = 4.0
    for t in range(0, T, 97):
        pos = 128 + _LONE_OFFSETS[(t // 97) % len(_LONE_OFFSETS)]
        key = torch.zeros(128)
        key[0] = 300.0 / (4.0 * batch.spec.sm_scale * 1.4426950408889634)
        pg = int(batch.page_table[t, pos // P])
        batch.k_pool[pg, :, pos % P, :] = key.to(torch.bfloat16)
    run_chunk_case(batch, cuda_device)
