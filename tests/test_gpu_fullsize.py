"""Full-size workloads in the launch configuration bench.py times, checked on sampled trajectories.

The whole batch runs on the GPU (append + decode, and for the mixed batch the chunk call too);
the oracle then recomputes a sample of trajectories one by one from a host copy of just their
pages (page renumbering does not change the oracle's result: see the permutation pin)."""
import numpy as np
import pytest
import torch

import oracle
from harness import DeviceBatch, assert_attn_close, assert_lse_close, dev_i32, make_ctx
from paper_2512_22560_b200 import rollart
from paper_2512_22560_b200 import workloads as W

pytestmark = pytest.mark.gpu


def sample_ids(lens, ids, k, rng):
    """shortest, longest, median and a few random members of `ids`"""
    order = ids[np.argsort(lens[ids], kind="stable")]
    pick = {int(order[0]), int(order[-1]), int(order[len(order) // 2])}
    while len(pick) < min(k, len(ids)):
        pick.add(int(rng.choice(ids)))
    return np.array(sorted(pick), dtype=np.int64)


@pytest.mark.parametrize("cfg", [1, 2, 3, 4])
def test_full_size_decode_sampled(cuda_device, cfg):
    spec = W.CONFIGS[cfg]
    batch = W.make_batch(spec, device=cuda_device)          # the seed and shapes bench.py uses
    ids = batch.decode_ids
    rows = batch.decode_rows()
    msl = int(batch.seq_lens_after[ids].max())
    ctx = make_ctx(spec, len(ids), msl)
    db = DeviceBatch(batch, cuda_device)
    # append only the decode trajectories' token, exactly as the bench step does
    ridx = torch.from_numpy(rows).to(cuda_device)
    q = db.q_new[ridx].contiguous()
    ctx.kv_append(db.k_pool, db.v_pool, db.page_table, db.lens_before, dev_i32(np.arange(len(ids) + 1), cuda_device),
                  db.k_new[ridx].contiguous(), db.v_new[ridx].contiguous(), traj_ids=dev_i32(ids, cuda_device),
                  seq_lens_out=db.lens_after)
    lens_after = db.lens_before.clone()
    lens_after[torch.from_numpy(ids.astype(np.int64)).to(cuda_device)] += 1
    out = torch.full_like(q, float("nan"))
    lse = torch.full((len(ids), spec.num_q_heads), float("nan"), device=cuda_device)
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, lens_after, q, spec.sm_scale, msl, out, lse=lse,
                    traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    assert torch.all(torch.isfinite(out.float())) and torch.all(torch.isfinite(lse))
    # run twice: bit-identical (fixed schedule and merge order)
    out2 = torch.empty_like(out)
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, lens_after, q, spec.sm_scale, msl, out2,
                    traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    # the fused call (what bench.py times) on a fresh copy of the pools: same bytes, same output bits
    fresh = W.make_batch(spec, device=cuda_device)
    out3 = torch.empty_like(out)
    lens3 = db.lens_before.clone()
    ctx.append_decode_attn(fresh.k_pool, fresh.v_pool, db.page_table, db.lens_before, db.k_new[ridx].contiguous(),
                           db.v_new[ridx].contiguous(), q, spec.sm_scale, msl, out3, traj_ids=dev_i32(ids, cuda_device),
                           seq_lens_out=lens3)
    ctx.check()
    assert torch.equal(out3.view(torch.int16), out.view(torch.int16))
    assert torch.equal(fresh.k_pool.view(torch.int16), db.k_pool.view(torch.int16))
    assert torch.equal(fresh.v_pool.view(torch.int16), db.v_pool.view(torch.int16))
    assert torch.equal(lens3, lens_after)
    del fresh

    rng = np.random.default_rng(cfg)
    pick = sample_ids(batch.seq_lens_before, ids, 5, rng)
    # host copy of the sampled trajectories' pages AFTER the GPU append; the oracle's append must
    # reproduce those bytes from the pre-append pages
    post = W.extract_trajs(db_as_batch(batch, db), pick)
    kp, vp = W.bf16_to_u16(post.k_pool), W.bf16_to_u16(post.v_pool)
    after = post.seq_lens_before + 1
    pos = {int(t): i for i, t in enumerate(ids)}
    sel = np.array([pos[int(t)] for t in pick])
    ref_o, ref_l = oracle.decode_attn(kp, vp, post.page_table, after, W.bf16_to_u16(q[torch.from_numpy(sel).to(cuda_device)]),
                                      spec.sm_scale)
    assert_attn_close(out[torch.from_numpy(sel).to(cuda_device)], ref_o, spec.name)
    assert_lse_close(lse[torch.from_numpy(sel).to(cuda_device)], ref_l, spec.name)
    # the appended token sits where the oracle's indexing says: last logical position of each sample
    P = spec.page_size
    for i, t in enumerate(pick):
        L = int(batch.seq_lens_before[t])
        pg = int(post.page_table[i, L // P])
        r = int(batch.new_indptr[t])
        assert np.array_equal(kp[pg, :, L % P, :], W.bf16_to_u16(batch.k_new[r]))
        assert np.array_equal(vp[pg, :, L % P, :], W.bf16_to_u16(batch.v_new[r]))
    ctx.close()


@pytest.mark.parametrize("cfg", [1, 2, 3])
def test_full_size_decode_with_needles(cuda_device, cfg):
    # The same full-size step with keys planted that dominate the softmax (outputs of order one instead of
    # ~1/sqrt(L): a wrong key, page or split would show): first and last token, page edges, the appended token,
    # and one every 2048 positions so that every block's span of the sampled trajectories holds some.
    spec = W.CONFIGS[cfg]
    batch = W.make_batch(spec, device=cuda_device)
    ids = batch.decode_ids
    rng = np.random.default_rng(100 + cfg)
    pick = sample_ids(batch.seq_lens_before, ids, 4, rng)
    P = spec.page_size
    pos = {}
    for t in pick:
        L = int(batch.seq_lens_before[t])
        special = {0, L - 1, min(L - 1, P - 1), min(L - 1, P), (L // P) * P if L % P else L - P, L}
        pos[int(t)] = sorted(special | set(range(1027, L, 2048)))
    W.plant_needles(batch, pos)
    rows = batch.decode_rows()
    msl = int(batch.seq_lens_after[ids].max())
    ctx = make_ctx(spec, len(ids), msl)
    db = DeviceBatch(batch, cuda_device)
    ridx = torch.from_numpy(rows).to(cuda_device)
    q = db.q_new[ridx].contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((len(ids), spec.num_q_heads), float("nan"), device=cuda_device)
    ctx.append_decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_before, db.k_new[ridx].contiguous(),
                           db.v_new[ridx].contiguous(), q, spec.sm_scale, msl, out, lse=lse, traj_ids=dev_i32(ids, cuda_device),
                           seq_lens_out=db.lens_after)
    ctx.check()
    post = W.extract_trajs(db_as_batch(batch, db), pick)
    kp, vp = W.bf16_to_u16(post.k_pool), W.bf16_to_u16(post.v_pool)
    where = {int(t): i for i, t in enumerate(ids)}
    sel = torch.from_numpy(np.array([where[int(t)] for t in pick])).to(cuda_device)
    ref_o, ref_l = oracle.decode_attn(kp, vp, post.page_table, post.seq_lens_before + 1, W.bf16_to_u16(q[sel]), spec.sm_scale)
    st = assert_attn_close(out[sel], ref_o, spec.name + " (needles)")
    assert st["rms_ref"] > 0.1, st
    assert_lse_close(lse[sel], ref_l, spec.name + " (needles)")
    ctx.close()


@pytest.mark.parametrize("cfg", [1, 2, 3])
def test_full_size_fp8_step_sampled(cuda_device, cfg):
    # The fused fp8 step (quantised append + decode in one launch) at full size, as bench.py times it; the oracle
    # recomputes sampled trajectories from a host copy of their pages' codes after the step.
    spec = W.CONFIGS[cfg]
    ks, vs = 0.03, 0.03
    batch = W.make_batch(spec, device=cuda_device)
    ids = batch.decode_ids
    rows = batch.decode_rows()
    msl = int(batch.seq_lens_after[ids].max())
    ctx = make_ctx(spec, len(ids), msl)
    # any codes will do for the existing cache (the oracle reads the same bytes): a clamped cast of the bf16 pools
    k8 = (batch.k_pool.float() / ks).clamp_(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)
    v8 = (batch.v_pool.float() / vs).clamp_(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)
    table, lens0 = dev_i32(batch.page_table, cuda_device), dev_i32(batch.seq_lens_before, cuda_device)
    lens1 = torch.full_like(lens0, -7)
    ridx = torch.from_numpy(rows).to(cuda_device)
    q, kn, vn = batch.q_new[ridx].contiguous(), batch.k_new[ridx].contiguous(), batch.v_new[ridx].contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((len(ids), spec.num_q_heads), float("nan"), device=cuda_device)
    tid = dev_i32(ids, cuda_device)
    ctx.append_decode_attn_fp8(k8, v8, table, lens0, kn, vn, q, spec.sm_scale, ks, vs, msl, out, lse=lse, traj_ids=tid,
                               seq_lens_out=lens1)
    ctx.check()
    assert torch.all(torch.isfinite(out.float())) and torch.all(torch.isfinite(lse))
    rng = np.random.default_rng(40 + cfg)
    pick = sample_ids(batch.seq_lens_before, ids, 4, rng)
    import dataclasses
    b8 = dataclasses.replace(batch)
    b8.k_pool, b8.v_pool = k8, v8
    post = W.extract_trajs(b8, pick)
    kp, vp = post.k_pool.numpy(), post.v_pool.numpy()
    where = {int(t): i for i, t in enumerate(ids)}
    sel = torch.from_numpy(np.array([where[int(t)] for t in pick])).to(cuda_device)
    ref_o, ref_l = oracle.decode_attn_fp8(kp, vp, post.page_table, post.seq_lens_before + 1, W.bf16_to_u16(q[sel]),
                                          spec.sm_scale, ks, vs)
    assert_attn_close(out[sel], ref_o, spec.name + " fp8")
    assert_lse_close(lse[sel], ref_l, spec.name + " fp8")
    # the appended token's codes are the oracle's quantisation of its row, at the slot the oracle's indexing names
    P = spec.page_size
    kq = oracle.fp8_quantize_rows(W.bf16_to_u16(kn[sel]), ks)
    vq = oracle.fp8_quantize_rows(W.bf16_to_u16(vn[sel]), vs)
    for i, t in enumerate(pick):
        L = int(batch.seq_lens_before[t])
        pg = int(post.page_table[i, L // P])
        assert np.array_equal(kp[pg, :, L % P, :], kq[i]) and np.array_equal(vp[pg, :, L % P, :], vq[i])
    assert torch.equal(lens1[tid.long()].cpu(), torch.from_numpy(batch.seq_lens_before[ids] + 1).to(torch.int32))
    ctx.close()


def db_as_batch(batch, db):
    """the batch with its pools replaced by the device pools after the GPU append"""
    import dataclasses
    b = dataclasses.replace(batch)
    b.k_pool, b.v_pool = db.k_pool, db.v_pool
    return b



def test_full_size_mixed_batch_chunk_sampled_rows(cuda_device):
    spec = W.CONFIGS[4]
    batch = W.make_batch(spec, device=cuda_device)
    ids = batch.chunk_ids
    rows, q_indptr = batch.chunk_rows()
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, len(ids), msl)
    db = DeviceBatch(batch, cuda_device)
    db.append(ctx)                                            # all 128 trajectories: chunks and single tokens
    q = db.q_new[torch.from_numpy(rows).to(cuda_device)].contiguous()
    out = torch.full_like(q, float("nan"))
    ctx.obs_chunk_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32(q_indptr, cuda_device), q, spec.sm_scale,
                       msl, out, traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    assert torch.all(torch.isfinite(out.float()))
    # stratified rows of three chunk trajectories: first/last row, tile edges, page edges, random
    rng = np.random.default_rng(44)
    order = np.argsort(batch.n_new[ids], kind="stable")
    pick_local = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2])})
    pick = ids[pick_local]
    post = W.extract_trajs(db_as_batch(batch, db), pick)
    kp, vp = W.bf16_to_u16(post.k_pool), W.bf16_to_u16(post.v_pool)
    after = post.seq_lens_before + post.n_new
    row_traj, row_count, q_rows = [], [], []
    for i, li in enumerate(pick_local):
        n = int(batch.n_new[ids[li]])
        cand = {0, 1, n - 1, n - 2, n // 2} | {r for e in range(32, n, 128) for r in (e - 1, e, e + 1)}
        cand |= {int(x) for x in rng.integers(0, n, size=24)}
        for j in sorted(c for c in cand if 0 <= c < n):
            row_traj.append(i)
            row_count.append(int(after[i]) - n + j + 1)
            q_rows.append(int(q_indptr[li]) + j)
    q_rows = np.array(q_rows)
    qsel = q[torch.from_numpy(q_rows).to(cuda_device)]
    ref_o, _ = oracle.attend_rows(kp, vp, post.page_table, row_traj, row_count, W.bf16_to_u16(qsel), spec.sm_scale)
    assert_attn_close(out[torch.from_numpy(q_rows).to(cuda_device)], ref_o, "cfg4 chunk rows")
    # the pairs take their units from a counter, in whatever order they finish: the result must not depend on it
    again = torch.full_like(q, float("nan"))
    ctx.obs_chunk_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32(q_indptr, cuda_device), q, spec.sm_scale,
                       msl, again, traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    assert torch.equal(again.view(torch.int16), out.view(torch.int16))
    ctx.close()


def test_full_size_mixed_batch_fp8_chunk_sampled_rows(cuda_device):
    # the chunk half of the mixed batch over fp8 pools, as bench.py times it: quantising append of everything, chunk
    # attention over the codes (expansion into the scratch pool + the bf16 kernel); sampled rows against the oracle,
    # which reads a host copy of the sampled trajectories' codes after the append
    import dataclasses
    spec = W.CONFIGS[4]
    ks, vs = 0.03, 0.03
    batch = W.make_batch(spec, device=cuda_device)
    ids = batch.chunk_ids
    rows, q_indptr = batch.chunk_rows()
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, len(ids), msl)
    k8 = (batch.k_pool.float() / ks).clamp_(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)
    v8 = (batch.v_pool.float() / vs).clamp_(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)
    table, lens0 = dev_i32(batch.page_table, cuda_device), dev_i32(batch.seq_lens_before, cuda_device)
    lens1 = torch.empty_like(lens0)
    ctx.kv_append_fp8(k8, v8, table, lens0, dev_i32(batch.new_indptr, cuda_device), batch.k_new, batch.v_new, ks, vs,
                      seq_lens_out=lens1)
    q = batch.q_new[torch.from_numpy(rows).to(cuda_device)].contiguous()
    out = torch.full_like(q, float("nan"))
    need = rollart.obs_chunk_fp8_scratch_size(len(ids), spec.num_kv_heads, spec.page_size, msl)
    scratch = torch.empty(need, dtype=torch.uint8, device=cuda_device)
    ctx.obs_chunk_attn_fp8(k8, v8, table, lens1, dev_i32(q_indptr, cuda_device), q, spec.sm_scale, ks, vs, msl, out, scratch,
                           traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    assert torch.all(torch.isfinite(out.float()))
    del scratch
    rng = np.random.default_rng(45)
    order = np.argsort(batch.n_new[ids], kind="stable")
    pick_local = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2])})
    pick = ids[pick_local]
    b8 = dataclasses.replace(batch)
    b8.k_pool, b8.v_pool = k8, v8
    post = W.extract_trajs(b8, pick)
    kp, vp = post.k_pool.numpy(), post.v_pool.numpy()
    after = post.seq_lens_before + post.n_new
    row_traj, row_count, q_rows = [], [], []
    for i, li in enumerate(pick_local):
        n = int(batch.n_new[ids[li]])
        cand = {0, 1, n - 1, n - 2, n // 2} | {r for e in range(32, n, 128) for r in (e - 1, e, e + 1)}
        cand |= {int(x) for x in rng.integers(0, n, size=24)}
        for j in sorted(c for c in cand if 0 <= c < n):
            row_traj.append(i)
            row_count.append(int(after[i]) - n + j + 1)
            q_rows.append(int(q_indptr[li]) + j)
    q_rows = torch.from_numpy(np.array(q_rows)).to(cuda_device)
    sm = float(np.float32(spec.sm_scale) * np.float32(ks))
    ref_o, _ = oracle.attend_rows(oracle.fp8_pool_as_bf16_bits(kp), oracle.fp8_pool_as_bf16_bits(vp), post.page_table, row_traj,
                                  row_count, W.bf16_to_u16(q[q_rows]), sm)
    assert_attn_close(out[q_rows], ref_o * float(np.float32(vs)), "cfg4 fp8 chunk rows")
    ctx.close()


def _stratified_rows(n, tile, rng, n_random):
    """first / last rows, rows around tile edges near the start, the middle and the end of an n-row chunk, random rows"""
    edges = [e for e in range(tile, n, tile)]
    near = edges[:3] + edges[len(edges) // 2: len(edges) // 2 + 3] + edges[-3:]
    cand = {0, 1, n - 2, n - 1} | {r for e in near for r in (e - 1, e, e + 1)}
    cand |= {int(x) for x in rng.integers(0, n, size=n_random)}
    return sorted(c for c in cand if 0 <= c < n)


def test_full_size_recompute_sampled_rows(cuda_device):
    # KV recomputation at the size bench.py times: whole contexts of up to 32 K tokens as one causal chunk onto empty
    # pages.  Thousands of M-tiles per (item, head), thousands of key tiles on the last ones.  Rows of the shortest,
    # the median and the longest trajectory against the oracle, out and lse.
    spec = W.RECOMPUTE
    batch = W.make_batch(spec, device=cuda_device)
    ids = batch.chunk_ids
    rows, q_indptr = batch.chunk_rows()
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, len(ids), msl)
    db = DeviceBatch(batch, cuda_device)
    db.append(ctx)
    q = db.q_new[torch.from_numpy(rows).to(cuda_device)].contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], spec.num_q_heads), float("nan"), device=cuda_device)
    ctx.obs_chunk_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32(q_indptr, cuda_device), q, spec.sm_scale,
                       msl, out, lse=lse, traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    assert torch.all(torch.isfinite(out.float())) and torch.all(torch.isfinite(lse))
    rng = np.random.default_rng(46)
    order = np.argsort(batch.n_new[ids], kind="stable")
    pick_local = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2])})
    pick = ids[pick_local]
    post = W.extract_trajs(db_as_batch(batch, db), pick)
    kp, vp = W.bf16_to_u16(post.k_pool), W.bf16_to_u16(post.v_pool)
    after = post.seq_lens_before + post.n_new
    tile = 128 // (spec.num_q_heads // spec.num_kv_heads)           # chunk tokens per 128-row tile of the kernel
    row_traj, row_count, q_rows = [], [], []
    for i, li in enumerate(pick_local):
        n = int(batch.n_new[ids[li]])
        for j in _stratified_rows(n, tile, rng, 64):
            row_traj.append(i)
            row_count.append(int(after[i]) - n + j + 1)
            q_rows.append(int(q_indptr[li]) + j)
    q_rows = torch.from_numpy(np.array(q_rows)).to(cuda_device)
    ref_o, ref_l = oracle.attend_rows(kp, vp, post.page_table, row_traj, row_count, W.bf16_to_u16(q[q_rows]), spec.sm_scale)
    assert_attn_close(out[q_rows], ref_o, "recompute rows")
    assert_lse_close(lse[q_rows], ref_l, "recompute rows")
    ctx.close()


def test_full_size_mixed_batch_chunk_lse_and_needles(cuda_device):
    # The chunk half of the mixed batch with keys planted that dominate the softmax of sampled chunk rows (outputs of
    # order one: a wrong key, page or tile would show): for each sampled row, keys aligned with that row's own
    # queries in the prior cache (first token, page edges, one every 2048 positions), at the first chunk token and at
    # the row's own position.  out and lse of those rows and of their neighbours against the oracle.
    spec = W.CONFIGS[4]
    batch = W.make_batch(spec, device=cuda_device)
    ids = batch.chunk_ids
    rows, q_indptr = batch.chunk_rows()
    g, P = spec.num_q_heads // spec.num_kv_heads, spec.page_size
    rng = np.random.default_rng(47)
    order = np.argsort(batch.n_new[ids], kind="stable")
    pick_local = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2])})
    tile = 128 // g
    sampled = {}                                                     # local index -> chunk rows with needles
    for li in pick_local:
        t = int(ids[li])
        n, prior = int(batch.n_new[t]), int(batch.seq_lens_before[t])
        edges = [e for e in range(tile, n, tile)]
        js = sorted({0, n - 1, n // 2} | {r for e in edges[:2] + edges[-2:] for r in (e - 1, e)} | {int(x) for x in rng.integers(0, n, size=6)})
        js = [j for j in js if 0 <= j < n]
        sampled[li] = js
        for k, j in enumerate(js):
            qrow = int(batch.new_indptr[t]) + j
            qv = batch.q_new[qrow].float().view(spec.num_kv_heads, g, spec.head_dim)
            count = prior + j + 1
            want = {0, P - 1, P, prior - 1, prior, count - 1} | set(range(1027, count, 2048))
            for pos in sorted(p_ for p_ in want if 0 <= p_ < count):
                pos = min(count - 1, pos + 3 * k) if pos not in (prior, count - 1) else pos     # rows do not share needles
                kvec = (3.0 * qv[:, pos % g, :]).to(torch.bfloat16)
                if pos < prior:
                    batch.k_pool[int(batch.page_table[t, pos // P]), :, pos % P, :] = kvec
                else:
                    batch.k_new[int(batch.new_indptr[t]) + (pos - prior)] = kvec
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, len(ids), msl)
    db = DeviceBatch(batch, cuda_device)
    db.append(ctx)
    q = db.q_new[torch.from_numpy(rows).to(cuda_device)].contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], spec.num_q_heads), float("nan"), device=cuda_device)
    ctx.obs_chunk_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32(q_indptr, cuda_device), q, spec.sm_scale,
                       msl, out, lse=lse, traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    post = W.extract_trajs(db_as_batch(batch, db), ids[pick_local])
    kp, vp = W.bf16_to_u16(post.k_pool), W.bf16_to_u16(post.v_pool)
    after = post.seq_lens_before + post.n_new
    row_traj, row_count, q_rows = [], [], []
    for i, li in enumerate(pick_local):
        n = int(batch.n_new[ids[li]])
        for j in sorted({r for j in sampled[li] for r in (j - 1, j, j + 1) if 0 <= r < n}):
            row_traj.append(i)
            row_count.append(int(after[i]) - n + j + 1)
            q_rows.append(int(q_indptr[li]) + j)
    q_rows = torch.from_numpy(np.array(q_rows)).to(cuda_device)
    ref_o, ref_l = oracle.attend_rows(kp, vp, post.page_table, row_traj, row_count, W.bf16_to_u16(q[q_rows]), spec.sm_scale)
    st = assert_attn_close(out[q_rows], ref_o, "cfg4 chunk rows (needles)")
    assert st["rms_ref"] > 0.1, st
    assert_lse_close(lse[q_rows], ref_l, "cfg4 chunk rows (needles)")
    ctx.close()


def test_full_size_mixed_batch_decode_half_with_needles(cuda_device):
    # the decode half of the mixed batch (64 single-token trajectories among 128) with planted keys, as the decode
    # needle test above does for the three decode workloads
    spec = W.CONFIGS[4]
    batch = W.make_batch(spec, device=cuda_device)
    ids = batch.decode_ids
    rng = np.random.default_rng(104)
    pick = sample_ids(batch.seq_lens_before, ids, 4, rng)
    P = spec.page_size
    pos = {}
    for t in pick:
        L = int(batch.seq_lens_before[t])
        special = {0, L - 1, min(L - 1, P - 1), min(L - 1, P), (L // P) * P if L % P else L - P, L}
        pos[int(t)] = sorted(special | set(range(1027, L, 2048)))
    W.plant_needles(batch, pos)
    rows = batch.decode_rows()
    msl = int(batch.seq_lens_after[ids].max())
    ctx = make_ctx(spec, len(ids), msl)
    db = DeviceBatch(batch, cuda_device)
    ridx = torch.from_numpy(rows).to(cuda_device)
    q = db.q_new[ridx].contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((len(ids), spec.num_q_heads), float("nan"), device=cuda_device)
    ctx.append_decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_before, db.k_new[ridx].contiguous(),
                           db.v_new[ridx].contiguous(), q, spec.sm_scale, msl, out, lse=lse, traj_ids=dev_i32(ids, cuda_device),
                           seq_lens_out=db.lens_after)
    ctx.check()
    post = W.extract_trajs(db_as_batch(batch, db), pick)
    where = {int(t): i for i, t in enumerate(ids)}
    sel = torch.from_numpy(np.array([where[int(t)] for t in pick])).to(cuda_device)
    ref_o, ref_l = oracle.decode_attn(W.bf16_to_u16(post.k_pool), W.bf16_to_u16(post.v_pool), post.page_table,
                                      post.seq_lens_before + 1, W.bf16_to_u16(q[sel]), spec.sm_scale)
    st = assert_attn_close(out[sel], ref_o, spec.name + " decode half (needles)")
    assert st["rms_ref"] > 0.1, st
    assert_lse_close(lse[sel], ref_l, spec.name + " decode half (needles)")
    ctx.close()


def test_full_size_kv_gather_sampled(cuda_device):
    # the hand-off gather at the size bench.py times (the long-horizon workload: 32 trajectories, 2.6 M tokens): every
    # byte of three sampled trajectories' rows against the oracle's gather over a host copy of their pages
    spec = W.CONFIGS[3]
    batch = W.make_batch(spec, device=cuda_device)
    lens = batch.seq_lens_before
    indptr = np.concatenate([[0], np.cumsum(lens.astype(np.int64))])
    assert indptr[-1] < 2 ** 31
    ctx = rollart.Context(0, 0)
    table, d_lens = dev_i32(batch.page_table, cuda_device), dev_i32(lens, cuda_device)
    k_out = torch.full((int(indptr[-1]), spec.num_kv_heads, spec.head_dim), float("nan"), dtype=torch.bfloat16, device=cuda_device)
    v_out = torch.full_like(k_out, float("nan"))
    ctx.kv_gather(batch.k_pool, batch.v_pool, table, d_lens, dev_i32(indptr, cuda_device), k_out, v_out)
    ctx.check()
    rng = np.random.default_rng(48)
    pick = sample_ids(lens, np.arange(spec.num_traj), 3, rng)
    post = W.extract_trajs(batch, pick)
    sub_indptr = np.concatenate([[0], np.cumsum(post.seq_lens_before.astype(np.int64))]).astype(np.int32)
    rk, rv = oracle.kv_gather(W.bf16_to_u16(post.k_pool), W.bf16_to_u16(post.v_pool), post.page_table, post.seq_lens_before, sub_indptr)
    for i, t in enumerate(pick):
        a, b = int(indptr[t]), int(indptr[t + 1])
        assert np.array_equal(W.bf16_to_u16(k_out[a:b]), rk[sub_indptr[i]:sub_indptr[i + 1]])
        assert np.array_equal(W.bf16_to_u16(v_out[a:b]), rv[sub_indptr[i]:sub_indptr[i + 1]])
    ctx.close()
