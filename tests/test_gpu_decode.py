"""Decode attention on the GPU vs the fp64 oracle (|err| <= 1e-2 + 2e-2 |ref|), through the C ABI."""
import dataclasses
import math

import numpy as np
import pytest
import torch

import oracle
from harness import (DeviceBatch, assert_attn_close, assert_lse_close, dev_i32, make_ctx, oracle_append)
from paper_2512_22560_b200 import rollart
from paper_2512_22560_b200 import workloads as W

pytestmark = pytest.mark.gpu


def run_decode_case(batch, device, poison=True, with_lse=True, max_seq_len=None):
    """append + decode on the GPU and in the oracle for every decode trajectory of `batch`."""
    spec = batch.spec
    if poison:
        W.poison_dead_slots(batch, batch.seq_lens_before)
    ids = batch.decode_ids
    rows = batch.decode_rows()
    msl = int(batch.seq_lens_after.max()) if max_seq_len is None else max_seq_len
    ctx = make_ctx(spec, len(ids), msl)
    db = DeviceBatch(batch, device)
    db.append(ctx)
    q = db.q_new[torch.from_numpy(rows).to(device)].contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((len(ids), spec.num_q_heads), float("nan"), device=device) if with_lse else None
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, q, spec.sm_scale, msl, out, lse=lse,
                    traj_ids=dev_i32(ids, device))
    ctx.check()
    kp, vp, after = oracle_append(batch)
    ref_o, ref_l = oracle.decode_attn(kp, vp, batch.page_table, after, W.bf16_to_u16(batch.q_new[rows]), spec.sm_scale,
                                      traj_ids=ids)
    st = assert_attn_close(out, ref_o, spec.name)
    if with_lse:
        assert_lse_close(lse, ref_l, spec.name)
    ctx.close()
    return out, st


def test_cfg0_tiny_decode_full(cuda_device):
    run_decode_case(W.make_batch(W.CONFIGS[0]), cuda_device)


@pytest.mark.parametrize("i,T,div", [(1, 16, 4), (2, 12, 16), (3, 4, 16), (4, 10, 8)])
def test_shrunk_configs(cuda_device, i, T, div):
    run_decode_case(W.make_batch(W.shrink(W.CONFIGS[i], T, div, 16), seed=200 + i), cuda_device)


@pytest.mark.parametrize("P", [16, 32, 64])
@pytest.mark.parametrize("hq,hkv", [(1, 1), (4, 2), (6, 2), (7, 1), (16, 2), (16, 1), (5, 5)])
def test_edge_lengths_groups_and_page_sizes(cuda_device, P, hq, hkv):
    lens = [0, 1, 2, P - 2, P - 1, P, 62, 63, 64, 65, 127, 128, 129, 191, 193, 255, 257, 700]
    spec = dataclasses.replace(W.CONFIGS[0], page_size=P, num_traj=len(lens), num_q_heads=hq, num_kv_heads=hkv,
                               name=f"edge_p{P}_{hq}_{hkv}")
    batch = W.make_layout(spec, seed=31)
    batch.seq_lens_before = np.array(lens, np.int32)
    pages = (batch.seq_lens_before + 1 + P - 1) // P
    batch.page_table, batch.num_pages = W.build_page_table(pages.astype(np.int64), 0.3, np.random.default_rng(8))
    W.fill_tensors(batch)
    run_decode_case(batch, cuda_device)


def test_zero_length_trajectory_gives_zero_and_minus_inf(cuda_device):
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=3, name="zero")
    batch = W.make_batch(spec, seed=4)
    db = DeviceBatch(batch, cuda_device)
    ctx = make_ctx(spec, 3, 600)
    lens = dev_i32([0, 5, 0], cuda_device)
    q = db.q_new[:3].contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((3, spec.num_q_heads), float("nan"), device=cuda_device)
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, lens, q, 0.1, 600, out, lse=lse)
    ctx.check()
    assert torch.all(out[0] == 0) and torch.all(out[2] == 0)
    assert torch.all(torch.isneginf(lse[0])) and torch.all(torch.isneginf(lse[2]))
    assert torch.all(torch.isfinite(out[1])) and torch.all(torch.isfinite(lse[1]))


def test_needles_give_order_one_outputs(cuda_device):
    spec = W.shrink(W.CONFIGS[2], 6, 8)
    batch = W.make_batch(spec, seed=77)
    P = spec.page_size
    pos = {}
    for t in range(spec.num_traj):
        L = int(batch.seq_lens_before[t])
        pos[t] = sorted({0, L - 1, min(L - 1, P - 1), (L // P) * P if L % P else L - P, L // 2, min(L - 1, 64), L})
    W.plant_needles(batch, pos)      # position L is the appended token itself
    out, st = run_decode_case(batch, cuda_device)
    assert st["rms_ref"] > 0.2


def test_rerun_is_bit_identical_and_schedule_change_stays_close(cuda_device):
    batch = W.make_batch(W.shrink(W.CONFIGS[3], 3, 8), seed=5)
    a, _ = run_decode_case(batch, cuda_device, poison=False)
    batch2 = W.make_batch(W.shrink(W.CONFIGS[3], 3, 8), seed=5)
    b, _ = run_decode_case(batch2, cuda_device, poison=False)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    # a different host bound changes how contexts are split; results stay within a few bf16 ulps
    batch3 = W.make_batch(W.shrink(W.CONFIGS[3], 3, 8), seed=5)
    c, _ = run_decode_case(batch3, cuda_device, poison=False, max_seq_len=5 * int(batch.seq_lens_after.max()))
    assert torch.allclose(a.float(), c.float(), atol=2e-3, rtol=2e-2)


def test_shared_prefix_pages(cuda_device):
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=2, name="shared")
    batch = W.make_batch(spec, seed=6)
    batch.seq_lens_before[:] = [100, 90]
    batch.page_table[1, :4] = batch.page_table[0, :4]          # 64 shared prefix tokens
    run_decode_case(batch, cuda_device, poison=False)


def test_device_side_errors(cuda_device):
    batch = W.make_batch(W.shrink(W.CONFIGS[0], 4, 2), seed=13)
    spec = batch.spec
    db = DeviceBatch(batch, cuda_device)
    ctx = make_ctx(spec, 4, 400)
    db.append(ctx)
    q = db.q_new.contiguous()
    out = torch.zeros_like(q)
    table = db.page_table.clone()
    table[1, 0] = -3
    ctx.decode_attn(db.k_pool, db.v_pool, table, db.lens_after, q, 0.1, 400, out)
    assert ctx.status() == rollart.ERR_BOUNDS and "decode_attn" in ctx.last_error()
    # a trajectory longer than the host bound is reported too
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, q, 0.1, 16, out)
    assert ctx.status() == rollart.ERR_BOUNDS
    # and the context still computes correctly afterwards
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, q, spec.sm_scale, 400, out)
    ctx.check()
    kp, vp, after = oracle_append(batch)
    ref, _ = oracle.decode_attn(kp, vp, batch.page_table, after, W.bf16_to_u16(batch.q_new), spec.sm_scale)
    assert_attn_close(out, ref)


def test_host_side_validation(cuda_device):
    batch = W.make_batch(W.shrink(W.CONFIGS[3], 2, 16), seed=14)
    spec = batch.spec
    db = DeviceBatch(batch, cuda_device)
    q = db.q_new.contiguous()
    out = torch.zeros_like(q)
    small = rollart.Context(0, 1024)
    with pytest.raises(rollart.RollartError) as e:
        small.decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_before, q, 0.1, 8000, out)
    assert e.value.status == rollart.ERR_WORKSPACE
    ctx = make_ctx(spec, 2, 8000)
    with pytest.raises(rollart.RollartError) as e:       # 64 q heads over 4 kv heads is fine, 3 kv heads is not
        ctx.decode_attn(db.k_pool[:, :3].contiguous(), db.v_pool[:, :3].contiguous(), db.page_table, db.lens_before, q,
                        0.1, 8000, out)
    assert e.value.status == rollart.ERR_INVALID_ARG


def test_more_items_than_one_launch_holds(cuda_device):
    # 1300 short trajectories: the decode call splits into several launches (the per-launch length table is bounded)
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=1300, len_lo=1, len_hi=90, name="many_items")
    run_decode_case(W.make_batch(spec, seed=71), cuda_device)


@pytest.mark.parametrize("lens", [[5, 5, 5], [1], [70, 3, 130, 2, 64]])
def test_fewer_tiles_than_blocks(cuda_device, lens):
    # a call far smaller than the machine: most blocks get nothing, and some spans of the tile line hold only the
    # fixed-cost padding that follows an (item, head), i.e. no piece at all
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=len(lens), num_q_heads=4, num_kv_heads=1, name="tiny_line")
    batch = W.make_layout(spec, seed=5)
    batch.seq_lens_before = np.array(lens, np.int32)
    pages = (batch.seq_lens_before + 1 + spec.page_size - 1) // spec.page_size
    batch.page_table, batch.num_pages = W.build_page_table(pages.astype(np.int64), 0.3, np.random.default_rng(9))
    W.fill_tensors(batch)
    run_decode_case(batch, cuda_device)


@pytest.mark.parametrize("i,T,div", [(0, 4, 1), (1, 16, 4), (3, 4, 16), (4, 10, 8)])
def test_fused_append_decode_equals_the_two_calls_and_the_oracle(cuda_device, i, T, div):
    batch = W.make_batch(W.shrink(W.CONFIGS[i], T, div, 16), seed=500 + i)
    spec = batch.spec
    W.poison_dead_slots(batch, batch.seq_lens_before)
    ids, rows = batch.decode_ids, batch.decode_rows()
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, len(ids), msl)
    db = DeviceBatch(batch, cuda_device)
    ridx = torch.from_numpy(rows).to(cuda_device)
    q, k_new, v_new = (x[ridx].contiguous() for x in (db.q_new, db.k_new, db.v_new))
    out = torch.full_like(q, float("nan"))
    lse = torch.full((len(ids), spec.num_q_heads), float("nan"), device=cuda_device)
    lens_out = db.lens_before.clone()
    ctx.append_decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_before, k_new, v_new, q, spec.sm_scale, msl, out, lse=lse,
                           traj_ids=dev_i32(ids, cuda_device), seq_lens_out=lens_out)
    ctx.check()
    # oracle: append only the decode trajectories' token, then decode
    kp, vp = W.bf16_to_u16(batch.k_pool), W.bf16_to_u16(batch.v_pool)
    after = oracle.kv_append(kp, vp, batch.page_table, batch.seq_lens_before, np.arange(len(ids) + 1, dtype=np.int32),
                             W.bf16_to_u16(batch.k_new[rows]), W.bf16_to_u16(batch.v_new[rows]), traj_ids=ids)
    ref_o, ref_l = oracle.decode_attn(kp, vp, batch.page_table, after, W.bf16_to_u16(batch.q_new[rows]), spec.sm_scale, traj_ids=ids)
    assert np.array_equal(W.bf16_to_u16(db.k_pool), kp) and np.array_equal(W.bf16_to_u16(db.v_pool), vp)
    assert np.array_equal(lens_out.cpu().numpy(), after)
    assert_attn_close(out, ref_o, spec.name + " fused")
    assert_lse_close(lse, ref_l, spec.name + " fused")
    # and bit-identical to a plain decode call over the pool the fused call left behind
    out2 = torch.empty_like(out)
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, lens_out, q, spec.sm_scale, msl, out2, traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))


def test_fused_step_skips_an_item_that_outgrows_the_bound(cuda_device):
    # max_seq_len one short for the longest trajectory: that item is rejected as a whole (error reported, row not
    # stored, length not advanced, output row 0); every other item is as the oracle says.
    batch = W.make_batch(W.shrink(W.CONFIGS[0], 4, 1), seed=77)
    spec = batch.spec
    ids, rows = batch.decode_ids, batch.decode_rows()
    longest = int(np.argmax(batch.seq_lens_after[ids]))
    msl = int(batch.seq_lens_after[ids].max()) - 1
    ctx = make_ctx(spec, len(ids), msl + 1)
    db = DeviceBatch(batch, cuda_device)
    ridx = torch.from_numpy(rows).to(cuda_device)
    q, k_new, v_new = (x[ridx].contiguous() for x in (db.q_new, db.k_new, db.v_new))
    out = torch.full_like(q, float("nan"))
    lens_out = torch.full_like(db.lens_before, -5)
    ctx.append_decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_before, k_new, v_new, q, spec.sm_scale, msl, out,
                           traj_ids=dev_i32(ids, cuda_device), seq_lens_out=lens_out)
    assert ctx.status() == rollart.ERR_BOUNDS
    keep = np.array([j for j in range(len(ids)) if j != longest])
    kp, vp = W.bf16_to_u16(batch.k_pool), W.bf16_to_u16(batch.v_pool)
    after = oracle.kv_append(kp, vp, batch.page_table, batch.seq_lens_before, np.arange(len(keep) + 1, dtype=np.int32),
                             W.bf16_to_u16(batch.k_new[rows[keep]]), W.bf16_to_u16(batch.v_new[rows[keep]]), traj_ids=ids[keep])
    assert np.array_equal(W.bf16_to_u16(db.k_pool), kp) and np.array_equal(W.bf16_to_u16(db.v_pool), vp)   # the rejected row was not stored
    got = lens_out.cpu().numpy()
    assert got[ids[longest]] == -5 and np.array_equal(got[ids[keep]], after[ids[keep]])
    ref_o, _ = oracle.decode_attn(kp, vp, batch.page_table, after, W.bf16_to_u16(batch.q_new[rows[keep]]), spec.sm_scale, traj_ids=ids[keep])
    assert_attn_close(out[torch.from_numpy(keep).to(cuda_device)], ref_o, "fused step, items within the bound")
    assert bool(torch.all(out[longest] == 0))
    ctx.close()


@pytest.mark.parametrize("i,T,div", [(0, 4, 1), (1, 16, 4), (3, 4, 16)])
def test_results_written_straight_to_pinned_host_memory(cuda_device, i, T, div):
    """out / lse may be page-locked host tensors: the kernel's stores then cross to the host; same bits as device buffers."""
    batch = W.make_batch(W.shrink(W.CONFIGS[i], T, div, 16), seed=700 + i)
    spec = batch.spec
    ids, rows = batch.decode_ids, batch.decode_rows()
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, len(ids), msl)
    db = DeviceBatch(batch, cuda_device)
    db.append(ctx)
    q = db.q_new[torch.from_numpy(rows).to(cuda_device)].contiguous()
    tid = dev_i32(ids, cuda_device)
    out_d = torch.full_like(q, float("nan"))
    lse_d = torch.full((len(ids), spec.num_q_heads), float("nan"), device=cuda_device)
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, q, spec.sm_scale, msl, out_d, lse=lse_d, traj_ids=tid)
    out_h = torch.full(tuple(q.shape), float("nan"), dtype=torch.bfloat16).pin_memory()
    lse_h = torch.full(tuple(lse_d.shape), float("nan")).pin_memory()
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, q, spec.sm_scale, msl, out_h, lse=lse_h, traj_ids=tid)
    ctx.check()                                                       # synchronises the stream: the host may read now
    assert torch.equal(out_h.view(torch.int16), out_d.cpu().view(torch.int16)) and torch.equal(lse_h, lse_d.cpu())
    kp, vp, after = oracle_append(batch)
    ref_o, _ = oracle.decode_attn(kp, vp, batch.page_table, after, W.bf16_to_u16(batch.q_new[rows]), spec.sm_scale, traj_ids=ids)
    assert_attn_close(out_h, ref_o, spec.name + " host out")
    with pytest.raises(ValueError):
        ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, q, spec.sm_scale, msl,
                        torch.empty(tuple(q.shape), dtype=torch.bfloat16), traj_ids=tid)          # pageable host memory
    ctx.close()


def test_decode_steps_replayed_from_a_cuda_graph(cuda_device):
    """The engine runs rollout with CUDA graphs (Sec. 7.1): the calls are asynchronous, allocate nothing and read their
    lengths on the device, so one captured step replays for every following token.  Four replayed steps (lengths
    advancing on the device) against four eager steps: pools, lengths and outputs bit for bit, and the last step
    against the oracle."""
    steps = 4
    batch = W.make_batch(W.shrink(W.CONFIGS[1], 12, 4, 16), seed=800)
    spec = batch.spec
    ids = batch.decode_ids
    n = len(ids)
    msl = int(batch.seq_lens_before.max()) + steps
    P = spec.page_size
    # pages for the extra tokens: one more table column, and the rows that need a page take one of the spare pages
    table = np.concatenate([batch.page_table, np.full((spec.num_traj, 1), -1, np.int32)], axis=1)
    used = set(int(p) for t in range(spec.num_traj) for p in table[t, : (int(batch.seq_lens_after[t]) + P - 1) // P])
    spare = [p for p in range(batch.num_pages) if p not in used]
    for t in ids:
        have = (int(batch.seq_lens_after[t]) + P - 1) // P
        want = (int(batch.seq_lens_before[t]) + steps + P - 1) // P
        for lp in range(have, want):
            table[t, lp] = spare.pop()
    g = torch.Generator(device="cpu").manual_seed(5)
    qs = torch.randn(steps, n, spec.num_q_heads, 128, generator=g).to(torch.bfloat16).to(cuda_device)
    kns = torch.randn(steps, n, spec.num_kv_heads, 128, generator=g).to(torch.bfloat16).to(cuda_device)
    vns = torch.randn(steps, n, spec.num_kv_heads, 128, generator=g).to(torch.bfloat16).to(cuda_device)
    tid = dev_i32(ids, cuda_device)
    d_table = dev_i32(table, cuda_device)
    ctx = make_ctx(spec, n, msl)

    def fresh():
        return (batch.k_pool.clone().to(cuda_device), batch.v_pool.clone().to(cuda_device),
                dev_i32(batch.seq_lens_before, cuda_device), dev_i32(batch.seq_lens_before, cuda_device))

    # eager
    kp, vp, la, lb = fresh()
    outs_e = torch.full_like(qs, float("nan"))
    for s in range(steps):
        ctx.append_decode_attn(kp, vp, d_table, la, kns[s], vns[s], qs[s], spec.sm_scale, msl, outs_e[s], traj_ids=tid,
                               seq_lens_out=lb)
        la.copy_(lb)
    ctx.check()
    # one captured step, replayed
    kp2, vp2, la2, lb2 = fresh()
    q_in, k_in, v_in = torch.empty_like(qs[0]), torch.empty_like(kns[0]), torch.empty_like(vns[0])
    o_out = torch.full_like(qs[0], float("nan"))
    side = torch.cuda.Stream(device=cuda_device)
    graph = torch.cuda.CUDAGraph()
    q_in.copy_(qs[0]); k_in.copy_(kns[0]); v_in.copy_(vns[0])
    torch.cuda.synchronize(cuda_device)
    with torch.cuda.graph(graph, stream=side):
        ctx.append_decode_attn(kp2, vp2, d_table, la2, k_in, v_in, q_in, spec.sm_scale, msl, o_out, traj_ids=tid, seq_lens_out=lb2)
        la2.copy_(lb2)
    outs_g = torch.full_like(qs, float("nan"))
    for s in range(steps):
        q_in.copy_(qs[s]); k_in.copy_(kns[s]); v_in.copy_(vns[s])
        graph.replay()
        outs_g[s].copy_(o_out)
    torch.cuda.synchronize(cuda_device)
    ctx.check()
    assert torch.equal(kp.view(torch.int16), kp2.view(torch.int16)) and torch.equal(vp.view(torch.int16), vp2.view(torch.int16))
    assert torch.equal(la, la2) and torch.equal(la.cpu(), torch.from_numpy(np.where(
        np.isin(np.arange(spec.num_traj), ids), batch.seq_lens_before + steps, batch.seq_lens_before)).to(torch.int32))
    assert torch.equal(outs_e.view(torch.int16), outs_g.view(torch.int16))
    # the last step against the oracle, over the pools the replays left behind
    ref_o, _ = oracle.decode_attn(W.bf16_to_u16(kp2), W.bf16_to_u16(vp2), table, la2.cpu().numpy(), W.bf16_to_u16(qs[-1]),
                                  spec.sm_scale, traj_ids=ids)
    assert_attn_close(outs_g[-1], ref_o, "graph replay, last step")
    ctx.close()


@pytest.mark.parametrize("i,T,div", [(0, 4, 1), (1, 16, 4), (3, 4, 16)])
def test_fused_step_driven_from_host_buffers(cuda_device, i, T, div):
    """q / k_new / v_new in pinned host memory, copied in by the call itself, result written to pinned host
    memory: pools, lengths and outputs bit for bit as with device buffers; a second step after the host has rewritten
    its buffers sees the new values."""
    batch = W.make_batch(W.shrink(W.CONFIGS[i], T, div, 16), seed=900 + i)
    spec = batch.spec
    ids, rows = batch.decode_ids, batch.decode_rows()
    n = len(ids)
    msl = int(batch.seq_lens_after.max()) + 1
    table = np.concatenate([batch.page_table, np.full((spec.num_traj, 1), -1, np.int32)], axis=1)
    P = spec.page_size
    used = set(int(p) for t in range(spec.num_traj) for p in table[t, : (int(batch.seq_lens_after[t]) + P - 1) // P])
    spare = [p for p in range(batch.num_pages) if p not in used]
    for t in ids:                                                # room for a second token
        have, want = (int(batch.seq_lens_after[t]) + P - 1) // P, (int(batch.seq_lens_before[t]) + 2 + P - 1) // P
        for lp in range(have, want):
            table[t, lp] = spare.pop()
    ctx = make_ctx(spec, n, msl)
    d_table, tid = dev_i32(table, cuda_device), dev_i32(ids, cuda_device)
    ridx = torch.from_numpy(rows)
    steps = [(batch.q_new[ridx].contiguous(), batch.k_new[ridx].contiguous(), batch.v_new[ridx].contiguous())]
    steps.append(tuple((x.float() * -0.5 + 0.25).to(torch.bfloat16) for x in steps[0]))
    staging = torch.empty(rollart.host_staging_size(n, spec.num_q_heads, spec.num_kv_heads), dtype=torch.uint8, device=cuda_device)
    res = {}
    for mode in ("device", "host"):
        kp, vp = batch.k_pool.clone().to(cuda_device), batch.v_pool.clone().to(cuda_device)
        la, lb = dev_i32(batch.seq_lens_before, cuda_device), dev_i32(batch.seq_lens_before, cuda_device)
        hq_, hk_, hv_ = (torch.empty_like(x).pin_memory() for x in steps[0])
        outs = []
        for q, kn, vn in steps:
            if mode == "device":
                out = torch.full_like(q, float("nan"), device=cuda_device)
                ctx.append_decode_attn(kp, vp, d_table, la, kn.to(cuda_device), vn.to(cuda_device), q.to(cuda_device),
                                       spec.sm_scale, msl, out, traj_ids=tid, seq_lens_out=lb)
            else:
                hq_.copy_(q); hk_.copy_(kn); hv_.copy_(vn)       # the host rewrites its buffers between the steps
                out = torch.full(tuple(q.shape), float("nan"), dtype=torch.bfloat16).pin_memory()
                ctx.append_decode_attn_host(kp, vp, d_table, la, hk_, hv_, hq_, spec.sm_scale, msl, out, staging, traj_ids=tid,
                                            seq_lens_out=lb)
            la.copy_(lb)
            ctx.check()
            outs.append(out.cpu().clone())
        res[mode] = (kp, vp, la.clone(), outs)
    a, b = res["device"], res["host"]
    assert torch.equal(a[0].view(torch.int16), b[0].view(torch.int16)) and torch.equal(a[1].view(torch.int16), b[1].view(torch.int16))
    assert torch.equal(a[2], b[2])
    for x, y in zip(a[3], b[3]):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))
    ref_o, _ = oracle.decode_attn(W.bf16_to_u16(b[0]), W.bf16_to_u16(b[1]), table, b[2].cpu().numpy(), W.bf16_to_u16(steps[1][0]),
                                  spec.sm_scale, traj_ids=ids)
    assert_attn_close(b[3][1], ref_o, spec.name + " host step")
    with pytest.raises(ValueError):                              # device tensors are not host buffers
        ctx.append_decode_attn_host(b[0], b[1], d_table, b[2], hk_.to(cuda_device), hv_, hq_, spec.sm_scale, msl,
                                    torch.empty(tuple(hq_.shape), dtype=torch.bfloat16).pin_memory(), staging, traj_ids=tid)
    with pytest.raises(rollart.RollartError) as e:
        ctx.append_decode_attn_host(b[0], b[1], d_table, b[2], hk_, hv_, hq_, spec.sm_scale, msl,
                                    torch.empty(tuple(hq_.shape), dtype=torch.bfloat16).pin_memory(), staging[:256], traj_ids=tid)
    assert e.value.status == rollart.ERR_WORKSPACE
    ctx.close()
