"""GPU parity of rollart_group_decode_attn: groups of trajectories that alias a shared prompt prefix.

The oracle has no notion of groups: the expected values are plain decode attention over each member's own
page-table row (which happens to list the same pages as its neighbours')."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2512_22560_b200 import rollart
from paper_2512_22560_b200 import workloads as W
from harness import DeviceBatch, assert_attn_close, assert_lse_close, dev_i32, oracle_append

pytestmark = pytest.mark.gpu


def group_ctx(spec, n_items, max_seq_len, device=0):
    return rollart.Context(device, rollart.group_decode_workspace_size(max(1, n_items), spec.num_q_heads,
                                                                       spec.num_kv_heads, max_seq_len))


def run_group_case(spec, seed, group_size, fraction, device, poison=True):
    batch = W.make_batch(spec, seed=seed)
    indptr, shared = W.share_group_prefix(batch, group_size, fraction)
    if poison:
        W.poison_dead_slots(batch, batch.seq_lens_before)
    msl = int(batch.seq_lens_after.max())
    T = spec.num_traj
    ctx = group_ctx(spec, T, msl)
    db = DeviceBatch(batch, device)
    db.append(ctx)
    q = db.q_new.contiguous()                       # decode-only specs: one row per trajectory
    out = torch.full_like(q, float("nan"))
    lse = torch.full((T, spec.num_q_heads), float("nan"), device=device)
    ctx.group_decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32(indptr, device),
                          dev_i32(shared, device), q, spec.sm_scale, msl, out, lse=lse)
    ctx.check()
    kp, vp, after = oracle_append(batch)
    ref_o, ref_l = oracle.decode_attn(kp, vp, batch.page_table, after, W.bf16_to_u16(batch.q_new), spec.sm_scale)
    assert_attn_close(out, ref_o, f"{spec.name} group={group_size} frac={fraction}")
    assert_lse_close(lse, ref_l, spec.name)
    # the plain decode call on the same inputs agrees to a few bf16 ulps (different split and rounding order)
    out2 = torch.full_like(q, float("nan"))
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, q, spec.sm_scale, msl, out2)
    ctx.check()
    assert torch.allclose(out.float(), out2.float(), atol=4e-3, rtol=2e-2)
    launches = ctx.launch_count
    ctx.close()
    return shared, launches


@pytest.mark.parametrize("group_size,fraction", [(8, 0.6), (8, 1.0), (3, 0.5), (1, 0.7), (8, 0.0), (40, 0.8)])
def test_group_decode_matches_oracle_gqa7(cuda_device, group_size, fraction):
    # 7 query heads per kv head (the 7B-like shape), page 16; 40 members exceed one 128-row tile (18 tokens at g = 7)
    spec = dataclasses.replace(W.shrink(W.CONFIGS[1], 40, 16), name="group_gqa7")
    shared, _ = run_group_case(spec, 31, group_size, fraction, cuda_device)
    if fraction > 0 and group_size > 1:
        assert shared.max() > 0


@pytest.mark.parametrize("cfg,div", [(2, 32), (3, 64), (4, 16)])
def test_group_decode_other_shapes(cuda_device, cfg, div):
    # g = 8 page 16, g = 16 page 64, g = 4 page 16
    spec = dataclasses.replace(W.shrink(W.CONFIGS[cfg], 24, div), chunk_fraction=0.0, name=f"group_cfg{cfg}")
    run_group_case(spec, 32 + cfg, 8, 0.75, cuda_device)


@pytest.mark.parametrize("group_size,num_traj", [(8, 600), (1, 600), (1, 1100), (2, 2300)])
def test_group_decode_many_items(cuda_device, group_size, num_traj):
    # more items (and, with small groups, more groups) than one launch of either kernel takes (512 items for the
    # decode kernel, 1024 groups for the prefix pass, whose longest-first order is per launch): the per-launch
    # offsets of every array
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=num_traj, len_lo=40, len_hi=200, name="group_many")
    run_group_case(spec, 35, group_size, 0.9, cuda_device, poison=False)


def test_member_without_private_keys_and_empty_prefix(cuda_device):
    # no append here: member 1's context IS the shared prefix (its private part is empty), and group 1 has no prefix
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=6, len_lo=256, len_hi=256, name="group_edges")   # 17 pages each
    batch = W.make_batch(spec, seed=36)
    batch.seq_lens_before[:] = [200, 128, 131, 70, 1, 0]
    batch.page_table[1:3, :8] = batch.page_table[0, :8]
    indptr = np.asarray([0, 3, 6], dtype=np.int32)
    shared = np.asarray([128, 0], dtype=np.int32)
    dev = cuda_device
    db = DeviceBatch(batch, dev)
    ctx = group_ctx(spec, 6, 256)
    q = db.q_new.contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((6, spec.num_q_heads), float("nan"), device=dev)
    ctx.group_decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_before, dev_i32(indptr, dev), dev_i32(shared, dev),
                          q, spec.sm_scale, 256, out, lse=lse)
    ctx.check()
    ref_o, ref_l = oracle.decode_attn(W.bf16_to_u16(batch.k_pool), W.bf16_to_u16(batch.v_pool), batch.page_table,
                                      batch.seq_lens_before, W.bf16_to_u16(batch.q_new), spec.sm_scale)
    assert_attn_close(out, ref_o, "edges")
    assert_lse_close(lse[:5], ref_l[:5], "edges")
    assert torch.all(out[5] == 0) and torch.all(torch.isneginf(lse[5]))     # no keys at all
    ctx.close()


def test_group_decode_reruns_are_bit_identical(cuda_device):
    spec = dataclasses.replace(W.shrink(W.CONFIGS[2], 16, 32), name="group_rerun")
    batch = W.make_batch(spec, seed=37)
    indptr, shared = W.share_group_prefix(batch, 8, 0.8)
    db = DeviceBatch(batch, cuda_device)
    msl = int(batch.seq_lens_before.max())
    ctx = group_ctx(spec, 16, msl)
    q = db.q_new.contiguous()
    outs = []
    for _ in range(3):
        out = torch.full_like(q, float("nan"))
        ctx.group_decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_before, dev_i32(indptr, cuda_device),
                              dev_i32(shared, cuda_device), q, spec.sm_scale, msl, out)
        ctx.check()
        outs.append(out)
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))
    assert torch.equal(outs[0].view(torch.int16), outs[2].view(torch.int16))
    ctx.close()


def test_group_decode_errors(cuda_device):
    dev = cuda_device
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=8, len_lo=100, len_hi=300, name="group_err")
    batch = W.make_batch(spec, seed=38)
    indptr, shared = W.share_group_prefix(batch, 4, 0.5)
    db = DeviceBatch(batch, dev)
    msl = int(batch.seq_lens_before.max())
    q = db.q_new.contiguous()
    out = torch.zeros_like(q)
    args = (db.k_pool, db.v_pool, db.page_table, db.lens_before)

    # host side: workspace sized for the plain decode call only
    small = rollart.Context(0, rollart.workspace_size(8, spec.num_q_heads, spec.num_kv_heads, msl))
    with pytest.raises(rollart.RollartError) as e:
        small.group_decode_attn(*args, dev_i32(indptr, dev), dev_i32(shared, dev), q, spec.sm_scale, msl, out)
    assert e.value.status == rollart.ERR_WORKSPACE
    assert small.launch_count == 0
    small.close()

    ctx = group_ctx(spec, 8, msl)
    # a shared length that is not a whole number of pages
    bad = shared.copy(); bad[0] += 3
    ctx.group_decode_attn(*args, dev_i32(indptr, dev), dev_i32(bad, dev), q, spec.sm_scale, msl, out)
    assert ctx.status() == rollart.ERR_BOUNDS and "group_decode" in ctx.last_error()
    # a shared length beyond a member's context
    bad = shared.copy(); bad[1] = (int(batch.seq_lens_before[4:8].min()) // 16 + 1) * 16
    ctx.group_decode_attn(*args, dev_i32(indptr, dev), dev_i32(bad, dev), q, spec.sm_scale, msl, out)
    assert ctx.status() == rollart.ERR_BOUNDS
    # a member whose row does not list the group's prefix pages
    table = db.page_table.clone()
    assert shared[0] >= 16
    table[2, 0] = table[5, 0]
    ctx.group_decode_attn(db.k_pool, db.v_pool, table, db.lens_before, dev_i32(indptr, dev), dev_i32(shared, dev), q,
                          spec.sm_scale, msl, out)
    assert ctx.status() == rollart.ERR_BOUNDS and "group_decode" in ctx.last_error()
    # an indptr that does not cover the items
    ctx.group_decode_attn(*args, dev_i32([0, 4, 7], dev), dev_i32(shared, dev), q, spec.sm_scale, msl, out)
    assert ctx.status() == rollart.ERR_BOUNDS
    ctx.group_decode_attn(*args, dev_i32([0, 5, 3], dev), dev_i32(shared, dev), q, spec.sm_scale, msl, out)
    assert ctx.status() == rollart.ERR_BOUNDS
    # the context still computes correctly afterwards
    ctx.group_decode_attn(*args, dev_i32(indptr, dev), dev_i32(shared, dev), q, spec.sm_scale, msl, out)
    ctx.check()
    ref_o, _ = oracle.decode_attn(W.bf16_to_u16(batch.k_pool), W.bf16_to_u16(batch.v_pool), batch.page_table,
                                  batch.seq_lens_before, W.bf16_to_u16(batch.q_new), spec.sm_scale)
    assert_attn_close(out, ref_o, "after errors")
    ctx.close()


def test_full_size_group_decode_sampled(cuda_device):
    """The GRPO workload bench.py times (512 trajectories in 64 groups), in its launch configuration: append, then
    the group call; sampled members are recomputed by the oracle from a host copy of just their pages."""
    dev = cuda_device
    spec = W.GROUP_DECODE
    layout = W.make_layout(spec, W.MASTER_SEED)
    indptr, shared = W.share_group_prefix(layout, W.GROUP_SIZE, W.GROUP_SHARED_FRACTION)
    batch = W.fill_tensors(layout, dev)
    db = DeviceBatch(batch, dev)
    msl = int(batch.seq_lens_after.max())
    ctx = group_ctx(spec, spec.num_traj, msl)
    db.append(ctx)
    q = db.q_new.contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((spec.num_traj, spec.num_q_heads), float("nan"), device=dev)
    ctx.group_decode_attn(db.k_pool, db.v_pool, db.page_table, db.lens_after, dev_i32(indptr, dev), dev_i32(shared, dev),
                          q, spec.sm_scale, msl, out, lse=lse)
    ctx.check()
    assert ctx.launch_count == 1 + 4                      # append; prepare, shared part, private part, merge
    assert torch.all(torch.isfinite(out.float())) and torch.all(torch.isfinite(lse))
    lens = batch.seq_lens_before
    order = np.argsort(lens, kind="stable")
    gi = int(np.argmax(shared))                           # the group with the longest prefix: first and last member
    pick = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2]), int(indptr[gi]), int(indptr[gi + 1] - 1), 77})
    b2 = dataclasses.replace(batch)
    b2.k_pool, b2.v_pool = db.k_pool, db.v_pool           # pools after the GPU append
    post = W.extract_trajs(b2, pick)
    sel = torch.tensor(pick, device=dev)
    ref_o, ref_l = oracle.decode_attn(W.bf16_to_u16(post.k_pool), W.bf16_to_u16(post.v_pool), post.page_table,
                                      post.seq_lens_before + 1, W.bf16_to_u16(q[sel]), spec.sm_scale)
    assert_attn_close(out[sel], ref_o, spec.name)
    assert_lse_close(lse[sel], ref_l, spec.name)
    ctx.close()


def test_full_size_fp8_group_decode_sampled(cuda_device):
    """The group call over fp8 pools on the GRPO workload at the size bench.py times: quantising append, group call,
    sampled members recomputed by the oracle's plain fp8 decode from a host copy of their pages' codes."""
    dev = cuda_device
    spec = W.GROUP_DECODE
    ks, vs = 0.03, 0.02
    layout = W.make_layout(spec, W.MASTER_SEED)
    indptr, shared = W.share_group_prefix(layout, W.GROUP_SIZE, W.GROUP_SHARED_FRACTION)
    batch = W.fill_tensors(layout, dev)
    # any codes will do for the existing cache (the oracle reads the same bytes); aliased prefix pages are the same
    # physical pages, so the members of a group see the same codes there
    k8 = (batch.k_pool.float() / ks).clamp_(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)
    v8 = (batch.v_pool.float() / vs).clamp_(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)
    T = spec.num_traj
    msl = int(batch.seq_lens_after.max())
    table, lens0 = dev_i32(batch.page_table, dev), dev_i32(batch.seq_lens_before, dev)
    lens1 = torch.empty_like(lens0)
    ctx = group_ctx(spec, T, msl)
    ctx.kv_append_fp8(k8, v8, table, lens0, dev_i32(batch.new_indptr, dev), batch.k_new, batch.v_new, ks, vs, seq_lens_out=lens1)
    q = batch.q_new.contiguous()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((T, spec.num_q_heads), float("nan"), device=dev)
    need = rollart.obs_chunk_fp8_scratch_size(len(indptr) - 1, spec.num_kv_heads, spec.page_size, msl)
    scratch = torch.empty(need, dtype=torch.uint8, device=dev)
    ctx.group_decode_attn_fp8(k8, v8, table, lens1, dev_i32(indptr, dev), dev_i32(shared, dev), q, spec.sm_scale, ks, vs, msl, out,
                              scratch, lse=lse)
    ctx.check()
    assert torch.all(torch.isfinite(out.float())) and torch.all(torch.isfinite(lse))
    del scratch
    lens = batch.seq_lens_before
    order = np.argsort(lens, kind="stable")
    gi = int(np.argmax(shared))
    pick = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2]), int(indptr[gi]), int(indptr[gi + 1] - 1), 77})
    b8 = dataclasses.replace(batch)
    b8.k_pool, b8.v_pool = k8, v8                         # codes after the GPU append
    post = W.extract_trajs(b8, pick)
    sel = torch.tensor(pick, device=dev)
    ref_o, ref_l = oracle.decode_attn_fp8(post.k_pool.numpy(), post.v_pool.numpy(), post.page_table, post.seq_lens_before + 1,
                                          W.bf16_to_u16(q[sel]), spec.sm_scale, ks, vs)
    assert_attn_close(out[sel], ref_o, spec.name + " fp8")
    assert_lse_close(lse[sel], ref_l, spec.name + " fp8")
    ctx.close()


def run_fp8_group_case(spec, seed, group_size, fraction, device, ks=0.03, vs=0.02):
    """The group call over fp8 pools: the cache is the oracle's quantisation of the bf16 recipe (members alias the same
    prefix pages, so they hold the same codes), the new token goes through the quantising append; expected values are
    the oracle's plain fp8 decode over each member's own row."""
    batch = W.make_batch(spec, seed=seed)
    indptr, shared = W.share_group_prefix(batch, group_size, fraction)
    T = spec.num_traj
    msl = int(batch.seq_lens_after.max())
    k8 = oracle.fp8_quantize_rows(W.bf16_to_u16(batch.k_pool), ks)
    v8 = oracle.fp8_quantize_rows(W.bf16_to_u16(batch.v_pool), vs)
    dk, dv = torch.from_numpy(k8.copy()).to(device), torch.from_numpy(v8.copy()).to(device)
    table, lens0 = dev_i32(batch.page_table, device), dev_i32(batch.seq_lens_before, device)
    lens1 = torch.empty_like(lens0)
    ctx = group_ctx(spec, T, msl)
    ctx.kv_append_fp8(dk, dv, table, lens0, dev_i32(batch.new_indptr, device), batch.k_new.to(device), batch.v_new.to(device),
                      ks, vs, seq_lens_out=lens1)
    after = oracle.kv_append_fp8(k8, v8, batch.page_table, batch.seq_lens_before, batch.new_indptr,
                                 W.bf16_to_u16(batch.k_new), W.bf16_to_u16(batch.v_new), ks, vs)
    q = batch.q_new.contiguous().to(device)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((T, spec.num_q_heads), float("nan"), device=device)
    n_groups = len(indptr) - 1
    need = rollart.obs_chunk_fp8_scratch_size(n_groups, spec.num_kv_heads, spec.page_size, msl)
    scratch = torch.full((need,), 0xFF, dtype=torch.uint8, device=device)
    ctx.group_decode_attn_fp8(dk, dv, table, lens1, dev_i32(indptr, device), dev_i32(shared, device), q, spec.sm_scale, ks, vs,
                              msl, out, scratch, lse=lse)
    ctx.check()
    assert np.array_equal(dk.cpu().numpy(), k8) and np.array_equal(dv.cpu().numpy(), v8)
    ref_o, ref_l = oracle.decode_attn_fp8(k8, v8, batch.page_table, after, W.bf16_to_u16(batch.q_new), spec.sm_scale, ks, vs)
    assert_attn_close(out, ref_o, f"{spec.name} fp8 group={group_size} frac={fraction}")
    assert_lse_close(lse, ref_l, spec.name + " fp8")
    out2 = torch.full_like(q, float("nan"))
    ctx.decode_attn_fp8(dk, dv, table, lens1, q, spec.sm_scale, ks, vs, msl, out2)
    ctx.check()
    assert torch.allclose(out.float(), out2.float(), atol=4e-3, rtol=2e-2)
    with pytest.raises(rollart.RollartError) as e:
        ctx.group_decode_attn_fp8(dk, dv, table, lens1, dev_i32(indptr, device), dev_i32(shared, device), q, spec.sm_scale, ks,
                                  vs, msl, out, scratch[:1024], lse=lse)
    assert e.value.status == rollart.ERR_WORKSPACE
    ctx.close()
    return shared


@pytest.mark.parametrize("group_size,fraction", [(8, 0.6), (8, 1.0), (3, 0.5), (1, 0.7), (8, 0.0), (40, 0.8)])
def test_fp8_group_decode_matches_oracle_gqa7(cuda_device, group_size, fraction):
    spec = dataclasses.replace(W.shrink(W.CONFIGS[1], 40, 16), name="fp8_group_gqa7")
    shared = run_fp8_group_case(spec, 31, group_size, fraction, cuda_device)
    if fraction > 0 and group_size > 1:
        assert shared.max() > 0


@pytest.mark.parametrize("cfg,div", [(2, 32), (3, 64), (4, 16)])
def test_fp8_group_decode_other_shapes(cuda_device, cfg, div):
    spec = dataclasses.replace(W.shrink(W.CONFIGS[cfg], 24, div), chunk_fraction=0.0, name=f"fp8_group_cfg{cfg}")
    run_fp8_group_case(spec, 32 + cfg, 8, 0.75, cuda_device)


@pytest.mark.parametrize("num_traj", [600, 1100])
def test_fp8_group_decode_many_items(cuda_device, num_traj):
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=num_traj, len_lo=40, len_hi=200, name="fp8_group_many")
    run_fp8_group_case(spec, 35, 1, 0.9, cuda_device)
