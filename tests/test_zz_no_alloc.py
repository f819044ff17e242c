"""The allocation-free decode entry point (rollart_decode_attn_noalloc) against the regular one.

Some users of this library are not allowed to allocate device memory at run time: an inference
engine that has already given the whole GPU to its KV-cache pool, or code that runs under a
"no cudaMalloc after start-up" rule because an allocation synchronises the device and can fail.
They cannot create a Context (that is where the regular path allocates its workspace), so the
library offers one call that keeps its scratch in a fixed array inside the library image.  This
test drives that call through the C ABI twice in a row, with different inputs, and checks each
result against what the regular rollart_decode_attn call gives for the same inputs (the two run
the same kernel on the same grid, so the results must be the same bits, which is stricter than
the tolerance of the other attention tests) and against the CPU oracle within that tolerance.  The
second call shows that whatever the first one left in the shared array does not leak into later
results.  A third test makes the documented warm-up call (n_items = 0: set-up only) and then a
call that launches.  This file is named so that pytest collects it last.
"""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from harness import ATOL, RTOL, DeviceBatch, assert_attn_close, assert_lse_close, dev_i32, make_ctx, oracle_append
from paper_2512_22560_b200 import rollart
from paper_2512_22560_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _regular(ctx, db, q, lens, spec, msl, ids):
    out = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], spec.num_q_heads), float("nan"), device=q.device)
    ctx.decode_attn(db.k_pool, db.v_pool, db.page_table, lens, q, spec.sm_scale, msl, out, lse=lse, traj_ids=ids)
    ctx.check()
    return out, lse


def _close(a, b):
    a, b = a.float(), b.float()
    return bool(torch.all((a - b).abs() <= ATOL + RTOL * b.abs()))


def test_noalloc_decode_matches_regular_entry_point_twice(cuda_device):
    # long, ragged contexts over few (item, head) units: most pieces are partial, so the shared
    # scratch (slots + piece records) is exercised, not just the direct-output path
    spec = W.shrink(W.CONFIGS[3], 5, 8)
    batch = W.make_batch(spec, seed=91)
    W.poison_dead_slots(batch, batch.seq_lens_before)
    db = DeviceBatch(batch, cuda_device)
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, spec.num_traj, msl)
    db.append(ctx)
    ctx.check()
    status = torch.full((4,), 7, dtype=torch.int32, device=cuda_device)

    # call 1: all trajectories
    q1 = db.q_new.contiguous()
    ref1, ref_lse1 = _regular(ctx, db, q1, db.lens_after, spec, msl, None)
    out1 = torch.full_like(q1, float("nan"))
    lse1 = torch.full_like(ref_lse1, float("nan"))
    rollart.decode_attn_noalloc(db.k_pool, db.v_pool, db.page_table, db.lens_after, q1, spec.sm_scale, msl, out1, lse=lse1,
                                device_status=status)
    torch.cuda.synchronize()
    assert status[0].item() == 0
    assert _close(out1, ref1)
    assert torch.allclose(lse1, ref_lse1, atol=1e-3, rtol=1e-3)
    assert torch.equal(out1.view(torch.int16), ref1.view(torch.int16)) and torch.equal(lse1, ref_lse1)
    # and against the oracle, so that this test does not lean on the regular entry point alone
    kp, vp, after = oracle_append(batch)
    qbits = W.bf16_to_u16(batch.q_new)
    o_ref, l_ref = oracle.decode_attn(kp, vp, batch.page_table, after, qbits, spec.sm_scale)
    assert_attn_close(out1, o_ref, "noalloc call 1")
    assert_lse_close(lse1, l_ref, "noalloc call 1")

    # call 2, right after: a different subset in a different order with other queries and shorter lengths
    ids = dev_i32([3, 0, 4], cuda_device)
    lens2 = (db.lens_after // 3).contiguous()
    q2 = (-db.q_new[[1, 2, 0]]).contiguous()
    ref2, ref_lse2 = _regular(ctx, db, q2, lens2, spec, msl, ids)
    out2 = torch.full_like(q2, float("nan"))
    lse2 = torch.full_like(ref_lse2, float("nan"))
    rollart.decode_attn_noalloc(db.k_pool, db.v_pool, db.page_table, lens2, q2, spec.sm_scale, msl, out2, lse=lse2,
                                traj_ids=ids, device_status=status)
    torch.cuda.synchronize()
    assert status[0].item() == 0
    assert _close(out2, ref2)
    assert torch.allclose(lse2, ref_lse2, atol=1e-3, rtol=1e-3)
    assert torch.equal(out2.view(torch.int16), ref2.view(torch.int16)) and torch.equal(lse2, ref_lse2)
    o_ref2, l_ref2 = oracle.decode_attn(kp, vp, batch.page_table, after // 3, W.bf16_to_u16(q2.cpu()), spec.sm_scale,
                                        traj_ids=np.array([3, 0, 4]))
    assert_attn_close(out2, o_ref2, "noalloc call 2")
    assert_lse_close(lse2, l_ref2, "noalloc call 2")
    ctx.close()


def test_noalloc_empty_call_is_the_warm_up(cuda_device):
    # An embedder makes this call at start-up, before it takes the rest of the device's memory: with n_items = 0 the
    # entry point does its per-device set-up (symbol address, shared-memory limit) and launches nothing.
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=3, name="noalloc_warm_up")
    batch = W.make_batch(spec, seed=93)
    db = DeviceBatch(batch, cuda_device)
    empty = torch.zeros(0, spec.num_q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    rollart.decode_attn_noalloc(db.k_pool, db.v_pool, db.page_table, db.lens_before, empty, spec.sm_scale, 600,
                                torch.zeros_like(empty))
    # then a call that launches, checked against the oracle
    q = db.q_new[:3].contiguous()
    out = torch.full_like(q, float("nan"))
    status = torch.full((4,), 5, dtype=torch.int32, device=cuda_device)
    rollart.decode_attn_noalloc(db.k_pool, db.v_pool, db.page_table, db.lens_before, q, spec.sm_scale, 600, out,
                                device_status=status)
    torch.cuda.synchronize()
    assert status[0].item() == 0
    ref, _ = oracle.decode_attn(W.bf16_to_u16(batch.k_pool), W.bf16_to_u16(batch.v_pool), batch.page_table,
                                batch.seq_lens_before, W.bf16_to_u16(batch.q_new[:3]), spec.sm_scale)
    assert_attn_close(out, ref, "noalloc after warm-up")


def test_noalloc_rejects_calls_beyond_its_fixed_scratch_and_reports_device_errors(cuda_device):
    spec = dataclasses.replace(W.CONFIGS[0], num_traj=3, name="noalloc_small")
    batch = W.make_batch(spec, seed=92)
    db = DeviceBatch(batch, cuda_device)
    # 1100 items x 2 kv heads = 2200 units > 2048: refused on the host with a message that names the limit
    n = 1100
    q = torch.zeros(n, spec.num_q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    out = torch.zeros_like(q)
    ids = dev_i32(np.zeros(n), cuda_device)
    with pytest.raises(rollart.RollartError) as e:
        rollart.decode_attn_noalloc(db.k_pool, db.v_pool, db.page_table, db.lens_before, q, 0.1, 600, out, traj_ids=ids)
    assert e.value.status == rollart.ERR_WORKSPACE and "2048" in str(e.value)
    # a page id outside the pool is reported through the caller's status word, not by a fault
    table = db.page_table.clone()
    table[1, 0] = batch.num_pages + 9
    status = torch.zeros(4, dtype=torch.int32, device=cuda_device)
    q3 = db.q_new[:3].contiguous()
    out3 = torch.zeros_like(q3)
    rollart.decode_attn_noalloc(db.k_pool, db.v_pool, table, db.lens_before, q3, 0.1, 600, out3, device_status=status)
    torch.cuda.synchronize()
    assert status[0].item() == rollart.ERR_BOUNDS
    # and the next call starts from a clean status word
    rollart.decode_attn_noalloc(db.k_pool, db.v_pool, db.page_table, db.lens_before, q3, 0.1, 600, out3, device_status=status)
    torch.cuda.synchronize()
    assert status[0].item() == 0 and bool(torch.all(torch.isfinite(out3.float())))
