"""fp8 (E4M3) KV pools on the GPU vs the oracle: the quantised append bit for bit, decode attention within tolerance."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from harness import assert_attn_close, assert_lse_close, dev_i32, make_ctx
from paper_2512_22560_b200 import rollart
from paper_2512_22560_b200 import workloads as W

pytestmark = pytest.mark.gpu

KS, VS = 0.03, 0.02      # pool scales: N(0,1) data / 0.03 spans the E4M3 range up to +-448 with a few saturated values


def run_fp8_case(batch, device, ks=KS, vs=VS, poison=True):
    """Quantise the existing cache with the oracle (as if every token had been appended through the fp8 call),
    then append the new rows and decode on the GPU and in the oracle."""
    spec = batch.spec
    ids = batch.decode_ids
    rows = batch.decode_rows()
    k8 = oracle.fp8_quantize_rows(W.bf16_to_u16(batch.k_pool), ks)
    v8 = oracle.fp8_quantize_rows(W.bf16_to_u16(batch.v_pool), vs)
    if poison:
        # dead slots (beyond each trajectory's length, and pages nobody owns) may hold anything, NaN codes included
        live = np.zeros(k8.shape[:1] + k8.shape[2:3], bool)
        P = spec.page_size
        for t in range(spec.num_traj):
            L = int(batch.seq_lens_before[t])
            for lp in range((L + P - 1) // P):
                live[batch.page_table[t, lp], : min(P, L - lp * P)] = True
        dead = ~live
        k8[np.broadcast_to(dead[:, None, :, None], k8.shape)] = 0x7F
        v8[np.broadcast_to(dead[:, None, :, None], v8.shape)] = 0xFF
    dk, dv = torch.from_numpy(k8.copy()).to(device), torch.from_numpy(v8.copy()).to(device)
    table, lens0 = dev_i32(batch.page_table, device), dev_i32(batch.seq_lens_before, device)
    lens1 = torch.full_like(lens0, -7)
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, len(ids), msl)
    ctx.kv_append_fp8(dk, dv, table, lens0, dev_i32(batch.new_indptr, device), batch.k_new.to(device), batch.v_new.to(device),
                      ks, vs, seq_lens_out=lens1)
    after = oracle.kv_append_fp8(k8, v8, batch.page_table, batch.seq_lens_before, batch.new_indptr,
                                 W.bf16_to_u16(batch.k_new), W.bf16_to_u16(batch.v_new), ks, vs)
    ctx.check()
    assert np.array_equal(dk.cpu().numpy(), k8) and np.array_equal(dv.cpu().numpy(), v8), "quantised append differs"
    assert np.array_equal(lens1.cpu().numpy(), after)
    q = batch.q_new[torch.from_numpy(rows)].contiguous()
    out = torch.full_like(q, float("nan"), device=device)
    lse = torch.full((len(ids), spec.num_q_heads), float("nan"), device=device)
    ctx.decode_attn_fp8(dk, dv, table, lens1, q.to(device), spec.sm_scale, ks, vs, msl, out, lse=lse,
                        traj_ids=dev_i32(ids, device))
    ctx.check()
    ref_o, ref_l = oracle.decode_attn_fp8(k8, v8, batch.page_table, after, W.bf16_to_u16(q), spec.sm_scale, ks, vs,
                                          traj_ids=ids)
    st = assert_attn_close(out, ref_o, spec.name + " fp8")
    assert_lse_close(lse, ref_l, spec.name + " fp8")
    ctx.close()
    return st


def test_cfg0_tiny(cuda_device):
    run_fp8_case(W.make_batch(W.CONFIGS[0]), cuda_device)


@pytest.mark.parametrize("i,T,div", [(1, 16, 4), (2, 12, 16), (3, 4, 16), (4, 10, 8)])
def test_shrunk_configs(cuda_device, i, T, div):
    run_fp8_case(W.make_batch(W.shrink(W.CONFIGS[i], T, div, 16), seed=300 + i), cuda_device)


@pytest.mark.parametrize("P", [16, 32, 64])
@pytest.mark.parametrize("hq,hkv", [(1, 1), (6, 2), (7, 1), (16, 1), (5, 5)])
def test_edge_lengths_groups_and_page_sizes(cuda_device, P, hq, hkv):
    lens = [0, 1, 2, P - 1, P, 62, 63, 64, 65, 127, 128, 129, 193, 257, 700]
    spec = dataclasses.replace(W.CONFIGS[0], page_size=P, num_traj=len(lens), num_q_heads=hq, num_kv_heads=hkv,
                               name=f"fp8_edge_p{P}_{hq}_{hkv}")
    batch = W.make_layout(spec, seed=33)
    batch.seq_lens_before = np.array(lens, np.int32)
    pages = (batch.seq_lens_before + 1 + P - 1) // P
    batch.page_table, batch.num_pages = W.build_page_table(pages.astype(np.int64), 0.3, np.random.default_rng(8))
    W.fill_tensors(batch)
    run_fp8_case(batch, cuda_device)


def test_append_of_chunks_saturation_and_scales(cuda_device):
    # observation chunks through the quantised append (rows straddle pages), data far beyond the code range
    spec = dataclasses.replace(W.shrink(W.CONFIGS[4], 6, 32, 16), name="fp8_chunks")
    batch = W.make_batch(spec, seed=9)
    batch.k_new = (batch.k_new.float() * 40.0).to(torch.bfloat16)         # most of these saturate at scale 0.03
    k8 = np.full(tuple(batch.k_pool.shape), 0x11, np.uint8)
    v8 = np.full(tuple(batch.v_pool.shape), 0x22, np.uint8)
    dk, dv = torch.from_numpy(k8.copy()).to(cuda_device), torch.from_numpy(v8.copy()).to(cuda_device)
    ctx = make_ctx(spec, spec.num_traj, int(batch.seq_lens_after.max()))
    ctx.kv_append_fp8(dk, dv, dev_i32(batch.page_table, cuda_device), dev_i32(batch.seq_lens_before, cuda_device),
                      dev_i32(batch.new_indptr, cuda_device), batch.k_new.to(cuda_device), batch.v_new.to(cuda_device), 0.03, 1.7)
    ctx.check()
    oracle.kv_append_fp8(k8, v8, batch.page_table, batch.seq_lens_before, batch.new_indptr, W.bf16_to_u16(batch.k_new),
                         W.bf16_to_u16(batch.v_new), 0.03, 1.7)
    assert np.array_equal(dk.cpu().numpy(), k8) and np.array_equal(dv.cpu().numpy(), v8)
    assert (k8 == 0x7E).sum() + (k8 == 0xFE).sum() > 1000
    ctx.close()


@pytest.mark.parametrize("i,T,div", [(0, 4, 1), (1, 16, 4), (3, 4, 16), (4, 10, 8)])
def test_fused_fp8_step_equals_the_two_calls(cuda_device, i, T, div):
    spec = W.CONFIGS[i] if i == 0 else W.shrink(W.CONFIGS[i], T, div, 16)
    batch = W.make_batch(spec, seed=500 + i)
    ids = batch.decode_ids
    rows = torch.from_numpy(batch.decode_rows())
    k8 = oracle.fp8_quantize_rows(W.bf16_to_u16(batch.k_pool), KS)
    v8 = oracle.fp8_quantize_rows(W.bf16_to_u16(batch.v_pool), VS)
    table, lens0 = dev_i32(batch.page_table, cuda_device), dev_i32(batch.seq_lens_before, cuda_device)
    tid = dev_i32(ids, cuda_device)
    q = batch.q_new[rows].contiguous().to(cuda_device)
    kn, vn = batch.k_new[rows].contiguous().to(cuda_device), batch.v_new[rows].contiguous().to(cuda_device)
    msl = int(batch.seq_lens_after.max())
    ctx = make_ctx(spec, len(ids), msl)
    res = []
    for fused in (False, True):
        dk, dv = torch.from_numpy(k8.copy()).to(cuda_device), torch.from_numpy(v8.copy()).to(cuda_device)
        lens1 = lens0.clone()
        out = torch.full_like(q, float("nan"))
        lse = torch.full((len(ids), spec.num_q_heads), float("nan"), device=cuda_device)
        if fused:
            lens_out = torch.full_like(lens0, -7)
            ctx.append_decode_attn_fp8(dk, dv, table, lens0, kn, vn, q, spec.sm_scale, KS, VS, msl, out, lse=lse, traj_ids=tid,
                                       seq_lens_out=lens_out)
            lens1[tid.long()] = lens_out[tid.long()]
        else:
            ctx.kv_append_fp8(dk, dv, table, lens0, dev_i32(np.arange(len(ids) + 1), cuda_device), kn, vn, KS, VS, traj_ids=tid,
                              seq_lens_out=lens1)
            ctx.decode_attn_fp8(dk, dv, table, lens1, q, spec.sm_scale, KS, VS, msl, out, lse=lse, traj_ids=tid)
        ctx.check()
        res.append((dk, dv, lens1, out, lse))
    a, b = res
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]), "pool bytes differ"
    assert torch.equal(a[2][tid.long()], b[2][tid.long()])
    assert torch.equal(a[3].view(torch.int16), b[3].view(torch.int16)) and torch.equal(a[4], b[4])
    ctx.close()


def test_host_side_validation(cuda_device):
    spec = W.CONFIGS[0]
    b = W.make_batch(spec)
    ctx = make_ctx(spec, spec.num_traj, 600)
    k8 = torch.zeros(tuple(b.k_pool.shape), dtype=torch.uint8, device=cuda_device)
    table, lens = dev_i32(b.page_table, cuda_device), dev_i32(b.seq_lens_before, cuda_device)
    q = b.q_new.to(cuda_device)
    out = torch.empty_like(q)
    for ks, vs in [(0.0, 1.0), (1.0, -1.0), (float("inf"), 1.0), (float("nan"), 1.0)]:
        with pytest.raises(rollart.RollartError):
            ctx.decode_attn_fp8(k8, k8, table, lens, q, spec.sm_scale, ks, vs, 600, out)
        with pytest.raises(rollart.RollartError):
            ctx.kv_append_fp8(k8, k8, table, lens, dev_i32(b.new_indptr, cuda_device), b.k_new.to(cuda_device),
                              b.v_new.to(cuda_device), ks, vs)
    with pytest.raises(ValueError):
        ctx.decode_attn_fp8(b.k_pool.to(cuda_device), b.v_pool.to(cuda_device), table, lens, q, spec.sm_scale, 1.0, 1.0, 600, out)
    ctx.close()


@pytest.mark.parametrize("i,T,div", [(0, 4, 1), (3, 3, 32), (4, 9, 16)])
def test_hand_over_of_an_fp8_cache(cuda_device, i, T, div):
    """gather the codes of whole trajectories, append them onto another worker's pool: every byte against the oracle,
    and decode attention over the received cache equals decode attention over the sender's."""
    batch = W.make_batch(W.shrink(W.CONFIGS[i], T, div, 8), seed=600 + i)
    spec = batch.spec
    P, H = spec.page_size, spec.num_kv_heads
    k8 = oracle.fp8_quantize_rows(W.bf16_to_u16(batch.k_pool), KS)
    v8 = oracle.fp8_quantize_rows(W.bf16_to_u16(batch.v_pool), VS)
    dk, dv = torch.from_numpy(k8.copy()).to(cuda_device), torch.from_numpy(v8.copy()).to(cuda_device)
    table, lens0 = dev_i32(batch.page_table, cuda_device), dev_i32(batch.seq_lens_before, cuda_device)
    ctx = make_ctx(spec, T, int(batch.seq_lens_before.max()) + 1)
    ids = np.array(sorted(range(T), key=lambda t: -t)[: max(2, T - 1)], np.int32)      # a subset in reverse order
    lens = batch.seq_lens_before[ids]
    indptr = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    total = int(indptr[-1])
    k_out = torch.full((total, H, 128), 0xEE, dtype=torch.uint8, device=cuda_device)
    v_out = torch.full_like(k_out, 0xEE)
    ctx.kv_gather_fp8(dk, dv, table, lens0, dev_i32(indptr, cuda_device), k_out, v_out, traj_ids=dev_i32(ids, cuda_device))
    ctx.check()
    ko, vo = oracle.kv_gather_fp8(k8, v8, batch.page_table, batch.seq_lens_before, indptr, traj_ids=ids)
    assert np.array_equal(k_out.cpu().numpy(), ko) and np.array_equal(v_out.cpu().numpy(), vo)
    # the receiving worker: empty trajectories on their own pages, pool bytes poisoned
    pages = (lens.astype(np.int64) + P - 1) // P
    table2, num_pages2 = W.build_page_table(pages, 0.25, np.random.default_rng(9))
    k2 = np.full((num_pages2, H, P, 128), 0x7F, np.uint8)
    v2 = np.full((num_pages2, H, P, 128), 0xFF, np.uint8)
    dk2, dv2 = torch.from_numpy(k2.copy()).to(cuda_device), torch.from_numpy(v2.copy()).to(cuda_device)
    zero = dev_i32(np.zeros(len(ids)), cuda_device)
    after = torch.empty_like(zero)
    ctx.kv_append_fp8_codes(dk2, dv2, dev_i32(table2, cuda_device), zero, dev_i32(indptr, cuda_device), k_out, v_out,
                            seq_lens_out=after)
    ctx.check()
    ref_after = oracle.kv_append_fp8_codes(k2, v2, table2, np.zeros(len(ids), np.int32), indptr, ko, vo)
    assert np.array_equal(after.cpu().numpy(), ref_after) and np.array_equal(ref_after, lens)
    assert np.array_equal(dk2.cpu().numpy(), k2) and np.array_equal(dv2.cpu().numpy(), v2)
    # decode over the received cache == decode over the sender's, bit for bit; and both within tolerance of the oracle
    live = np.flatnonzero(lens > 0)
    q = batch.q_new[: len(live)].contiguous().to(cuda_device)
    o1, o2 = torch.full_like(q, float("nan")), torch.full_like(q, float("nan"))
    msl = int(lens.max())
    ctx.decode_attn_fp8(dk, dv, table, lens0, q, spec.sm_scale, KS, VS, msl, o1, traj_ids=dev_i32(ids[live], cuda_device))
    ctx.decode_attn_fp8(dk2, dv2, dev_i32(table2, cuda_device), after, q, spec.sm_scale, KS, VS, msl, o2,
                        traj_ids=dev_i32(live, cuda_device))
    ctx.check()
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))
    ref_o, _ = oracle.decode_attn_fp8(k2, v2, table2, ref_after, W.bf16_to_u16(batch.q_new[: len(live)]), spec.sm_scale, KS, VS,
                                      traj_ids=live.astype(np.int32))
    assert_attn_close(o2, ref_o, spec.name + " fp8 hand-over")
    # asking for more rows than a trajectory holds is reported, not read
    bad = indptr.copy()
    bad[-1] += 1
    big = torch.zeros(total + 1, H, 128, dtype=torch.uint8, device=cuda_device)
    ctx.kv_gather_fp8(dk, dv, table, lens0, dev_i32(bad, cuda_device), big, big.clone(), traj_ids=dev_i32(ids, cuda_device))
    assert ctx.status() == rollart.ERR_BOUNDS and "kv_gather" in ctx.last_error()
    ctx.close()
